// Tree-masked attention for whole runs of consecutive query tokens (prompt prefill, the training
// mask of Section 2.2) on the Blackwell tensor cores, with 128-row tiles.
//
// A unit is up to 256 query rows of one kv head - 2 * (128 / group) consecutive tokens of one
// thread times the group's query heads - and the chain they attend, from its first token to the
// last query's own position.  One persistent CTA per SM claims units from a device counter.
//   warps 0-3 and 4-7  two softmax warpgroups.  Warpgroup w owns the unit's tokens
//              w * (128 / group) onward: its own Q operand in shared memory, its own S
//              (double-buffered) and O accumulators in tensor memory.  Row r of a warpgroup is
//              TMEM lane r, so one thread owns one whole row: the row maximum and sum need no
//              shuffles.  Every row is masked at its own position.  P (bf16) is written over the
//              first half of the S buffer it was made from and read from there by the MMA.
//   warp 8     claims units (one phase of that fetch per tile issued, so that its memory
//              round trips pass in the background) and copies, by TMA, the units' query rows
//              (double-buffered) and their 64-token K tiles into a ring.
//   warp 11    copies the V tiles into a second ring.
//   warps 9, 10  one MMA issuer per warpgroup (lane 0 issues): per K/V tile S = Q K^T (M 128,
//              N 64, K 128) and, one tile behind, O += P V (M 128, N 128, K 64, A operand in
//              tensor memory).  K and V tiles are shared by the two warpgroups: a 32 KiB tile
//              pair feeds 256 query rows.  The first warpgroup's rows end earlier in the chain
//              than the second's; it skips the tiles beyond its last row.
// Why the roles are cut this way (measured, cycles of the SM clock): a tcgen05.mma holds its
// issuing thread until the tensor pipe takes it (M 128 x N 64 x K 16 every 48 cycles, N 128
// every 64), a look at an mbarrier costs a thread 100-250 cycles on a busy SM, and a warp's
// tensor copy instruction about 70 cycles per 2 KiB box.  So two threads issue MMAs (one keeps
// the pipe busy while the other synchronises), each looks at its next step's barriers before
// it needs the answer, and the sixteen boxes of a tile pair are issued by two warps.
// All waits are bounded; a wait that gives up raises the error word and every role unwinds to
// the common exit where TMEM is released.
#include <algorithm>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "apar_internal.h"
#include "ptx.cuh"
#include "tcgen05.cuh"

namespace apar {
namespace {

constexpr int kTile = 64;                          // tokens per K/V stage and per S tile
constexpr int kTileBlk = kTile / kBlock;           // 4 blocks
constexpr int kBlkBytes = kBlock * kDim * 2;       // one block of one kv head: 4 KiB
constexpr int kRowsWg = 128;                       // query rows of a warpgroup
constexpr int kKS = 3, kVS = 3;                    // ring depths
constexpr int kStage = kTile * kDim * 2;           // K (or V) of a stage: 16 KiB
constexpr int kStageHalf = kStage / 2;             // one 64-dim half: [64 rows][128 B]
constexpr int kQBytes = kRowsWg * kDim * 2;        // 32 KiB: [2 halves][128 rows][128 B]
constexpr int kQHalf = kQBytes / 2;
constexpr int kOffV = kKS * kStage;
constexpr int kOffQ = kOffV + kVS * kStage;        // Q: [2 buffers][2 warpgroups]
constexpr int kOffBar = kOffQ + 4 * kQBytes;
constexpr int kOffDesc = kOffBar + 512;
constexpr int kDescRing = 3;
constexpr int kClaimAhead = 8;                     // K tiles before a unit's end at which the next is claimed
constexpr uint32_t kPollLimit = kSpin * 16;        // for the roles that poll without suspending
constexpr float kSlack = 8.f;                      // the reference of a row moves only past 2^8
constexpr int kTmemCols = 512;

struct PrefillUnit {                               // a claimed unit, as the roles read it
  int32_t table_row, chain_tok, n_tiles, kvh;      // n_tiles == 0: no more units
  int32_t q_first, n_q, pos0, tiles_wg0;           // tiles the first warpgroup takes part in
  int32_t ids[64];                                 // first block ids of the chain
};
constexpr int kSmemPrefill = kOffDesc + kDescRing * (int)sizeof(PrefillUnit) + 1024;
static_assert(kSmemPrefill <= 227 * 1024, "shared memory");

enum { B_KFULL = 0, B_KEMPTY = B_KFULL + kKS, B_VFULL = B_KEMPTY + kKS, B_VEMPTY = B_VFULL + kVS,
       B_DFULL = B_VEMPTY + kVS, B_DEMPTY = B_DFULL + kDescRing,
       B_QFULL = B_DEMPTY + kDescRing, B_QEMPTY = B_QFULL + 2,
       B_WG = B_QEMPTY + 2,                        // per warpgroup from here, B_WG_N each
       W_SFULL = 0, W_PFULL = 2, W_PFREE = 4, W_ODONE = 6, B_WG_N = 7,
       B_TOTAL = B_WG + 2 * B_WG_N };
static_assert(8 * B_TOTAL + 16 <= 512, "barrier area");

__device__ __forceinline__ uint32_t kv_off(int row, int c) {  // a 64-token stage
  return (uint32_t)((c >> 3) * kStageHalf + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}

__global__ void __launch_bounds__(384)
attn_prefill_kernel(const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v,
                    const __grid_constant__ CUtensorMap tm_q, const AttnArgs a,
                    const PrefillItem* __restrict__ items, int n_items,
                    int* __restrict__ ticket) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (s32(smem_raw) + 1023u) & ~1023u;
  uint8_t* bp = smem_raw + (base - s32(smem_raw));
  const uint32_t bars = base + kOffBar;
  auto bar = [&](int i) { return bars + 8u * i; };
  auto wbar = [&](int w, int i) { return bars + 8u * (B_WG + w * B_WG_N + i); };
  volatile int* cta_abort = (volatile int*)(bp + kOffBar + 8 * B_TOTAL);
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(bp + kOffBar + 8 * B_TOTAL + 8);
  PrefillUnit* descs = (PrefillUnit*)(bp + kOffDesc);

  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_units = n_items * HKV;
  const int tok_wg = kRowsWg / G;                  // tokens whose rows one warpgroup holds

  if (threadIdx.x == 0) {
    *cta_abort = *(volatile int*)a.d_error;        // an earlier kernel gave up: do not pile up
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_v) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_q) : "memory");
    for (int s = 0; s < kKS; ++s) {
      bar_init(bar(B_KFULL + s), 1);
      bar_init(bar(B_KEMPTY + s), 2);              // both MMA issuers
    }
    for (int s = 0; s < kVS; ++s) {
      bar_init(bar(B_VFULL + s), 1);
      bar_init(bar(B_VEMPTY + s), 2);
    }
    for (int d = 0; d < kDescRing; ++d) {
      bar_init(bar(B_DFULL + d), 1);
      bar_init(bar(B_DEMPTY + d), 11);             // softmax warps, MMA issuers, V producer
    }
    for (int b = 0; b < 2; ++b) {
      bar_init(bar(B_QFULL + b), 1);
      bar_init(bar(B_QEMPTY + b), 2);
    }
    for (int w = 0; w < 2; ++w) {
      for (int b = 0; b < 2; ++b) {
        bar_init(wbar(w, W_SFULL + b), 1);
        bar_init(wbar(w, W_PFULL + b), 4);
        bar_init(wbar(w, W_PFREE + b), 1);
      }
      bar_init(wbar(w, W_ODONE), 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(s32((const void*)tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // TMEM columns of warpgroup w: S buffers at 256 w and 256 w + 64 (the first 32 columns of a
  // buffer take P, as bf16 pairs, once its scores are in registers), O at 256 w + 128
  const bool dead = *cta_abort != 0;

  if (dead) {
    // nothing is claimed; the exit count of the launch stays complete (see the producer's end)
    if (warp == 8 && lane == 0) {
      const int gone = atomicAdd(ticket + 1, 1);
      if (gone == (int)gridDim.x - 1) {
        ticket[0] = 0;
        ticket[1] = 0;
      }
    }
  } else if (warp == 8) {
    // ---------------------------------------------------------------- producer + unit fetch
    // Fetch of the next unit, one phase per call, so that the global-memory round trips of its
    // chain (ticket -> work item -> block ids) pass while K/V tiles are issued.
    int f_phase = 0, f_units = 0;     // descriptions published so far (the end mark included)
    bool f_end = false;
    int f_tick = 0, f_id0 = 0, f_id1 = 0;
    int4 f_item = make_int4(0, 0, 0, 0);
    auto fetch_step = [&](bool may_claim) {
      if (f_phase == 0) {
        if (f_end || !may_claim) return;
        if (lane == 0) f_tick = atomicAdd(ticket, 1);
        f_phase = 1;
      } else if (f_phase == 1) {
        f_tick = __shfl_sync(0xffffffffu, f_tick, 0);
        if (f_tick >= n_units) {
          f_phase = 3;                              // publish the end mark
        } else {
          // The list is walked once per kv head: the units that run at the same time are
          // neighbouring query tiles of one head and find their K and V in the L2 cache.
          if (lane == 0) f_item = __ldg((const int4*)items + f_tick % n_items);
          f_phase = 2;
        }
      } else if (f_phase == 2) {
        f_item.x = __shfl_sync(0xffffffffu, f_item.x, 0);
        f_item.y = __shfl_sync(0xffffffffu, f_item.y, 0);
        f_item.z = __shfl_sync(0xffffffffu, f_item.z, 0);
        f_item.w = __shfl_sync(0xffffffffu, f_item.w, 0);
        const int32_t* tab = a.d_tables + (size_t)f_item.x * a.shape.table_stride;
        f_id0 = lane < a.shape.table_stride ? tab[lane] : 0;
        f_id1 = lane + 32 < a.shape.table_stride ? tab[lane + 32] : 0;
        f_phase = 3;
      } else {
        const int slot = f_units % kDescRing;
        int ok = f_units < kDescRing ||
                 bar_test(bar(B_DEMPTY + slot), ((f_units / kDescRing) - 1) & 1);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) return;
        PrefillUnit* d = descs + slot;
        if (f_tick >= n_units) {
          if (lane == 0) d->n_tiles = 0;
          f_end = true;
        } else {
          if (lane == 0) {
            const int pos0 = f_item.z, n_q = f_item.w;
            d->table_row = f_item.x;
            d->q_first = f_item.y;
            d->pos0 = pos0;
            d->n_q = n_q;
            d->chain_tok = pos0 + n_q;
            d->n_tiles = (pos0 + n_q + kTile - 1) / kTile;
            d->tiles_wg0 = (pos0 + min(n_q, tok_wg) + kTile - 1) / kTile;
            d->kvh = f_tick / n_items;
          }
          d->ids[lane] = f_id0;
          d->ids[lane + 32] = f_id1;
        }
        __syncwarp();
        if (lane == 0) bar_arrive(bar(B_DFULL + slot));
        ++f_units;
        f_phase = 0;
      }
    };

    // K and V tiles are two independent sequences over the units (a K tile is free again as
    // soon as its Q K^T products are done, a V tile one softmax later), each with its own ring
    // and its own warp: a warp's tensor copy instruction takes some seventy cycles per box, a
    // tile is eight boxes of 2 KiB for K and eight for V, and one warp issuing both could not
    // keep up with the tensor pipe.  This warp copies K; warp 11 copies V.
    struct Cursor {
      int unit = 0, t = 0, n_tiles = 0, n_blk = 0, kvh = 0;   // unit ordinal, tile in the unit
      bool active = false, done = false;
      const int32_t* table = nullptr;
      int id_cur = 0, id_next = 0;
    } kc;
    auto open_unit = [&](Cursor& c) {
      const PrefillUnit* d = descs + c.unit % kDescRing;
      const int n_tiles = d->n_tiles;
      if (n_tiles == 0) {
        c.done = true;
        return;
      }
      c.n_tiles = n_tiles;
      c.n_blk = (d->chain_tok + kBlock - 1) / kBlock;
      c.kvh = d->kvh;
      c.table = a.d_tables + (size_t)d->table_row * a.shape.table_stride;
      c.id_cur = d->ids[lane];
      c.id_next = d->ids[lane + 32];
      c.t = 0;
      c.active = true;
    };
    // Issues tile c.t of the cursor's unit into ring slot (g mod stages) if that slot is free.
    auto issue = [&](Cursor& c, int g, int stages, int empty0, int full0, uint32_t ring,
                     const CUtensorMap* map) -> bool {
      const int s = g % stages;
      int ready = g < stages || bar_test(bar(empty0 + s), ((g / stages) - 1) & 1);
      ready = __shfl_sync(0xffffffffu, ready, 0);
      if (!ready) return false;
      const int t = c.t;
      if (t > 0 && (t & 7) == 0) {                  // 32 block ids last for 8 tiles
        c.id_cur = c.id_next;
        const int nxt = (t + 8) * kTileBlk + lane;
        c.id_next = nxt < c.n_blk ? c.table[nxt] : 0;
      }
      const int blk = t * kTileBlk + (lane >> 1);
      const int bid = __shfl_sync(0xffffffffu, c.id_cur, blk & 31);
      if (lane == 0)
        bar_expect_tx(bar(full0 + s), (uint32_t)min(kTileBlk, c.n_blk - t * kTileBlk) * kBlkBytes);
      __syncwarp();
      if (lane < 2 * kTileBlk && blk < c.n_blk)
        tma_2d(ring + s * kStage + (lane & 1) * kStageHalf + (lane >> 1) * (kBlock * 128), map,
               (lane & 1) * 64, (bid * HKV + c.kvh) * kBlock, bar(full0 + s));
      if (++c.t == c.n_tiles) {
        c.active = false;
        ++c.unit;
      }
      return true;
    };

    // The query rows of a unit: for each warpgroup its tokens x the group's heads, as two
    // 64-dim halves, into the Q buffer the unit's parity selects - as soon as the unit is known
    // and the unit two before it has finished its Q K^T products.
    int qu = 0;                       // units whose rows have been requested
    bool q_done = false;
    auto issue_q = [&]() -> bool {
      const PrefillUnit* d = descs + qu % kDescRing;
      if (d->n_tiles == 0) {
        q_done = true;
        return false;
      }
      const int qb = qu & 1;
      int ready = qu < 2 || bar_test(bar(B_QEMPTY + qb), ((qu >> 1) - 1) & 1);
      ready = __shfl_sync(0xffffffffu, ready, 0);
      if (!ready) return false;
      const uint32_t half_bytes = (uint32_t)(tok_wg * G) * 128u;
      if (lane == 0) bar_expect_tx(bar(B_QFULL + qb), 4u * half_bytes);
      __syncwarp();
      if (lane < 4)
        tma_3d(base + kOffQ + (qb * 2 + (lane >> 1)) * kQBytes + (lane & 1) * kQHalf, &tm_q,
               (lane & 1) * 64, d->kvh * G, d->q_first + (lane >> 1) * tok_wg, bar(B_QFULL + qb));
      ++qu;
      return true;
    };
    int kg = 0;                       // K tiles issued so far, all units
    uint32_t idle = 0;
    for (int i = 0; i < 4 && f_units == 0; ++i) fetch_step(true);   // the first unit at once
    while (!(kc.done && q_done)) {
      bool did = false, did_k = false;
      if (!q_done && qu < f_units && issue_q()) did = true;
      if (!kc.active && !kc.done && kc.unit < f_units) open_unit(kc);
      if (kc.active && issue(kc, kg, kKS, B_KEMPTY, B_KFULL, base, &tm_k)) {
        ++kg;
        did = did_k = true;
      }
      // claim the next unit towards the end of the K stream of the current one (or at once
      // when the K cursor has nothing to do); one phase per tile issued or per idle pass
      const bool near_end = !kc.active || kc.n_tiles - kc.t <= kClaimAhead;
      const bool room = f_units <= kc.unit + (kc.active ? 1 : 0);
      if (did_k || !kc.active) fetch_step(near_end && room);
      if (did) {
        idle = 0;
      } else {
        ++idle;
        int stop = idle > kPollLimit || ((idle & 255) == 0 && *cta_abort);
        if (__shfl_sync(0xffffffffu, stop, 0)) {
          if (lane == 0 && idle > kPollLimit) {
            *cta_abort = 1;
            atomicCAS(a.d_error, 0, 16000 + kg % 1000);
          }
          break;
        }
      }
    }
    // After a wait that gave up, the copies this warp still has in flight are waited for (with
    // a limit of their own) before the CTA's shared memory goes away.  (Otherwise every copy
    // has been consumed: its consumer waited for it.)
    if (*cta_abort && lane == 0) {
      for (int g = max(0, kg - kKS); g < kg; ++g)
        for (uint32_t i = 0; i < kSpin && !bar_try(bar(B_KFULL + g % kKS), (g / kKS) & 1); ++i) {}
      for (int x = max(0, qu - 2); x < qu; ++x)
        for (uint32_t i = 0; i < kSpin && !bar_try(bar(B_QFULL + (x & 1)), (x >> 1) & 1); ++i) {}
    }
    // ticket[0] unit counter, ticket[1] producers that have stopped claiming: the last one puts
    // both back to zero, so that nothing has to be cleared between launches
    if (lane == 0) {
      const int gone = atomicAdd(ticket + 1, 1);
      if (gone == (int)gridDim.x - 1) {
        ticket[0] = 0;
        ticket[1] = 0;
      }
    }
  } else if (warp == 11) {
    // ---------------------------------------------------------------- V producer
    int vg = 0;                       // V tiles issued so far, all units
    bool ok = true;
    for (int u = 0; ok; ++u) {
      const int ds = u % kDescRing;
      ok = __all_sync(0xffffffffu, bar_wait(bar(B_DFULL + ds), (u / kDescRing) & 1, cta_abort,
                                            a.d_error, 18000));
      if (!ok) break;
      const PrefillUnit* d = descs + ds;
      const int n_tiles = __shfl_sync(0xffffffffu, d->n_tiles, 0);
      if (n_tiles == 0) break;
      const int n_blk = (__shfl_sync(0xffffffffu, d->chain_tok, 0) + kBlock - 1) / kBlock;
      const int kvh = __shfl_sync(0xffffffffu, d->kvh, 0);
      const int32_t* table =
          a.d_tables + (size_t)__shfl_sync(0xffffffffu, d->table_row, 0) * a.shape.table_stride;
      int id_cur = d->ids[lane], id_next = d->ids[lane + 32];
      __syncwarp();
      if (lane == 0) bar_arrive(bar(B_DEMPTY + ds));   // what it needs of the description is copied
      for (int t = 0; t < n_tiles; ++t, ++vg) {
        const int s = vg % kVS;
        if (vg >= kVS) {
          ok = __all_sync(0xffffffffu, bar_wait(bar(B_VEMPTY + s), ((vg / kVS) - 1) & 1, cta_abort,
                                                a.d_error, 18100));
          if (!ok) break;
        }
        if (t > 0 && (t & 7) == 0) {                // 32 block ids last for 8 tiles
          id_cur = id_next;
          const int nxt = (t + 8) * kTileBlk + lane;
          id_next = nxt < n_blk ? table[nxt] : 0;
        }
        const int blk = t * kTileBlk + (lane >> 1);
        const int bid = __shfl_sync(0xffffffffu, id_cur, blk & 31);
        if (lane == 0)
          bar_expect_tx(bar(B_VFULL + s), (uint32_t)min(kTileBlk, n_blk - t * kTileBlk) * kBlkBytes);
        __syncwarp();
        if (lane < 2 * kTileBlk && blk < n_blk)
          tma_2d(base + kOffV + s * kStage + (lane & 1) * kStageHalf + (lane >> 1) * (kBlock * 128),
                 &tm_v, (lane & 1) * 64, (bid * HKV + kvh) * kBlock, bar(B_VFULL + s));
      }
    }
    if (*cta_abort && lane == 0)      // (as in the K producer: copies in flight after a give-up)
      for (int g = max(0, vg - kVS); g < vg; ++g)
        for (uint32_t i = 0; i < kSpin && !bar_try(bar(B_VFULL + g % kVS), (g / kVS) & 1); ++i) {}
  } else if (warp >= 9) {
    // ---------------------------------------------------------------- MMA issuers
    // One warp per warpgroup of query rows (warp 9: the first, warp 10: the second), each with
    // warp-uniform control flow and lane 0 issuing.  A tcgen05.mma occupies its issuing thread
    // until the tensor pipe takes it, and a look at a barrier takes that thread more than a
    // hundred cycles: with two issuers, one's products keep the pipe busy while the other
    // synchronises.  Per K/V tile j an issuer issues S = Q K^T of tile j, then O += P V of
    // tile j - 1, so that the pipe computes the next scores while the softmax warps are at
    // work on the last ones.  MMAs of one thread execute in issue order: Q K^T of tile j + 2
    // overwrites the S buffer that held P of tile j after P V of tile j has read it.
    constexpr uint32_t kIdescQK = instr_desc(kTile, false, kRowsWg);
    constexpr uint32_t kIdescPV = instr_desc(kDim, true, kRowsWg);
    constexpr unsigned kAll = 0xffffffffu;
    const int w = warp - 9;
    const bool lead = lane == 0;
    const uint32_t tm_w = tmem + 256u * w;
    int j = 0;                                  // K/V tiles so far, all units
    int qg = 0, pg = 0;                         // S tiles / P V products issued by this warp
    int pv_j = -1, pv_t = 0, pv_tok = 0, pv_unit = 0;   // the P V that is due
    bool pv_last = false;
    bool ok = true;
    bool k_seen = false;                        // tile j's K was there at the last look
    auto look_pv = [&]() -> bool {              // what the due P V waits for, looked at now
      bool r = bar_test(wbar(w, W_PFULL + (pg & 1)), (pg >> 1) & 1);
      r = r && bar_test(bar(B_VFULL + pv_j % kVS), (pv_j / kVS) & 1);
      if (pv_t == 0 && pv_unit > 0) r = r && bar_test(wbar(w, W_ODONE), (pv_unit - 1) & 1);
      return r;
    };
    auto do_pv = [&](bool seen) -> bool {
      const int vs = pv_j % kVS;
      const uint32_t vb = base + kOffV + vs * kStage;
      const int nk = min(kTileBlk, (pv_tok - pv_t * kTile + kBlock - 1) / kBlock);
      if (!__all_sync(kAll, seen)) {
        bool w8 = bar_wait(wbar(w, W_PFULL + (pg & 1)), (pg >> 1) & 1, cta_abort, a.d_error,
                           17300 + w);
        w8 = w8 && bar_wait(bar(B_VFULL + vs), (pv_j / kVS) & 1, cta_abort, a.d_error, 17200 + w);
        if (pv_t == 0 && pv_unit > 0)           // the unit before has read its O out
          w8 = w8 && bar_wait(wbar(w, W_ODONE), (pv_unit - 1) & 1, cta_abort, a.d_error, 17400 + w);
        if (!__all_sync(kAll, w8)) return false;
      }
      tc_fence_after();
      if (lead) {
        // operands are formed once per tile; inside the unrolled loop only constants are added
        const uint64_t vd = smem_desc(vb, kStageHalf, 1024);
        const uint32_t p = tm_w + 64u * (pg & 1);
        const uint32_t acc0 = pv_t != 0;
        if (nk == kTileBlk) {
#pragma unroll
          for (int kk = 0; kk < kTileBlk; ++kk)
            umma_bf16_ts(tm_w + 128u, p + 8u * kk, vd + (uint64_t)(kk * (kBlock * 128) >> 4),
                         kIdescPV, kk ? 1u : acc0);
        } else {
          for (int kk = 0; kk < nk; ++kk)
            umma_bf16_ts(tm_w + 128u, p + 8u * kk, vd + (uint64_t)(kk * (kBlock * 128) >> 4),
                         kIdescPV, kk ? 1u : acc0);
        }
        umma_commit(wbar(w, W_PFREE + (pg & 1)));
        umma_commit(bar(B_VEMPTY + vs));        // this warpgroup is done with the V tile
        if (pv_last) bar_arrive(bar(B_DEMPTY + pv_unit % kDescRing));
      }
      ++pg;
      // (a look at the next tile's K, for the next step: the products just issued run while
      // the answer comes)
      k_seen = bar_test(bar(B_KFULL + (pv_j + 2) % kKS), ((pv_j + 2) / kKS) & 1);
      return true;
    };
    for (int u = 0; ok; ++u) {
      const int ds = u % kDescRing;
      ok = __all_sync(kAll, bar_wait(bar(B_DFULL + ds), (u / kDescRing) & 1, cta_abort, a.d_error,
                                     17000));
      if (!ok) break;
      const PrefillUnit* d = descs + ds;
      const int n_tiles = __shfl_sync(kAll, d->n_tiles, 0);
      if (n_tiles == 0) break;
      const int my_tiles = w == 0 ? __shfl_sync(kAll, d->tiles_wg0, 0) : n_tiles;
      const int chain_tok = __shfl_sync(kAll, d->chain_tok, 0);
      const uint64_t qd = smem_desc(base + kOffQ + ((u & 1) * 2 + w) * kQBytes, 16, 1024);
      for (int t = 0; t < n_tiles; ++t, ++j) {
        const int s = j % kKS;
        if (t >= my_tiles) {
          // beyond this warpgroup's last row: the P V that is still due, and the tile is let go
          if (pv_j >= 0 && !do_pv(false)) {
            ok = false;
            break;
          }
          pv_j = -1;
          k_seen = false;
          // (the tile's copies have been requested, so the releases before these of the two
          // stages are complete: these arrivals cannot be counted for them)
          if (!__all_sync(kAll, bar_wait(bar(B_KFULL + s), (j / kKS) & 1, cta_abort, a.d_error,
                                         17600) &&
                                    bar_wait(bar(B_VFULL + j % kVS), (j / kVS) & 1, cta_abort,
                                             a.d_error, 17601))) {
            ok = false;
            break;
          }
          if (lead) {
            bar_arrive(bar(B_KEMPTY + s));
            bar_arrive(bar(B_VEMPTY + j % kVS));
          }
          continue;
        }
        if (!__all_sync(kAll, k_seen) || t == 0) {
          bool w8 = bar_wait(bar(B_KFULL + s), (j / kKS) & 1, cta_abort, a.d_error, 17100);
          if (t == 0)
            w8 = w8 && bar_wait(bar(B_QFULL + (u & 1)), (u >> 1) & 1, cta_abort, a.d_error, 17500);
          if (!__all_sync(kAll, w8)) {
            ok = false;
            break;
          }
        }
        k_seen = false;
        tc_fence_after();
        if (lead) {
          const uint64_t kd = smem_desc(base + s * kStage, 16, 1024);
          const uint32_t sd = tm_w + 64u * (qg & 1);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            umma_bf16(sd, qd + (uint64_t)(((ks >> 2) * kQHalf + (ks & 3) * 32) >> 4),
                      kd + (uint64_t)(((ks >> 2) * kStageHalf + (ks & 3) * 32) >> 4), kIdescQK,
                      ks > 0);
          umma_commit(wbar(w, W_SFULL + (qg & 1)));
          umma_commit(bar(B_KEMPTY + s));         // this warpgroup is done with the K tile
          if (t == my_tiles - 1) umma_commit(bar(B_QEMPTY + (u & 1)));   // done with the unit's rows
        }
        ++qg;
        if (pv_j >= 0) {
          const bool seen = look_pv();          // (answers while the products above run)
          if (!do_pv(seen)) {
            ok = false;
            break;
          }
        }
        pv_j = j;
        pv_t = t;
        pv_tok = chain_tok;
        pv_unit = u;
        pv_last = t == my_tiles - 1;
      }
    }
    if (ok && pv_j >= 0) do_pv(false);
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- softmax warpgroups
    const int w = warp >> 2, wq = warp & 3;
    const int row = wq * 32 + lane;                    // this thread's row = its TMEM lane
    const uint32_t lane_sel = (uint32_t)(wq * 32) << 16;
    const uint32_t tm_s = tmem + 256u * w, tm_o = tmem + 256u * w + 128u;
    const float c = a.scale_log2e;
    const float cc = c > 0.f ? c : 1.f;                // what is left to apply inside the exponent
    bool alive = true;
    int gw = 0, all0 = 0;             // S tiles of this warpgroup / tiles of all earlier units
    for (int u = 0; alive; ++u) {
      const PrefillUnit* d = descs + u % kDescRing;
      if (!bar_wait(bar(B_DFULL + u % kDescRing), (u / kDescRing) & 1, cta_abort, a.d_error,
                    11000 + u % 1000))
        break;
      const int n_tiles = d->n_tiles;
      if (n_tiles == 0) break;
      const int my_tiles = w == 0 ? d->tiles_wg0 : n_tiles, chain_tok = d->chain_tok;
      // this thread's row: token row / group of the warpgroup's tokens, head row % group of the
      // kv head's group; rows past the unit's own are padding (they see every key, their
      // result is dropped)
      const int R = max(0, min(tok_wg, d->n_q - w * tok_wg)) * G;
      const int lim = row < R ? d->pos0 + w * tok_wg + row / G + 1 : chain_tok;
      const long long out_row =
          row < R ? ((long long)d->q_first + w * tok_wg + row / G) * HQ + d->kvh * G + row % G : -1;
      float ref = -INFINITY, l = 0.f;
      for (int t = 0; t < my_tiles; ++t) {
        const int g = gw + t, b = g & 1;
        if (!bar_wait(wbar(w, W_SFULL + b), (g >> 1) & 1, cta_abort, a.d_error, 12000 + t % 1000)) {
          alive = false;
          break;
        }
        tc_fence_after();
        uint32_t sr[64];
        TMEM_LD_32((tm_s + 64u * b) | lane_sel, sr, 0);
        TMEM_LD_32((tm_s + 64u * b + 32u) | lane_sel, sr, 32);
        tmem_wait_ld();
        // The raw scores stay in registers; the scale is applied to the row maximum and, fused
        // with the subtraction of the reference, inside the exponent.  A key the row may not
        // see becomes -inf (rows of K past the chain's end hold unspecified bits); tiles that
        // every row of the warp sees in full skip that pass.  (A scale that is not positive is
        // applied up front, so that the maximum of the raw values is the maximum.)
        if (!(c > 0.f)) {
#pragma unroll
          for (int j = 0; j < 64; ++j) sr[j] = __float_as_uint(__uint_as_float(sr[j]) * c);
        }
        const int see = lim - t * kTile;
        if (!__all_sync(0xffffffffu, see >= kTile)) {
#pragma unroll
          for (int j = 0; j < 64; ++j)
            if (j >= see) sr[j] = 0xff800000u;
        }
        // (four independent chains: one chain of 64 would wait for itself)
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 64; j += 8) {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            mx4[e] = fmaxf(mx4[e], fmaxf(__uint_as_float(sr[j + 2 * e]),
                                         __uint_as_float(sr[j + 2 * e + 1])));
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * cc;
        const bool move = mx > ref + kSlack || ref == -INFINITY;
        const float ref_new = move ? mx : ref;
        const bool rescale = t > 0 && __any_sync(0xffffffffu, move);
        if (rescale) {
          // (P V of tile g - 1 has to be complete; that of tile g - 3, which used the same
          // barrier, is: this tile's scores came after it)
          if (!bar_wait(wbar(w, W_PFREE + ((g - 1) & 1)), ((g - 1) >> 1) & 1, cta_abort, a.d_error,
                        13000 + t % 1000)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const float f = move ? ex2(ref - ref_new) : 1.f;
          l *= f;
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t orow[32];
            TMEM_LD_32((tm_o + 32u * q4) | lane_sel, orow, 0);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) orow[j] = __float_as_uint(__uint_as_float(orow[j]) * f);
            TMEM_ST_32((tm_o + 32u * q4) | lane_sel, orow);
          }
          tmem_wait_st();
          tc_fence_before();
        }
        ref = ref_new;
        uint32_t pk[32];
        float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float p0 = ex2(fmaf(__uint_as_float(sr[2 * j]), cc, -ref));
          const float p1 = ex2(fmaf(__uint_as_float(sr[2 * j + 1]), cc, -ref));
          l4[j & 3] += p0 + p1;
          pk[j] = pack2(p0, p1);
        }
        l += (l4[0] + l4[1]) + (l4[2] + l4[3]);
        // P takes the place of the scores it was made from
        TMEM_ST_32((tm_s + 64u * b) | lane_sel, pk);
        tmem_wait_st();
        // The chain's last block, where it is not full: its rows past the end are cleared in the
        // V tile (0 x unspecified bits could be NaN).  Both warpgroups do it when both take
        // the unit's last tile: each before its own P is handed over.
        const int tile_tok = chain_tok - t * kTile;
        if (tile_tok < kTile && wq == 0) {
          const int vt = all0 + t, vs = vt % kVS;
          if (!bar_wait(bar(B_VFULL + vs), (vt / kVS) & 1, cta_abort, a.d_error, 14000 + t % 1000)) {
            alive = false;
            break;
          }
          uint8_t* vptr = bp + kOffV + vs * kStage;
          const int last = ((tile_tok + kBlock - 1) / kBlock) * kBlock;
          for (int x = lane; x < (last - tile_tok) * 16; x += 32)
            *(uint4*)(vptr + kv_off(tile_tok + (x >> 4), x & 15)) = make_uint4(0u, 0u, 0u, 0u);
          fence_async_smem();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) bar_arrive(wbar(w, W_PFULL + b));
      }
      if (!alive) break;
      {
        const int gl = gw + my_tiles - 1;            // this warpgroup's last product of the unit
        if (!bar_wait(wbar(w, W_PFREE + (gl & 1)), (gl >> 1) & 1, cta_abort, a.d_error, 15000)) break;
      }
      tc_fence_after();
      {
        const float inv = 1.f / l;
        uint4* dst = (uint4*)((__nv_bfloat16*)a.out + out_row * kDim);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t orow[32];
          TMEM_LD_32((tm_o + 32u * q4) | lane_sel, orow, 0);
          tmem_wait_ld();
          if (out_row >= 0) {
#pragma unroll
            for (int j = 0; j < 32; j += 8)
              dst[4 * q4 + (j >> 3)] = make_uint4(
                  pack2(__uint_as_float(orow[j]) * inv, __uint_as_float(orow[j + 1]) * inv),
                  pack2(__uint_as_float(orow[j + 2]) * inv, __uint_as_float(orow[j + 3]) * inv),
                  pack2(__uint_as_float(orow[j + 4]) * inv, __uint_as_float(orow[j + 5]) * inv),
                  pack2(__uint_as_float(orow[j + 6]) * inv, __uint_as_float(orow[j + 7]) * inv));
          }
        }
      }
      // O has been read and this unit's description is no longer needed by this warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        bar_arrive(wbar(w, W_ODONE));
        bar_arrive(bar(B_DEMPTY + u % kDescRing));
      }
      gw += my_tiles;
      all0 += n_tiles;
    }
  }
  // ---- common exit: every role arrives here, then the allocating warp frees TMEM
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem),
                 "r"(kTmemCols) : "memory");
  }
}

}  // namespace

cudaError_t launch_attention_prefill(const AttnArgs& a, const CUtensorMap* tm_q,
                                     const PrefillItem* d_items, int n_items, cudaStream_t st) {
  if (n_items <= 0) return cudaSuccess;
  if (a.d_ticket == nullptr || tm_q == nullptr || a.shape.group > kRowsWg) return cudaErrorInvalidValue;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_prefill_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPrefill);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const long long n_units = (long long)n_items * a.shape.num_kv_heads;
  const int grid = (int)std::min<long long>(n_units, a.num_sms);
  return launch_kernel(attn_prefill_kernel, dim3(grid), dim3(384), kSmemPrefill, st, false, *a.tm_k,
                       *a.tm_v, *tm_q, a, d_items, n_items, a.d_ticket);
}

}  // namespace apar

// Blackwell tensor-core attention path (tcgen05 + TMEM) for work items with many query rows:
// a run of blocks shared by up to 64 (query, head) rows.
//
// One CTA owns one work item and one kv head of it, or a few consecutive kv heads that it works
// through back to back.  Roles:
//   warps 0-3  softmax: warp w owns query rows 16w .. 16w+15, which are TMEM lanes 32w .. 32w+15
//              of an M = 64 accumulator.  S is read with the 16-lane x 256-bit TMEM load, which
//              spreads a row over the four threads of a quad, so that all 32 lanes work; they
//              keep the running reference maximum and the row sum, write P = exp2(S - ref) as
//              bf16 into shared memory in the K-major 128-byte-swizzled operand layout, rescale
//              O in TMEM in the rare case the reference has to move, and write the results at
//              the end (O rows are read back one row per thread, lanes 0-15).
//   warp 4     producer: walks the block table, TMA tensor copies of 16-token K/V tiles into
//              two rings of 64-token stages - K (two deep, released as soon as Q K^T has
//              read it) and V (three deep, released after P V) - same tile layout as the
//              mma.sync path.
//   warp 5     one elected thread issues S = Q K^T (M 64, N 64, K 128 as 8 MMAs) into one of two
//              S buffers and O += P V (M 64, N 128, K 64 as 4 MMAs) with tcgen05.mma, and
//              signals completion with tcgen05.commit on mbarriers.  Owns the TMEM allocation.
// All waits are bounded; a wait that gives up raises an error word and every role unwinds to
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

constexpr int kTileTok = 64;                       // tokens per stage and per S tile
constexpr int kTileBlocks = kTileTok / kBlock;     // 4
constexpr int kKStages = 2, kVStages = 3;
constexpr int kHalf = kTileTok * 128;              // one 64-dim half of 64 rows: 8 KiB
constexpr int kKV = 2 * kHalf;                     // K (or V) of a stage: 16 KiB
constexpr int kVOff = kKStages * kKV;              // V ring after the K ring
constexpr int kQOff = kVOff + kVStages * kKV;      // Q operand: [2 halves][64 rows][64 dims]
constexpr int kPOff = kQOff + kKV;                 // P operand: [64 rows][64 tokens]
constexpr int kBarOff = kPOff + kHalf;
constexpr int kUserOff = kBarOff + 256;             // the item's UserRef entries (at most 64)
constexpr int kSmem = kUserOff + 64 * 8 + 1024;
constexpr int kTmemCols = 256;                     // S0 | S1 | O
constexpr int kWavesMin = 6, kHeadsMax = 2;        // see launch_attention_umma
constexpr float kRefSlack = 8.f;                   // P stays below 2^8 before the reference moves

enum Bar { KFULL0 = 0, KEMPTY0 = KFULL0 + kKStages, VFULL0 = KEMPTY0 + kKStages,
           VEMPTY0 = VFULL0 + kVStages, SFULL0 = VEMPTY0 + kVStages, SFREE0 = SFULL0 + 2,
           PFULL = SFREE0 + 2, PFREE, QFULL, ODONE, NBARS };

__device__ __forceinline__ uint32_t swz_off(int row, int c) {   // as in the mma.sync path
  return (uint32_t)((c >> 3) * kHalf + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}
// One CTA owns one work item and `heads_per_cta` consecutive kv heads of it, which it works
// through one after the other.  All of them share the item's block table, token range and
// users; only the Q rows and the output rows differ.  The mbarrier phases run on across the
// heads (tile g = head ordinal x tiles per head + tile), so that the producer and the MMA
// thread run ahead into the next head while the softmax warps write out the current one: the
// start-up and write-out latencies, which dominate short items, are hidden for all heads of
// a CTA but the first and the last.
__global__ void __launch_bounds__(192, 2)
attn_umma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const AttnArgs a, int item_begin, int heads_per_cta) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (s32(smem_raw) + 1023u) & ~1023u;
  uint8_t* bp = smem_raw + (base - s32(smem_raw));
  const uint32_t bars = base + kBarOff;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile int* cta_abort = (volatile int*)(bp + kBarOff + 8 * NBARS);
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(bp + kBarOff + 8 * NBARS + 8);

  const WorkItem it = a.d_items[item_begin + blockIdx.x];
  const int U = heads_per_cta, kvh0 = blockIdx.y * U;
  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  const int tok_end = it.tok_end < 0 ? a.d_lens[it.table_row] : it.tok_end;
  const int n_tok = tok_end - it.tok_begin;
  const int n_blk = (n_tok + kBlock - 1) / kBlock;
  const int n_tiles = (n_tok + kTileTok - 1) / kTileTok;
  const int total = U * n_tiles;                   // tiles of the whole CTA
  const int32_t* table = a.d_tables + (size_t)it.table_row * a.shape.table_stride +
                         it.tok_begin / kBlock;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int R = it.n_users * G;
  const int n_active = (R + 15) >> 4;              // softmax warps that own real rows
  UserRef* s_users = (UserRef*)(bp + kUserOff);

  // Everything that only needs the item is started before the one CTA-wide barrier of the
  // prologue, so that these latencies overlap: descriptor prefetch, barrier init, TMEM
  // allocation, the first block ids (producer), the item's users (softmax warps).
  if (threadIdx.x == 0) {
    // an earlier CTA gave up a wait: do not pile up (one reader, so the whole CTA agrees)
    *cta_abort = *(volatile int*)a.d_error;
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_v) : "memory");
    for (int s = 0; s < kKStages; ++s) {
      bar_init(bar(KFULL0 + s), 1);
      bar_init(bar(KEMPTY0 + s), 1);
    }
    for (int s = 0; s < kVStages; ++s) {
      bar_init(bar(VFULL0 + s), 1);
      bar_init(bar(VEMPTY0 + s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      bar_init(bar(SFULL0 + b), 1);
      bar_init(bar(SFREE0 + b), n_active);
    }
    bar_init(bar(PFULL), n_active);
    bar_init(bar(PFREE), 1);
    bar_init(bar(QFULL), n_active);
    bar_init(bar(ODONE), n_active);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  int ids0 = 0, ids1 = 0;                          // block ids 0-31 and 32-63 of the run
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(s32((const void*)tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else if (warp == 4) {
    ids0 = lane < n_blk ? table[lane] : 0;
    ids1 = 32 + lane < n_blk ? table[32 + lane] : 0;
  } else {
    if (threadIdx.x < it.n_users) s_users[threadIdx.x] = a.d_users[it.user_begin + threadIdx.x];
    // Q rows of warps without real rows stay zero for the whole CTA
    if (warp >= n_active) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = lane + 32 * k;
        *(uint4*)(bp + kQOff + swz_off(warp * 16 + (i >> 4), i & 15)) = make_uint4(0u, 0u, 0u, 0u);
      }
      fence_async_smem();
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (*cta_abort) {
    if (warp == 5)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem),
                   "r"(kTmemCols) : "memory");
    return;
  }
  const uint32_t tm_o = tmem + 128u;      // S buffer b sits at columns [64 b, 64 b + 64)
  if (threadIdx.x == 0) pdl_launch_dependents();

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    // K and V tiles are two independent sequences over all heads of the CTA; each tile is
    // issued as soon as its ring slot has been released.  Block ids are fetched 32 at a time
    // (eight tiles), one batch ahead; every head walks the same ids again.
    int kid_cur = ids0, vid_cur = ids0, kid_next = ids1, vid_next = ids1;
    int k_next = 0, v_next = 0;             // tiles issued, all heads
    int kt = 0, kh = 0, vt = 0, vh = 0;     // the same as (tile within the head, head ordinal)
    uint32_t idle = 0;
    while (k_next < total || v_next < total) {
      bool did = false;
      if (k_next < total) {
        const int g = k_next, t = kt, s = g % kKStages;
        int ready = g < kKStages || bar_try(bar(KEMPTY0 + s), ((g / kKStages) - 1) & 1);
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (ready) {
          if (t == 0 && kh > 0) {
            kid_cur = ids0;
            kid_next = ids1;
          } else if (t > 0 && (t & 7) == 0) {
            kid_cur = kid_next;
            const int nxt = (t + 8) * kTileBlocks + lane;
            kid_next = nxt < n_blk ? table[nxt] : 0;
          }
          const int blk = t * kTileBlocks + (lane >> 1);
          const int bid = __shfl_sync(0xffffffffu, kid_cur, blk & 31);
          if (lane == 0)
            bar_expect_tx(bar(KFULL0 + s),
                          (uint32_t)min(kTileBlocks, n_blk - t * kTileBlocks) * kTileBytes);
          __syncwarp();
          if (lane < 2 * kTileBlocks && blk < n_blk)
            tma_2d(base + s * kKV + (lane & 1) * kHalf + (lane >> 1) * (kBlock * 128), &tm_k,
                   (lane & 1) * 64, (bid * HKV + kvh0 + kh) * kBlock, bar(KFULL0 + s));
          ++k_next;
          if (++kt == n_tiles) { kt = 0; ++kh; }
          did = true;
        }
      }
      if (v_next < total) {
        const int g = v_next, t = vt, s = g % kVStages;
        int ready = g < kVStages || bar_try(bar(VEMPTY0 + s), ((g / kVStages) - 1) & 1);
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (ready) {
          if (t == 0 && vh > 0) {
            vid_cur = ids0;
            vid_next = ids1;
          } else if (t > 0 && (t & 7) == 0) {
            vid_cur = vid_next;
            const int nxt = (t + 8) * kTileBlocks + lane;
            vid_next = nxt < n_blk ? table[nxt] : 0;
          }
          const int blk = t * kTileBlocks + (lane >> 1);
          const int bid = __shfl_sync(0xffffffffu, vid_cur, blk & 31);
          if (lane == 0)
            bar_expect_tx(bar(VFULL0 + s),
                          (uint32_t)min(kTileBlocks, n_blk - t * kTileBlocks) * kTileBytes);
          __syncwarp();
          if (lane < 2 * kTileBlocks && blk < n_blk)
            tma_2d(base + kVOff + s * kKV + (lane & 1) * kHalf + (lane >> 1) * (kBlock * 128),
                   &tm_v, (lane & 1) * 64, (bid * HKV + kvh0 + vh) * kBlock, bar(VFULL0 + s));
          ++v_next;
          if (++vt == n_tiles) { vt = 0; ++vh; }
          did = true;
        }
      }
      if (did) {
        idle = 0;
      } else {
        ++idle;
        int stop = idle > kSpin || ((idle & 255) == 0 && *cta_abort);
        if (__shfl_sync(0xffffffffu, stop, 0)) {
          if (lane == 0 && idle > kSpin) {
            *cta_abort = 1;
            atomicCAS(a.d_error, 0, 6000 + (k_next % 25) * 40 + v_next % 40);
          }
          break;
        }
      }
    }
    // After a wait that gave up, the copies still in flight are waited for (with a limit of
    // their own) before the CTA's shared memory goes away.
    if (*cta_abort && lane == 0) {
      for (int g = max(0, k_next - kKStages); g < k_next; ++g)
        for (uint32_t i = 0; i < kSpin && !bar_try(bar(KFULL0 + g % kKStages), (g / kKStages) & 1); ++i) {}
      for (int g = max(0, v_next - kVStages); g < v_next; ++g)
        for (uint32_t i = 0; i < kSpin && !bar_try(bar(VFULL0 + g % kVStages), (g / kVStages) & 1); ++i) {}
    }
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issuer
    constexpr uint32_t kIdescQK = instr_desc(kTileTok, false);
    constexpr uint32_t kIdescPV = instr_desc(kDim, true);
    // One thread issues everything.  It polls for whichever step can go next - Q K^T of the
    // next tile as soon as its K has landed, an S buffer is free and (first tile of a head) the
    // head's Q is staged; P V of the oldest pending tile as soon as the softmax warps have
    // published P and (first tile of a head) drained the previous head's O - so that neither
    // waits for the other.
    if (lane == 0) {
      int qk_next = 0, pv_next = 0;         // tiles issued, all heads
      int qt = 0, qh = 0, pt = 0, ph = 0;   // the same as (tile within the head, head ordinal)
      uint32_t idle = 0;
      while (pv_next < total) {
        bool did = false;
        if (qk_next < total) {
          const int g = qk_next, s = g % kKStages, b = g & 1;
          if (bar_try(bar(KFULL0 + s), (g / kKStages) & 1) &&
              (g < 2 || bar_try(bar(SFREE0 + b), ((g >> 1) - 1) & 1)) &&
              (qt > 0 || bar_try(bar(QFULL), qh & 1))) {
            tc_fence_after();
            const uint32_t kb = base + s * kKV, qb = base + kQOff;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t off = (ks >> 2) * kHalf + (ks & 3) * 32;
              umma_bf16(tmem + 64u * b, smem_desc(qb + off, 16, 1024),
                        smem_desc(kb + off, 16, 1024), kIdescQK, ks > 0);
            }
            umma_commit(bar(SFULL0 + b));
            umma_commit(bar(KEMPTY0 + s));
            ++qk_next;
            if (++qt == n_tiles) { qt = 0; ++qh; }
            did = true;
          }
        }
        if (pv_next < qk_next) {
          const int g = pv_next, s = g % kVStages;
          if (bar_try(bar(PFULL), g & 1) && bar_try(bar(VFULL0 + s), (g / kVStages) & 1) &&
              (pt > 0 || ph == 0 || bar_try(bar(ODONE), (ph - 1) & 1))) {
            tc_fence_after();
            const uint32_t vb = base + kVOff + s * kKV, pb = base + kPOff;
            // blocks past the end of the item were never loaded: leave their k-steps out
            const int nk = min(kTileBlocks, (n_tok - pt * kTileTok + kBlock - 1) / kBlock);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              if (kk < nk)
                umma_bf16(tm_o, smem_desc(pb + kk * 32, 16, 1024),
                          smem_desc(vb + kk * (kBlock * 128), kHalf, 1024), kIdescPV,
                          (pt | kk) != 0);
            umma_commit(bar(PFREE));
            umma_commit(bar(VEMPTY0 + s));
            ++pv_next;
            if (++pt == n_tiles) { pt = 0; ++ph; }
            did = true;
          }
        }
        if (did) {
          idle = 0;
        } else if (++idle > kSpin || ((idle & 255) == 0 && *cta_abort)) {
          if (idle > kSpin) atomicCAS(a.d_error, 0, 7000 + (qk_next % 25) * 40 + pv_next % 40);
          *cta_abort = 1;
          break;
        }
      }
    }
    __syncwarp();
  } else if (warp < n_active) {
    // ---------------------------------------------------------------- softmax warps 0-3
    // Warp w owns query rows 16w .. 16w+15 of every head: it stages them into the A-operand
    // layout (rows past R as zeros), runs their softmax and writes their results.
    auto stage_q = [&](int kvh) {
      // all eight loads of a thread are issued before the first store, so that their
      // latencies overlap
      uint4 qv[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = lane + 32 * k, row = warp * 16 + (i >> 4), c = i & 15;
        qv[k] = make_uint4(0u, 0u, 0u, 0u);
        if (row < R)
          qv[k] = __ldg((const uint4*)a.q +
                        ((size_t)s_users[row / G].query * HQ + kvh * G + row % G) * 16 + c);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = lane + 32 * k;
        *(uint4*)(bp + kQOff + swz_off(warp * 16 + (i >> 4), i & 15)) = qv[k];
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) bar_arrive(bar(QFULL));
    };
    stage_q(kvh0);

    const int row = warp * 16 + (lane & 15);
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    const float c = a.scale_log2e;
    // S is read with the 16-lane x 256-bit TMEM load, which deals a 16 x 64 tile over all 32
    // threads like an MMA accumulator fragment: thread 4g + qd holds, for k = 0..7, columns
    // 8k + 2qd and 8k + 2qd + 1 of row g (registers 4k, 4k + 1) and of row g + 8 (registers
    // 4k + 2, 4k + 3).  A row is thus shared by the four threads of a quad: the maximum is
    // reduced over the quad for every tile, the row sum only once at the end.
    const int g8 = lane >> 2, qd = lane & 3;
    bool alive = true;
    for (int h = 0; h < U && alive; ++h) {
      const int kvh = kvh0 + h;
      const int g0 = h * n_tiles;            // tiles of earlier heads
      float ref_lo = -INFINITY, ref_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
      for (int t = 0; t < n_tiles; ++t) {
        const int g = g0 + t, b = g & 1;
        if (!bar_wait(bar(SFULL0 + b), (g >> 1) & 1, cta_abort, a.d_error, 2000 + t % 1000)) {
          alive = false;
          break;
        }
        tc_fence_after();
        uint32_t sr[32];
        TMEM_LD_16x256((tmem + 64u * b) | lane_sel, sr);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) bar_arrive(bar(SFREE0 + b));
        const int tile_tok = min(kTileTok, n_tok - t * kTileTok);
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const bool in = 8 * k + 2 * qd + e < tile_tok;
            const float x_lo = in ? __uint_as_float(sr[4 * k + e]) * c : -INFINITY;
            const float x_hi = in ? __uint_as_float(sr[4 * k + 2 + e]) * c : -INFINITY;
            sr[4 * k + e] = __float_as_uint(x_lo);
            sr[4 * k + 2 + e] = __float_as_uint(x_hi);
            mx_lo = fmaxf(mx_lo, x_lo);
            mx_hi = fmaxf(mx_hi, x_hi);
          }
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const bool move_lo = mx_lo > ref_lo + kRefSlack || ref_lo == -INFINITY;
        const bool move_hi = mx_hi > ref_hi + kRefSlack || ref_hi == -INFINITY;
        const float new_lo = move_lo ? mx_lo : ref_lo, new_hi = move_hi ? mx_hi : ref_hi;
        const bool rescale = t > 0 && __any_sync(0xffffffffu, move_lo || move_hi);
        if (rescale) {
          // rare: a reference moves, so O (which P V(t-1) still accumulates into) is rescaled,
          // by the thread that owns the whole row in the 32-lane layout (lanes 0-15)
          if (!bar_wait(bar(PFREE), (g - 1) & 1, cta_abort, a.d_error, 3000 + t % 1000)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const float f_lo = move_lo ? ex2(ref_lo - new_lo) : 1.f;
          const float f_hi = move_hi ? ex2(ref_hi - new_hi) : 1.f;
          l_lo *= f_lo;
          l_hi *= f_hi;
          const float fa = __shfl_sync(0xffffffffu, f_lo, 4 * (lane & 7));
          const float fb = __shfl_sync(0xffffffffu, f_hi, 4 * (lane & 7));
          const float f = (lane & 8) ? fb : fa;
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
        ref_lo = new_lo;
        ref_hi = new_hi;
        uint32_t pk_lo[8], pk_hi[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float a0 = ex2(__uint_as_float(sr[4 * k]) - ref_lo);
          const float a1 = ex2(__uint_as_float(sr[4 * k + 1]) - ref_lo);
          const float b0 = ex2(__uint_as_float(sr[4 * k + 2]) - ref_hi);
          const float b1 = ex2(__uint_as_float(sr[4 * k + 3]) - ref_hi);
          l_lo += a0 + a1;
          l_hi += b0 + b1;
          pk_lo[k] = pack2(a0, a1);
          pk_hi[k] = pack2(b0, b1);
        }
        // P(g) overwrites the buffer that the previous P V reads
        if (g > 0 && !rescale &&
            !bar_wait(bar(PFREE), (g - 1) & 1, cta_abort, a.d_error, 3000 + t % 1000)) {
          alive = false;
          break;
        }
        {
          // rows 16w + g and 16w + g + 8 have the same (row & 7), hence the same swizzle
          const int r_lo = warp * 16 + g8;
          uint8_t* p_lo = bp + kPOff + r_lo * 128 + 4 * qd;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int off = (k ^ (r_lo & 7)) << 4;
            *(uint32_t*)(p_lo + off) = pk_lo[k];
            *(uint32_t*)(p_lo + 8 * 128 + off) = pk_hi[k];
          }
        }
        // rows of V past the valid length hold unspecified bits: zero them before P V
        if (tile_tok < kTileTok && warp == 0) {
          const int vs = g % kVStages;
          if (!bar_wait(bar(VFULL0 + vs), (g / kVStages) & 1, cta_abort, a.d_error,
                        4000 + t % 1000)) {
            alive = false;
            break;
          }
          uint8_t* vptr = bp + kVOff + vs * kKV;
          const int first = tile_tok, last = ((tile_tok + kBlock - 1) / kBlock) * kBlock;
          for (int x = lane; x < (last - first) * 16; x += 32)
            *(uint4*)(vptr + swz_off(first + (x >> 4), x & 15)) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) bar_arrive(bar(PFULL));
      }
      if (!alive) break;
      // every Q K^T of this head has completed (this warp has seen its last S tile): the next
      // head's rows can take the Q buffer while the last P V is still running
      if (h + 1 < U) stage_q(kvh + 1);
      if (!bar_wait(bar(PFREE), (g0 + n_tiles - 1) & 1, cta_abort, a.d_error, 5000)) break;
      tc_fence_after();
      // row sums over the quad, then to the lane that writes the row out
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
      const float la = __shfl_sync(0xffffffffu, l_lo, 4 * (lane & 7));
      const float lb = __shfl_sync(0xffffffffu, l_hi, 4 * (lane & 7));
      const float ra = __shfl_sync(0xffffffffu, ref_lo, 4 * (lane & 7));
      const float rb = __shfl_sync(0xffffffffu, ref_hi, 4 * (lane & 7));
      const float l = (lane & 8) ? lb : la, ref = (lane & 8) ? rb : ra;
      // ---- O rows out of TMEM: the thread that owns a row writes it, 32 columns at a time
      {
        const bool mine = lane < 16 && row < R;
        UserRef ur = UserRef{0, -1};
        if (mine) ur = s_users[row / G];
        const int head = kvh * G + row % G;
        const float inv = 1.f / l;
        uint4* dst_out = (uint4*)((__nv_bfloat16*)a.out + ((size_t)ur.query * HQ + head) * kDim);
        const size_t prow = (size_t)(ur.slot + it.slot_add) * HQ + head;
        float4* dst_part = (float4*)(a.part_o + prow * kDim);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t orow[32];
          TMEM_LD_32((tm_o + 32u * q4) | lane_sel, orow, 0);
          tmem_wait_ld();
          if (mine) {
            if (ur.slot < 0) {
#pragma unroll
              for (int j = 0; j < 32; j += 8)
                dst_out[4 * q4 + (j >> 3)] = make_uint4(
                    pack2(__uint_as_float(orow[j]) * inv, __uint_as_float(orow[j + 1]) * inv),
                    pack2(__uint_as_float(orow[j + 2]) * inv, __uint_as_float(orow[j + 3]) * inv),
                    pack2(__uint_as_float(orow[j + 4]) * inv, __uint_as_float(orow[j + 5]) * inv),
                    pack2(__uint_as_float(orow[j + 6]) * inv, __uint_as_float(orow[j + 7]) * inv));
            } else {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                dst_part[8 * q4 + (j >> 2)] =
                    make_float4(__uint_as_float(orow[j]), __uint_as_float(orow[j + 1]),
                                __uint_as_float(orow[j + 2]), __uint_as_float(orow[j + 3]));
            }
          }
        }
        if (mine && ur.slot >= 0) a.part_ml[prow] = make_float2(ref, l);
      }
      // O has been read: the next head's first P V may overwrite it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) bar_arrive(bar(ODONE));
    }
  }
  // ---- common exit: every role arrives here, then the allocating warp frees TMEM
  if (a.pdl && threadIdx.x == 0) pdl_wait();      // this grid completes after its predecessor
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem),
                 "r"(kTmemCols) : "memory");
  }
}


// ---------------------------------------------------------------------------- persistent form
// The same roles and the same per-tile pipeline, but a CTA does not end with its work item: two
// CTAs per SM stay resident and claim units - one (work item, kv head) each - from a device
// counter, longest items first.  The producer claims the next unit while the current one is
// still streaming and publishes its description (item fields, users, first block ids) in a
// small ring in shared memory, so that across a unit boundary the K/V rings never run dry, the
// MMA thread issues the next unit's Q K^T while the softmax warps still write the previous
// unit's rows out, and barrier initialisation, TMEM allocation and CTA start-up are paid once
// per CTA instead of once per unit.  All four softmax warps take part in every unit (rows past
// the unit's own are zero queries whose results are dropped), so that every barrier has a
// fixed number of arrivals whatever the unit's width.
constexpr int kDescSlots = 3;
constexpr int kClaimTiles = 8;      // the next unit is claimed this many K tiles before the end
constexpr uint32_t kPollSpin = kSpin * 16;   // bound of the roles that poll without suspending
                                             // (a pass of theirs is some tens of cycles)
struct UnitDesc {
  int32_t table_row, tok_begin, n_tok, n_tiles;     // n_tiles == 0: no more units
  int32_t kvh, n_users, slot_add, pad;
  UserRef users[64];
  int32_t ids[64];                                  // first block ids of the run
};
constexpr int kDescOff = kUserOff;
constexpr int kSmemP = kDescOff + kDescSlots * (int)sizeof(UnitDesc) + 1024;
enum BarP { DFULL0 = NBARS, DEMPTY0 = DFULL0 + kDescSlots, NBARS_P = DEMPTY0 + kDescSlots };
static_assert(8 * NBARS_P + 16 <= 256, "barrier area");

__global__ void __launch_bounds__(192, 2)
attn_umma_persist_kernel(const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, const AttnArgs a,
                         int item_begin, int n_units, int* __restrict__ ticket) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (s32(smem_raw) + 1023u) & ~1023u;
  uint8_t* bp = smem_raw + (base - s32(smem_raw));
  const uint32_t bars = base + kBarOff;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile int* cta_abort = (volatile int*)(bp + kBarOff + 8 * NBARS_P);
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(bp + kBarOff + 8 * NBARS_P + 8);
  UnitDesc* descs = (UnitDesc*)(bp + kDescOff);

  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *cta_abort = *(volatile int*)a.d_error;
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_v) : "memory");
    for (int s = 0; s < kKStages; ++s) {
      bar_init(bar(KFULL0 + s), 1);
      bar_init(bar(KEMPTY0 + s), 1);
    }
    for (int s = 0; s < kVStages; ++s) {
      bar_init(bar(VFULL0 + s), 1);
      bar_init(bar(VEMPTY0 + s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      bar_init(bar(SFULL0 + b), 1);
      bar_init(bar(SFREE0 + b), 4);
    }
    bar_init(bar(PFULL), 4);
    bar_init(bar(PFREE), 1);
    bar_init(bar(QFULL), 4);
    bar_init(bar(ODONE), 4);
    for (int d = 0; d < kDescSlots; ++d) {
      bar_init(bar(DFULL0 + d), 1);
      bar_init(bar(DEMPTY0 + d), 5);               // four softmax warps and the MMA thread
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(s32((const void*)tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (*cta_abort) {
    if (warp == 5)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem),
                   "r"(kTmemCols) : "memory");
    if (threadIdx.x == 128) {                 // keeps the launch's exit count complete
      const int gone = atomicAdd(ticket + 1, 1);
      if (gone == (int)gridDim.x - 1) {
        ticket[0] = 0;
        ticket[1] = 0;
      }
    }
    return;
  }
  const uint32_t tm_o = tmem + 128u;
  if (threadIdx.x == 0) pdl_launch_dependents();

  if (warp == 4) {
    // ---------------------------------------------------------------- producer + unit fetch
    // Fetch of the next unit, one phase per call so that the global-memory round trips of its
    // chain (ticket -> work item -> lengths, users, block ids) pass while K/V tiles are issued.
    int f_phase = 0, f_units = 0;     // descriptors published so far (the end mark included)
    bool f_end = false;
    int f_tick = 0;
    int4 f_item = make_int4(0, 0, 0, 0);
    int f_row = 0, f_tok_begin = 0, f_tok_end = 0, f_user_begin = 0, f_n_users = 0, f_slot_add = 0;
    int f_len = 0, f_id0 = 0, f_id1 = 0;
    UserRef f_u0 = UserRef{0, -1}, f_u1 = UserRef{0, -1};
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
          // a unit's kv heads follow each other (they walk the same block ids)
          const int item = f_tick / HKV;
          const int4* ip = (const int4*)(a.d_items + item_begin + item);
          if (lane < 2) f_item = __ldg(ip + lane);
          f_phase = 2;
        }
      } else if (f_phase == 2) {
        f_row = __shfl_sync(0xffffffffu, f_item.x, 0);
        f_tok_begin = __shfl_sync(0xffffffffu, f_item.y, 0);
        f_tok_end = __shfl_sync(0xffffffffu, f_item.z, 0);
        f_user_begin = __shfl_sync(0xffffffffu, f_item.w, 0);
        f_n_users = __shfl_sync(0xffffffffu, f_item.x, 1);
        f_slot_add = __shfl_sync(0xffffffffu, f_item.y, 1);
        if (f_tok_end < 0 && lane == 0) f_len = a.d_lens[f_row];
        const int32_t* tab = a.d_tables + (size_t)f_row * a.shape.table_stride;
        const int p0 = f_tok_begin / kBlock + lane;          // stays inside the table row
        f_id0 = p0 < a.shape.table_stride ? tab[p0] : 0;
        f_id1 = p0 + 32 < a.shape.table_stride ? tab[p0 + 32] : 0;
        if (lane < f_n_users) f_u0 = a.d_users[f_user_begin + lane];
        if (lane + 32 < f_n_users) f_u1 = a.d_users[f_user_begin + lane + 32];
        f_phase = 3;
      } else {
        const int slot = f_units % kDescSlots;
        int ok = f_units < kDescSlots ||
                 bar_test(bar(DEMPTY0 + slot), ((f_units / kDescSlots) - 1) & 1);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) return;
        UnitDesc* d = descs + slot;
        const bool end = f_tick >= n_units;
        if (end) {
          if (lane == 0) d->n_tiles = 0;
          f_end = true;
        } else {
          const int tok_end = f_tok_end < 0 ? __shfl_sync(0xffffffffu, f_len, 0) : f_tok_end;
          if (lane == 0) {
            d->table_row = f_row;
            d->tok_begin = f_tok_begin;
            d->n_tok = tok_end - f_tok_begin;
            d->n_tiles = (tok_end - f_tok_begin + kTileTok - 1) / kTileTok;
            d->kvh = f_tick % HKV;
            d->n_users = f_n_users;
            d->slot_add = f_slot_add;
          }
          d->ids[lane] = f_id0;
          d->ids[lane + 32] = f_id1;
          if (lane < f_n_users) d->users[lane] = f_u0;
          if (lane + 32 < f_n_users) d->users[lane + 32] = f_u1;
        }
        __syncwarp();
        if (lane == 0) bar_arrive(bar(DFULL0 + slot));
        ++f_units;
        f_phase = 0;
      }
    };

    // K and V tiles are two independent sequences over the units; each has its own cursor.
    struct Cursor {
      int unit = 0, t = 0, n_tiles = 0, n_blk = 0, kvh = 0;   // unit ordinal, tile in the unit
      bool active = false, done = false;
      const int32_t* table = nullptr;
      int id_cur = 0, id_next = 0;
    } kc, vc;
    auto open_unit = [&](Cursor& c) {
      const UnitDesc* d = descs + c.unit % kDescSlots;
      const int n_tiles = d->n_tiles;
      if (n_tiles == 0) {
        c.done = true;
        return;
      }
      c.n_tiles = n_tiles;
      c.n_blk = (d->n_tok + kBlock - 1) / kBlock;
      c.kvh = d->kvh;
      c.table = a.d_tables + (size_t)d->table_row * a.shape.table_stride + d->tok_begin / kBlock;
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
      if (t > 0 && (t & 7) == 0) {
        c.id_cur = c.id_next;
        const int nxt = (t + 8) * kTileBlocks + lane;
        c.id_next = nxt < c.n_blk ? c.table[nxt] : 0;
      }
      const int blk = t * kTileBlocks + (lane >> 1);
      const int bid = __shfl_sync(0xffffffffu, c.id_cur, blk & 31);
      if (lane == 0)
        bar_expect_tx(bar(full0 + s),
                      (uint32_t)min(kTileBlocks, c.n_blk - t * kTileBlocks) * kTileBytes);
      __syncwarp();
      if (lane < 2 * kTileBlocks && blk < c.n_blk)
        tma_2d(ring + s * kKV + (lane & 1) * kHalf + (lane >> 1) * (kBlock * 128), map,
               (lane & 1) * 64, (bid * HKV + c.kvh) * kBlock, bar(full0 + s));
      if (++c.t == c.n_tiles) {
        c.active = false;
        ++c.unit;
      }
      return true;
    };

    int kg = 0, vg = 0;               // tiles issued so far, all units
    uint32_t idle = 0;
    // the first unit: its fetch is driven to the end at once
    for (int i = 0; i < 4 && f_units == 0; ++i) fetch_step(true);
    // (both cursors have to reach the end mark: V tiles can be released and issued ahead of the
    // K tiles of the same unit when a K copy comes in late)
    while (!(kc.done && vc.done)) {
      bool did = false;
      if (!kc.active && !kc.done && kc.unit < f_units) open_unit(kc);
      bool did_k = false;
      if (kc.active && issue(kc, kg, kKStages, KEMPTY0, KFULL0, base, &tm_k)) {
        ++kg;
        did = did_k = true;
      }
      if (!vc.active && !vc.done && vc.unit < f_units) open_unit(vc);
      if (vc.active && issue(vc, vg, kVStages, VEMPTY0, VFULL0, base + kVOff, &tm_v)) {
        ++vg;
        did = true;
      }
      // claim the next unit towards the end of the K stream of the current one (or at once
      // when the K cursor has nothing to do); one phase per tile issued or per idle pass
      const bool near_end = !kc.active || kc.n_tiles - kc.t <= kClaimTiles;
      const bool room = f_units <= kc.unit + (kc.active ? 1 : 0);
      if (did_k || !kc.active) fetch_step(near_end && room);
      if (did) {
        idle = 0;
      } else {
        ++idle;
        int stop = idle > kPollSpin || ((idle & 255) == 0 && *cta_abort);
        if (__shfl_sync(0xffffffffu, stop, 0)) {
          if (lane == 0 && idle > kPollSpin) {
            *cta_abort = 1;
            atomicCAS(a.d_error, 0, 6000 + (kg % 25) * 40 + vg % 40);
          }
          break;
        }
      }
    }
    // After a wait that gave up, the copies this warp still has in flight are waited for (with
    // a limit of their own) before the CTA's shared memory goes away.  (Otherwise every copy
    // has been consumed: its consumer waited for it.)
    if (*cta_abort && lane == 0) {
      for (int g = max(0, kg - kKStages); g < kg; ++g)
        for (uint32_t i = 0; i < kSpin && !bar_try(bar(KFULL0 + g % kKStages), (g / kKStages) & 1); ++i) {}
      for (int g = max(0, vg - kVStages); g < vg; ++g)
        for (uint32_t i = 0; i < kSpin && !bar_try(bar(VFULL0 + g % kVStages), (g / kVStages) & 1); ++i) {}
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
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issuer
    constexpr uint32_t kIdescQK = instr_desc(kTileTok, false);
    constexpr uint32_t kIdescPV = instr_desc(kDim, true);
    if (lane == 0) {
      int qk_g = 0, pv_g = 0;                 // tiles issued, all units
      int qu = 0, qt = 0, q_tiles = -1;       // Q K^T cursor: unit ordinal, tile, tiles (-1: unknown)
      int pu = 0, pt = 0, p_tiles = -1, p_tok = 0;
      bool q_done = false;
      uint32_t idle = 0;
      while (true) {
        bool did = false;
        if (!q_done && q_tiles < 0 && bar_test(bar(DFULL0 + qu % kDescSlots), (qu / kDescSlots) & 1)) {
          q_tiles = descs[qu % kDescSlots].n_tiles;
          if (q_tiles == 0) q_done = true;
        }
        if (!q_done && q_tiles > 0) {
          const int g = qk_g, s = g % kKStages, b = g & 1;
          if (bar_test(bar(KFULL0 + s), (g / kKStages) & 1) &&
              (g < 2 || bar_test(bar(SFREE0 + b), ((g >> 1) - 1) & 1)) &&
              (qt > 0 || bar_test(bar(QFULL), qu & 1))) {
            tc_fence_after();
            const uint32_t kb = base + s * kKV, qb = base + kQOff;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t off = (ks >> 2) * kHalf + (ks & 3) * 32;
              umma_bf16(tmem + 64u * b, smem_desc(qb + off, 16, 1024),
                        smem_desc(kb + off, 16, 1024), kIdescQK, ks > 0);
            }
            umma_commit(bar(SFULL0 + b));
            umma_commit(bar(KEMPTY0 + s));
            ++qk_g;
            if (++qt == q_tiles) {
              qt = 0;
              ++qu;
              q_tiles = -1;
            }
            did = true;
          }
        }
        if (pv_g < qk_g) {
          if (p_tiles < 0) {                  // (published: the Q K^T cursor has read it before)
            p_tiles = descs[pu % kDescSlots].n_tiles;
            p_tok = descs[pu % kDescSlots].n_tok;
          }
          const int g = pv_g, s = g % kVStages;
          if (bar_test(bar(PFULL), g & 1) && bar_test(bar(VFULL0 + s), (g / kVStages) & 1) &&
              (pt > 0 || pu == 0 || bar_test(bar(ODONE), (pu - 1) & 1))) {
            tc_fence_after();
            const uint32_t vb = base + kVOff + s * kKV, pb = base + kPOff;
            const int nk = min(kTileBlocks, (p_tok - pt * kTileTok + kBlock - 1) / kBlock);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              if (kk < nk)
                umma_bf16(tm_o, smem_desc(pb + kk * 32, 16, 1024),
                          smem_desc(vb + kk * (kBlock * 128), kHalf, 1024), kIdescPV,
                          (pt | kk) != 0);
            umma_commit(bar(PFREE));
            umma_commit(bar(VEMPTY0 + s));
            ++pv_g;
            if (++pt == p_tiles) {
              bar_arrive(bar(DEMPTY0 + pu % kDescSlots));     // done with this description
              pt = 0;
              ++pu;
              p_tiles = -1;
            }
            did = true;
          }
        }
        if (q_done && pv_g == qk_g) break;
        if (did) {
          idle = 0;
        } else if (++idle > kPollSpin || ((idle & 255) == 0 && *cta_abort)) {
          if (idle > kPollSpin) atomicCAS(a.d_error, 0, 7000 + (qk_g % 25) * 40 + pv_g % 40);
          *cta_abort = 1;
          break;
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- softmax warps 0-3
    const int row = warp * 16 + (lane & 15);
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    const float c = a.scale_log2e;
    const float cc = c > 0.f ? c : 1.f;               // what is left to apply inside the exponent
    const int g8 = lane >> 2, qd = lane & 3;
    // rows 16w .. 16w+15 of unit description d into the A-operand layout (rows past the unit's
    // own as zeros)
    auto stage_q = [&](const UnitDesc* d) {
      const int R = d->n_users * G, kvh = d->kvh;
      uint4 qv[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = lane + 32 * k, r = warp * 16 + (i >> 4), cc = i & 15;
        qv[k] = make_uint4(0u, 0u, 0u, 0u);
        if (r < R)
          qv[k] = __ldg((const uint4*)a.q +
                        ((size_t)d->users[r / G].query * HQ + kvh * G + r % G) * 16 + cc);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = lane + 32 * k;
        *(uint4*)(bp + kQOff + swz_off(warp * 16 + (i >> 4), i & 15)) = qv[k];
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) bar_arrive(bar(QFULL));
    };
    bool alive = bar_wait(bar(DFULL0), 0, cta_abort, a.d_error, 1000);
    if (alive && descs[0].n_tiles > 0) stage_q(descs);
    int g0 = 0;                                       // tiles of earlier units
    for (int u = 0; alive; ++u) {
      const UnitDesc* d = descs + u % kDescSlots;     // published: waited for below / above
      const int n_tiles = d->n_tiles;
      if (n_tiles == 0) break;
      const int n_tok = d->n_tok, R = d->n_users * G, kvh = d->kvh, slot_add = d->slot_add;
      float ref_lo = -INFINITY, ref_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
      for (int t = 0; t < n_tiles; ++t) {
        const int g = g0 + t, b = g & 1;
        if (!bar_wait(bar(SFULL0 + b), (g >> 1) & 1, cta_abort, a.d_error, 2000 + t % 1000)) {
          alive = false;
          break;
        }
        tc_fence_after();
        uint32_t sr[32];
        TMEM_LD_16x256((tmem + 64u * b) | lane_sel, sr);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) bar_arrive(bar(SFREE0 + b));
        const int tile_tok = min(kTileTok, n_tok - t * kTileTok);
        // The raw scores stay in registers; the scale is applied to the row maximum and, fused
        // with the subtraction of the reference, inside the exponent.  A key past the unit's
        // last token becomes -inf (rows of K past the valid length hold unspecified bits); full
        // tiles skip that pass.  (A scale that is not positive is applied up front, so that the
        // maximum of the raw values is the maximum.)
        if (!(c > 0.f)) {
#pragma unroll
          for (int j = 0; j < 32; ++j) sr[j] = __float_as_uint(__uint_as_float(sr[j]) * c);
        }
        if (tile_tok < kTileTok) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              if (8 * k + 2 * qd + e >= tile_tok) sr[4 * k + e] = sr[4 * k + 2 + e] = 0xff800000u;
            }
          }
        }
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          mx_lo = fmaxf(mx_lo, fmaxf(__uint_as_float(sr[4 * k]), __uint_as_float(sr[4 * k + 1])));
          mx_hi = fmaxf(mx_hi, fmaxf(__uint_as_float(sr[4 * k + 2]), __uint_as_float(sr[4 * k + 3])));
        }
        mx_lo *= cc;
        mx_hi *= cc;
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const bool move_lo = mx_lo > ref_lo + kRefSlack || ref_lo == -INFINITY;
        const bool move_hi = mx_hi > ref_hi + kRefSlack || ref_hi == -INFINITY;
        const float new_lo = move_lo ? mx_lo : ref_lo, new_hi = move_hi ? mx_hi : ref_hi;
        const bool rescale = t > 0 && __any_sync(0xffffffffu, move_lo || move_hi);
        if (rescale) {
          if (!bar_wait(bar(PFREE), (g - 1) & 1, cta_abort, a.d_error, 3000 + t % 1000)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const float f_lo = move_lo ? ex2(ref_lo - new_lo) : 1.f;
          const float f_hi = move_hi ? ex2(ref_hi - new_hi) : 1.f;
          l_lo *= f_lo;
          l_hi *= f_hi;
          const float fa = __shfl_sync(0xffffffffu, f_lo, 4 * (lane & 7));
          const float fb = __shfl_sync(0xffffffffu, f_hi, 4 * (lane & 7));
          const float f = (lane & 8) ? fb : fa;
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
        ref_lo = new_lo;
        ref_hi = new_hi;
        uint32_t pk_lo[8], pk_hi[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float a0 = ex2(fmaf(__uint_as_float(sr[4 * k]), cc, -ref_lo));
          const float a1 = ex2(fmaf(__uint_as_float(sr[4 * k + 1]), cc, -ref_lo));
          const float b0 = ex2(fmaf(__uint_as_float(sr[4 * k + 2]), cc, -ref_hi));
          const float b1 = ex2(fmaf(__uint_as_float(sr[4 * k + 3]), cc, -ref_hi));
          l_lo += a0 + a1;
          l_hi += b0 + b1;
          pk_lo[k] = pack2(a0, a1);
          pk_hi[k] = pack2(b0, b1);
        }
        if (g > 0 && !rescale &&
            !bar_wait(bar(PFREE), (g - 1) & 1, cta_abort, a.d_error, 3000 + t % 1000)) {
          alive = false;
          break;
        }
        {
          const int r_lo = warp * 16 + g8;
          uint8_t* p_lo = bp + kPOff + r_lo * 128 + 4 * qd;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int off = (k ^ (r_lo & 7)) << 4;
            *(uint32_t*)(p_lo + off) = pk_lo[k];
            *(uint32_t*)(p_lo + 8 * 128 + off) = pk_hi[k];
          }
        }
        if (tile_tok < kTileTok && warp == 0) {
          const int vs = g % kVStages;
          if (!bar_wait(bar(VFULL0 + vs), (g / kVStages) & 1, cta_abort, a.d_error,
                        4000 + t % 1000)) {
            alive = false;
            break;
          }
          uint8_t* vptr = bp + kVOff + vs * kKV;
          const int first = tile_tok, last = ((tile_tok + kBlock - 1) / kBlock) * kBlock;
          for (int x = lane; x < (last - first) * 16; x += 32)
            *(uint4*)(vptr + swz_off(first + (x >> 4), x & 15)) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) bar_arrive(bar(PFULL));
      }
      if (!alive) break;
      // This warp has seen the unit's last S tile, so every Q K^T of the unit has completed:
      // the next unit's rows can take the Q buffer while the last P V is still running.
      const UnitDesc* dn = descs + (u + 1) % kDescSlots;
      if (!bar_wait(bar(DFULL0 + (u + 1) % kDescSlots), ((u + 1) / kDescSlots) & 1, cta_abort,
                    a.d_error, 1000 + (u + 1) % 1000))
        break;
      // the users of this unit are read below: copy what the write-out needs before the
      // description can be reused (it cannot before this warp's own arrival, see the end)
      if (dn->n_tiles > 0) stage_q(dn);
      if (!bar_wait(bar(PFREE), (g0 + n_tiles - 1) & 1, cta_abort, a.d_error, 5000)) break;
      tc_fence_after();
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
      const float la = __shfl_sync(0xffffffffu, l_lo, 4 * (lane & 7));
      const float lb = __shfl_sync(0xffffffffu, l_hi, 4 * (lane & 7));
      const float ra = __shfl_sync(0xffffffffu, ref_lo, 4 * (lane & 7));
      const float rb = __shfl_sync(0xffffffffu, ref_hi, 4 * (lane & 7));
      const float l = (lane & 8) ? lb : la, ref = (lane & 8) ? rb : ra;
      {
        const bool mine = lane < 16 && row < R;
        UserRef ur = UserRef{0, -1};
        if (mine) ur = d->users[row / G];
        const int head = kvh * G + row % G;
        const float inv = 1.f / l;
        uint4* dst_out = (uint4*)((__nv_bfloat16*)a.out + ((size_t)ur.query * HQ + head) * kDim);
        const size_t prow = (size_t)(ur.slot + slot_add) * HQ + head;
        float4* dst_part = (float4*)(a.part_o + prow * kDim);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t orow[32];
          TMEM_LD_32((tm_o + 32u * q4) | lane_sel, orow, 0);
          tmem_wait_ld();
          if (mine) {
            if (ur.slot < 0) {
#pragma unroll
              for (int j = 0; j < 32; j += 8)
                dst_out[4 * q4 + (j >> 3)] = make_uint4(
                    pack2(__uint_as_float(orow[j]) * inv, __uint_as_float(orow[j + 1]) * inv),
                    pack2(__uint_as_float(orow[j + 2]) * inv, __uint_as_float(orow[j + 3]) * inv),
                    pack2(__uint_as_float(orow[j + 4]) * inv, __uint_as_float(orow[j + 5]) * inv),
                    pack2(__uint_as_float(orow[j + 6]) * inv, __uint_as_float(orow[j + 7]) * inv));
            } else {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                dst_part[8 * q4 + (j >> 2)] =
                    make_float4(__uint_as_float(orow[j]), __uint_as_float(orow[j + 1]),
                                __uint_as_float(orow[j + 2]), __uint_as_float(orow[j + 3]));
            }
          }
        }
        if (mine && ur.slot >= 0) a.part_ml[prow] = make_float2(ref, l);
      }
      // O has been read and this unit's description is no longer needed by this warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        bar_arrive(bar(ODONE));
        bar_arrive(bar(DEMPTY0 + u % kDescSlots));
      }
      g0 += n_tiles;
    }
  }
  // ---- common exit: every role arrives here, then the allocating warp frees TMEM
  if (a.pdl && threadIdx.x == 0) pdl_wait();
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem),
                 "r"(kTmemCols) : "memory");
  }
}

}  // namespace

cudaError_t launch_attention_umma(const AttnArgs& a, int item_begin, int n_items,
                                  cudaStream_t st) {
  if (n_items <= 0) return cudaSuccess;
  static bool configured[64] = {};
  static int sm_count[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_umma_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_umma_persist_kernel,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemP);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const int hkv = a.shape.num_kv_heads;
  if (a.umma_mode != 1 && a.d_ticket != nullptr) {
    // persistent form: two resident CTAs per SM claim (item, kv head) units from a counter
    const long long n_units = (long long)n_items * hkv;
    const int grid = (int)std::min<long long>(n_units, 2LL * sm_count[dev]);
    return launch_kernel(attn_umma_persist_kernel, dim3(grid), dim3(192), kSmemP, st, a.pdl != 0,
                         *a.tm_k, *a.tm_v, a, item_begin, (int)n_units, a.d_ticket);
  }
  // Heads per CTA: up to kHeadsMax, if that leaves at least kWavesMin CTAs for each of the
  // machine's CTA slots (two per SM), so that the hardware scheduler can still even out the
  // load.  Measured: two heads per CTA take 2-3 % off the kernel, four or eight cost more in
  // uneven last waves than the hidden start-up saves (the kernel is bound by HBM, not by the
  // latencies that running on into the next head hides).
  int u = 1;
  for (int c = 2; c <= kHeadsMax && c <= hkv; c *= 2)
    if (hkv % c == 0 && (long long)n_items * (hkv / c) >= (long long)kWavesMin * 2 * sm_count[dev])
      u = c;
  if (a.umma_heads >= 1 && hkv % a.umma_heads == 0) u = a.umma_heads;   // forced (testing)
  return launch_kernel(attn_umma_kernel, dim3(n_items, hkv / u), dim3(192), kSmem, st, a.pdl != 0,
                       *a.tm_k, *a.tm_v, a, item_begin, u);
}

}  // namespace apar

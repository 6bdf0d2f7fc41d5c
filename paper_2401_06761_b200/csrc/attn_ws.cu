// Warp-stream attention path for work items with at most 16 query rows per kv head (the tails of
// GQA threads, small sets of siblings): one CTA owns a whole work item, *all* kv heads (or a
// group of them when there are too few items to fill the machine).
//
// The four consumer warps each stream different kv heads, independently of one another: warp w
// takes heads w, w+4, ...  Every warp has its own ring of three 16-token slots (K and V tile of
// one block, 8 KiB) filled by the producer warp with TMA tensor copies, its own mbarriers, and
// keeps Q (as mma.sync A-fragments, fetched straight from global memory one head ahead), the
// online-softmax state and O in registers.  There is no CTA-wide synchronisation inside the
// loop, no folding between warps, and the fixed cost of a CTA (item, users, first TMA round
// trip, write-out) is paid once per item instead of once per (item, head), which is what the
// short tails of decode batches are sensitive to.  Two CTAs per SM, each with four rings of
// three 8 KiB slots, keep up to 192 KiB in flight and overlap one CTA's start-up and
// write-out with the other's streaming.
#include <algorithm>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "apar_internal.h"
#include "ptx.cuh"

namespace apar {
namespace {

constexpr int kSlots = 3;                           // ring depth per consumer warp
constexpr int kSlotBytes = 2 * kTileBytes;          // K tile + V tile of one block: 8 KiB
constexpr int kRingBytes = 4 * kSlots * kSlotBytes; // 128 KiB
constexpr int kUsersOffW = kRingBytes;              // UserRef[16]
constexpr int kBarsOffW = kUsersOffW + 16 * 8;      // full[4][kSlots], empty[4][kSlots]
constexpr int kSmemW = kBarsOffW + 2 * 4 * kSlots * 8 + 64 + 1024;
constexpr float kSlack = 8.f;                       // the reference max moves only past 2^8

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// (row of the block, 16-byte chunk c of 16) inside a [2 halves][16 rows][64 dims] tile written
// by TMA with the 128-byte swizzle.
__device__ __forceinline__ uint32_t blk_off(int row, int c) {
  return (uint32_t)((c >> 3) * 2048 + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}

__global__ void __launch_bounds__(160, 2)
attn_ws_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const AttnArgs a, int item_begin, int heads_per_cta) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (s32(smem_raw) + 1023u) & ~1023u;
  uint8_t* bp = smem_raw + (base - s32(smem_raw));
  UserRef* s_users = (UserRef*)(bp + kUsersOffW);
  const uint32_t bars = base + kBarsOffW;
  auto full_bar = [&](int w, int s) { return bars + 8u * (w * kSlots + s); };
  auto empty_bar = [&](int w, int s) { return bars + 8u * (4 * kSlots + w * kSlots + s); };
  volatile int* cta_abort = (volatile int*)(bp + kBarsOffW + 2 * 4 * kSlots * 8);

  const WorkItem it = a.d_items[item_begin + blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  const int tok_end = it.tok_end < 0 ? a.d_lens[it.table_row] : it.tok_end;
  const int n_tok = tok_end - it.tok_begin;
  const int n_blk = (n_tok + kBlock - 1) / kBlock;
  const int32_t* table = a.d_tables + (size_t)it.table_row * a.shape.table_stride +
                         it.tok_begin / kBlock;
  const int R = it.n_users * G;                    // rows per kv head, <= 16
  // this CTA's kv heads: [h_begin, h_begin + n_heads); warp w takes h_begin + w, + w + 4, ...
  const int h_begin = blockIdx.y * heads_per_cta;
  const int n_heads = min(heads_per_cta, HKV - h_begin);
  // started before the CTA's only barrier so that the latencies overlap: descriptor prefetch
  // and barrier init (thread 0), the first block id (producer), the item's users
  if (threadIdx.x == 0) {
    *cta_abort = *(volatile int*)a.d_error;   // an earlier CTA gave up a wait: do not pile up
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_v) : "memory");
    for (int i = 0; i < 4 * kSlots; ++i) {
      bar_init(bars + 8u * i, 1);
      bar_init(bars + 8u * (4 * kSlots + i), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  int bid_first = 0;
  if (warp == 4) bid_first = n_blk > 0 ? table[0] : 0;
  else if (threadIdx.x < it.n_users) s_users[threadIdx.x] = a.d_users[it.user_begin + threadIdx.x];
  __syncthreads();
  if (*cta_abort) return;
  if (threadIdx.x == 0) pdl_launch_dependents();

  if (warp == 4) {
    // ------------------------------------------------------------------ producer warp
    // Lanes 0-15 work on their own: lane = 4 * stream + op, op = K lo, K hi, V lo, V hi.  The
    // four lanes of a stream poll the same "slot free" barrier and each issues its own copy;
    // the op-0 lane also posts the byte count.
    if (lane < 16) {
      const int w = lane >> 2, op = lane & 3;
      const int heads_w = max(0, n_heads - w + 3) >> 2;
      const int total = heads_w * n_blk;
      const CUtensorMap* map = (op >> 1) ? &tm_v : &tm_k;
      int bid_next = bid_first;
      for (int c = 0, hi = 0, b = 0; c < total; ++c) {
        const int bid = bid_next;
        const int b1 = b + 1 == n_blk ? 0 : b + 1;
        if (c + 1 < total) bid_next = table[b1];            // one block ahead of its use
        const int s = c % kSlots;
        if (c >= kSlots &&
            !bar_wait(empty_bar(w, s), ((c / kSlots) - 1) & 1, cta_abort, a.d_error, 8000 + w))
          break;
        if (op == 0) bar_expect_tx(full_bar(w, s), kSlotBytes);
        const int h = h_begin + w + 4 * hi;
        tma_2d(base + (w * kSlots + s) * kSlotBytes + (op >> 1) * kTileBytes + (op & 1) * 2048, map,
              (op & 1) * 64, (bid * HKV + h) * kBlock, full_bar(w, s));
        b = b1;
        if (b == 0) ++hi;
      }
    }
    if (a.pdl) pdl_wait();                         // this grid completes after its predecessor
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const int w = warp;
  const int heads_w = max(0, n_heads - w + 3) >> 2;
  const int g = lane >> 2, tq = lane & 3;
  const int jm = lane >> 3, jr = lane & 7;
  const float cs = a.scale_log2e;

  // Q rows g and g+8 of head h as A-fragments, straight from global memory.
  auto load_q = [&](int h, uint32_t (&qa)[8][4]) {
    const uint32_t* p0 = nullptr;
    const uint32_t* p1 = nullptr;
    if (g < R)
      p0 = (const uint32_t*)a.q + ((size_t)s_users[g / G].query * HQ + h * G + g % G) * 64;
    if (g + 8 < R)
      p1 = (const uint32_t*)a.q +
           ((size_t)s_users[(g + 8) / G].query * HQ + h * G + (g + 8) % G) * 64;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = p0 ? __ldg(p0 + ks * 8 + tq) : 0u;
      qa[ks][2] = p0 ? __ldg(p0 + ks * 8 + 4 + tq) : 0u;
      qa[ks][1] = p1 ? __ldg(p1 + ks * 8 + tq) : 0u;
      qa[ks][3] = p1 ? __ldg(p1 + ks * 8 + 4 + tq) : 0u;
    }
  };

  uint32_t qa[8][4], qn[8][4];
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) qn[ks][0] = qn[ks][1] = qn[ks][2] = qn[ks][3] = 0u;
  if (heads_w > 0) load_q(h_begin + w, qa);
  int c = 0;                                       // blocks consumed so far by this warp
  bool alive = true, waited = false;
  for (int hi = 0; hi < heads_w && alive; ++hi) {
    const int h = h_begin + w + 4 * hi;
    if (hi + 1 < heads_w) load_q(h + 4, qn);       // lands while this head streams
    float o[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float ref0 = -INFINITY, ref1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    for (int b = 0; b < n_blk; ++b, ++c) {
      const int s = c % kSlots;
      if (!bar_wait(full_bar(w, s), (c / kSlots) & 1, cta_abort, a.d_error, 9000 + w)) {
        alive = false;
        break;
      }
      const uint32_t kb = base + (w * kSlots + s) * kSlotBytes, vb = kb + kTileBytes;
      const int nv = min(kBlock, n_tok - b * kBlock);
      // S = Q K^T for the 16 tokens of the block
      float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
      {
        const int row = (jm >> 1) * 8 + jr;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t kf[4];
          ldsm4(kb + blk_off(row, 2 * ks + (jm & 1)), kf);
          mma16816(acc0, qa[ks], kf[0], kf[1]);
          mma16816(acc1, qa[ks], kf[2], kf[3]);
        }
      }
      if (nv < kBlock) {   // rows of V past the valid length hold unspecified bits: zero them
        uint8_t* vptr = bp + (w * kSlots + s) * kSlotBytes + kTileBytes;
        for (int x = lane; x < (kBlock - nv) * 16; x += 32)
          *(uint4*)(vptr + blk_off(nv + (x >> 4), x & 15)) = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
      }
      float sc[2][4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int t0 = 2 * tq + (e & 1);
        sc[0][e] = t0 < nv ? acc0[e] * cs : -INFINITY;
        sc[1][e] = t0 + 8 < nv ? acc1[e] * cs : -INFINITY;
      }
      float mx0 = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
      float mx1 = fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      // the reference only moves when the maximum outgrows it by 2^8 (P stays below 256)
      const bool mv0 = mx0 > ref0 + kSlack || ref0 == -INFINITY;
      const bool mv1 = mx1 > ref1 + kSlack || ref1 == -INFINITY;
      if (__any_sync(0xffffffffu, mv0 || mv1)) {
        const float f0 = mv0 ? ex2(ref0 - mx0) : 1.f, f1 = mv1 ? ex2(ref1 - mx1) : 1.f;
        if (mv0) ref0 = mx0;
        if (mv1) ref1 = mx1;
        l0 *= f0;
        l1 *= f1;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          o[j][0] *= f0; o[j][1] *= f0; o[j][2] *= f1; o[j][3] *= f1;
        }
      }
      float p[2][4];
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        p[n][0] = ex2(sc[n][0] - ref0);
        p[n][1] = ex2(sc[n][1] - ref0);
        p[n][2] = ex2(sc[n][2] - ref1);
        p[n][3] = ex2(sc[n][3] - ref1);
      }
      l0 += p[0][0] + p[0][1] + p[1][0] + p[1][1];
      l1 += p[0][2] + p[0][3] + p[1][2] + p[1][3];
      uint32_t pa[4] = {pack2(p[0][0], p[0][1]), pack2(p[0][2], p[0][3]),
                        pack2(p[1][0], p[1][1]), pack2(p[1][2], p[1][3])};
      {
        const int row = (jm & 1) * 8 + jr;
#pragma unroll
        for (int jp = 0; jp < 8; ++jp) {
          uint32_t vf[4];
          ldsm4t(vb + blk_off(row, 2 * jp + (jm >> 1)), vf);
          mma16816(o[2 * jp], pa, vf[0], vf[1]);
          mma16816(o[2 * jp + 1], pa, vf[2], vf[3]);
        }
      }
      __syncwarp();
      if (lane == 0) bar_arrive(empty_bar(w, s));
    }
    if (!alive) break;
    // ---- this head's rows: straight from the accumulator fragments
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    // the partial results a finishing item folds come from earlier kernels of the call
    if (a.pdl && fin_count(it) > 0 && !waited) {
      pdl_wait();
      waited = true;
    }
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int r = g + 8 * half;
      if (r < R) {
        const UserRef ur = s_users[r / G];
        const int head = h * G + r % G;
        float L = half ? l1 : l0, M = half ? ref1 : ref0;
        // a finishing item folds the partial results of the rest of the chain into its own
        for (int pj = 0; pj < fin_count(it); ++pj) {
          const size_t prow = (size_t)(it.fin_begin + pj) * HQ + head;
          const float2 ml = a.part_ml[prow];
          const float2* src = (const float2*)(a.part_o + prow * kDim) + tq;
          const float mn = fmaxf(M, ml.x);
          const float f0 = M == -INFINITY ? 0.f : ex2(M - mn);
          const float f1 = ml.x == -INFINITY ? 0.f : ex2(ml.x - mn);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 x = src[4 * j];
            o[j][2 * half] = o[j][2 * half] * f0 + x.x * f1;
            o[j][2 * half + 1] = o[j][2 * half + 1] * f0 + x.y * f1;
          }
          L = L * f0 + ml.y * f1;
          M = mn;
        }
        if (ur.slot < 0 || fin_count(it) > 0) {
          const float inv = 1.f / L;
          uint32_t* dst = (uint32_t*)a.out + ((size_t)ur.query * HQ + head) * 64 + tq;
#pragma unroll
          for (int j = 0; j < 16; ++j)
            dst[4 * j] = pack2(o[j][2 * half] * inv, o[j][2 * half + 1] * inv);
        } else {
          const size_t prow = (size_t)(ur.slot + it.slot_add) * HQ + head;
          float2* dst = (float2*)(a.part_o + prow * kDim) + tq;
#pragma unroll
          for (int j = 0; j < 16; ++j) dst[4 * j] = make_float2(o[j][2 * half], o[j][2 * half + 1]);
          if (tq == 0) a.part_ml[prow] = make_float2(M, L);
        }
      }
    }
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
#pragma unroll
      for (int e = 0; e < 4; ++e) qa[ks][e] = qn[ks][e];
  }
  if (a.pdl) pdl_wait();                           // this grid completes after its predecessor
}


// ---------------------------------------------------------------------------- persistent form
// Every warp is a stream of its own: it claims units - one (work item, kv head) each - from a
// device counter (longest items first), issues its own TMA copies into a private ring of three
// slots, and computes.  There is no producer warp, no "slot free" barrier (the warp that read a
// slot is the one that refills it) and nothing shared between the warps of a CTA.  The copies
// run up to three blocks ahead of the arithmetic *across unit boundaries*: while a warp works
// on unit i its loads already fetch the first blocks of unit i+1, whose description (and, one
// step later, whose query rows) were fetched in the background, one step of that fetch per
// block computed.  So a warp's ring never drains between units, and what a CTA pays once per
// item in the other form (launch, barrier set-up, first round trips) is paid once per warp.
struct WsUnit {                       // what a warp needs to know about a unit
  const int32_t* table;               // first block id of the run
  int32_t n_tok, n_blk, h;            // tokens, blocks, kv head
  int32_t user_begin, n_users, slot_add, fin_n, fin_begin;
  uint32_t fin_flags;                 // folded parts that carry a ready flag (bit = part)
  bool valid;
};
constexpr int kUsersOffP = 4 * kSlots * kSlotBytes;          // UserRef[4 warps][2][16]
constexpr int kBarsOffP = kUsersOffP + 4 * 2 * 16 * 8;       // full[4][kSlots]
constexpr int kSmemWP = kBarsOffP + 4 * kSlots * 8 + 64 + 1024;

__global__ void __launch_bounds__(128, 2)
attn_ws_persist_kernel(const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const AttnArgs a, int item_begin,
                       int n_units, int* __restrict__ ticket) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (s32(smem_raw) + 1023u) & ~1023u;
  uint8_t* bp = smem_raw + (base - s32(smem_raw));
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  UserRef* users2 = (UserRef*)(bp + kUsersOffP) + w * 32;      // [2][16] of this warp
  const uint32_t bars = base + kBarsOffP + 8u * (w * kSlots);
  auto full_bar = [&](int s) { return bars + 8u * s; };
  volatile int* cta_abort = (volatile int*)(bp + kBarsOffP + 4 * kSlots * 8);
  const uint32_t ring = base + w * kSlots * kSlotBytes;
  uint8_t* ring_ptr = bp + w * kSlots * kSlotBytes;

  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  if (threadIdx.x == 0) {
    *cta_abort = *(volatile int*)a.d_error;   // an earlier CTA gave up a wait: do not pile up
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tm_v) : "memory");
    for (int i = 0; i < 4 * kSlots; ++i) bar_init(base + kBarsOffP + 8u * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool dead_on_arrival = *cta_abort != 0;
  if (threadIdx.x == 0) pdl_launch_dependents();

  const int g = lane >> 2, tq = lane & 3;
  const int jm = lane >> 3, jr = lane & 7;
  const float cs = a.scale_log2e;
  // ticket[0] unit counter, ticket[1] warps that have left, ticket[2] launches completed.  The
  // last warp to leave puts the first two back to zero and counts the launch, so that nobody
  // has to clear anything between launches (and a replayed CUDA graph finds the same state).
  // The launch count only changes when every warp has left: all warps read the same value,
  // and "ready" for a partial result of this launch is that value plus one.
  const int ready_mark = *(volatile int*)(ticket + 2) + 1;
  auto leave = [&]() {
    if (lane == 0) {
      const int gone = atomicAdd(ticket + 1, 1);
      if (gone == (int)gridDim.x * 4 - 1) {
        ticket[0] = 0;
        ticket[1] = 0;
        __threadfence();
        atomicAdd(ticket + 2, 1);
      }
    }
  };

  if (dead_on_arrival) {               // an earlier kernel gave up a wait: claim nothing
    leave();
    if (a.pdl) pdl_wait();
    return;
  }

  // ---- background fetch of unit descriptions: ticket -> work item -> (length) -> done
  WsUnit cur, nxt, nn;
  cur.valid = nxt.valid = nn.valid = false;
  int f_phase = 0, f_tick = 0, f_len = 0;
  int4 f_item = make_int4(0, 0, 0, 0);
  bool no_more = false;               // the counter has run past the last unit
  // one phase per call; returns true when `nn` has just become final (valid or "no more")
  auto fetch_step = [&]() -> bool {
    if (f_phase == 0) {
      if (no_more) return false;
      if (lane == 0) f_tick = atomicAdd(ticket, 1);
      f_phase = 1;
      return false;
    }
    if (f_phase == 1) {
      f_tick = __shfl_sync(0xffffffffu, f_tick, 0);
      if (f_tick >= n_units) {
        no_more = true;
        nn.valid = false;
        f_phase = 0;
        return true;
      }
      const int4* ip = (const int4*)(a.d_items + item_begin + f_tick / HKV);
      if (lane < 2) f_item = __ldg(ip + lane);
      f_phase = 2;
      return false;
    }
    if (f_phase == 2) {
      const int row = __shfl_sync(0xffffffffu, f_item.x, 0);
      const int tok_begin = __shfl_sync(0xffffffffu, f_item.y, 0);
      const int tok_end = __shfl_sync(0xffffffffu, f_item.z, 0);
      nn.user_begin = __shfl_sync(0xffffffffu, f_item.w, 0);
      nn.n_users = __shfl_sync(0xffffffffu, f_item.x, 1);
      nn.slot_add = __shfl_sync(0xffffffffu, f_item.y, 1);
      nn.fin_n = __shfl_sync(0xffffffffu, f_item.z, 1) & 0xff;
      nn.fin_flags = (uint32_t)__shfl_sync(0xffffffffu, f_item.z, 1) >> 8;
      nn.fin_begin = __shfl_sync(0xffffffffu, f_item.w, 1);
      nn.table = a.d_tables + (size_t)row * a.shape.table_stride + tok_begin / kBlock;
      nn.h = f_tick % HKV;
      nn.n_tok = tok_end - tok_begin;           // final unless the run is open-ended
      if (tok_end < 0) {
        if (lane == 0) f_len = a.d_lens[row];
        nn.n_tok = -tok_begin;                  // + the thread's length, next phase
        f_phase = 3;
        return false;
      }
      nn.n_blk = (nn.n_tok + kBlock - 1) / kBlock;
      nn.valid = true;
      f_phase = 0;
      return true;
    }
    nn.n_tok += __shfl_sync(0xffffffffu, f_len, 0);
    nn.n_blk = (nn.n_tok + kBlock - 1) / kBlock;
    nn.valid = true;
    f_phase = 0;
    return true;
  };
  bool nn_final = false;               // nn holds a finished fetch (a unit, or "no more")
  auto fetch_to_end = [&]() {
    while (!nn_final) nn_final = fetch_step();
  };

  // ---- query rows of a unit as A-fragments (rows g and g+8), users through shared memory
  uint32_t qa[8][4], qn[8][4];
  UserRef u_reg = UserRef{0, -1};
  auto load_users = [&](const WsUnit& u) {       // phase 1 of 2: into a register
    if (lane < u.n_users) u_reg = a.d_users[u.user_begin + lane];
  };
  auto load_q = [&](const WsUnit& u, int which, uint32_t (&q)[8][4]) {   // phase 2 of 2
    UserRef* us = users2 + which * 16;
    if (lane < u.n_users) us[lane] = u_reg;
    __syncwarp();
    const int R = u.n_users * G;
    const uint32_t* p0 = nullptr;
    const uint32_t* p1 = nullptr;
    if (g < R) p0 = (const uint32_t*)a.q + ((size_t)us[g / G].query * HQ + u.h * G + g % G) * 64;
    if (g + 8 < R)
      p1 = (const uint32_t*)a.q + ((size_t)us[(g + 8) / G].query * HQ + u.h * G + (g + 8) % G) * 64;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      q[ks][0] = p0 ? __ldg(p0 + ks * 8 + tq) : 0u;
      q[ks][2] = p0 ? __ldg(p0 + ks * 8 + 4 + tq) : 0u;
      q[ks][1] = p1 ? __ldg(p1 + ks * 8 + tq) : 0u;
      q[ks][3] = p1 ? __ldg(p1 + ks * 8 + 4 + tq) : 0u;
    }
  };

  // ---- copies: the load cursor runs ahead of the arithmetic, into the next unit if need be
  int c_load = 0, c_done = 0;          // blocks whose copies were issued / that were computed
  int l_blk = 0;                       // next block of the load cursor's unit
  bool l_in_next = false;              // the load cursor has moved on to `nxt`
  int bid_next = 0;                    // block id of the load cursor's next block, prefetched
  bool bid_ready = false;
  auto issue_loads = [&]() {
    while (c_load - c_done < kSlots) {
      const WsUnit& u = l_in_next ? nxt : cur;
      if (l_blk >= u.n_blk) {
        if (l_in_next || !nxt.valid) return;     // nothing further is known yet
        l_in_next = true;
        l_blk = 0;
        bid_ready = false;
        continue;
      }
      if (!bid_ready) bid_next = u.table[l_blk];
      const int bid = bid_next;
      bid_ready = l_blk + 1 < u.n_blk;
      if (bid_ready) bid_next = u.table[l_blk + 1];            // one block ahead of its use
      const int s = c_load % kSlots;
      if (lane == 0) bar_expect_tx(full_bar(s), kSlotBytes);
      __syncwarp();
      if (lane < 4) {
        const CUtensorMap* map = (lane >> 1) ? &tm_v : &tm_k;
        tma_2d(ring + s * kSlotBytes + (lane >> 1) * kTileBytes + (lane & 1) * 2048, map,
               (lane & 1) * 64, (bid * HKV + u.h) * kBlock, full_bar(s));
      }
      ++l_blk;
      ++c_load;
    }
  };

  // ---- the first unit: fetched at once; its successor's fetch starts right away
  fetch_to_end();
  cur = nn;
  nn_final = false;
  if (!cur.valid) {
    leave();
    if (a.pdl) pdl_wait();
    return;
  }
  load_users(cur);
  load_q(cur, 0, qa);
  int which = 0;                       // half of users2 that belongs to `cur`
  int q_phase = 0;                     // next unit's users / query rows: 0 none, 1 users in
                                       // flight, 2 rows in flight
  issue_loads();
  bool alive = true, waited = false;
  while (alive) {
    float o[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float ref0 = -INFINITY, ref1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    const int R = cur.n_users * G;
    const UserRef* s_users = users2 + which * 16;

    for (int b = 0; b < cur.n_blk; ++b) {
      // background work, one step per block: the unit after next, then the next unit's rows
      if (!nxt.valid && !no_more) {
        if (!nn_final) nn_final = fetch_step();
        if (nn_final) {
          nxt = nn;
          nn_final = false;
          q_phase = 0;
        }
      } else if (nxt.valid && q_phase < 2) {
        if (q_phase == 0) load_users(nxt);
        else load_q(nxt, which ^ 1, qn);
        ++q_phase;
      } else if (!nn_final && !no_more) {
        nn_final = fetch_step();
      }
      issue_loads();
      const int s = c_done % kSlots;
      if (!bar_wait(full_bar(s), (c_done / kSlots) & 1, cta_abort, a.d_error, 9000 + w)) {
        alive = false;
        break;
      }
      const uint32_t kb = ring + s * kSlotBytes, vb = kb + kTileBytes;
      const int nv = min(kBlock, cur.n_tok - b * kBlock);
      float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
      {
        const int row = (jm >> 1) * 8 + jr;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t kf[4];
          ldsm4(kb + blk_off(row, 2 * ks + (jm & 1)), kf);
          mma16816(acc0, qa[ks], kf[0], kf[1]);
          mma16816(acc1, qa[ks], kf[2], kf[3]);
        }
      }
      if (nv < kBlock) {   // rows of V past the valid length hold unspecified bits: zero them
        uint8_t* vptr = ring_ptr + s * kSlotBytes + kTileBytes;
        for (int x = lane; x < (kBlock - nv) * 16; x += 32)
          *(uint4*)(vptr + blk_off(nv + (x >> 4), x & 15)) = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
      }
      float sc[2][4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int t0 = 2 * tq + (e & 1);
        sc[0][e] = t0 < nv ? acc0[e] * cs : -INFINITY;
        sc[1][e] = t0 + 8 < nv ? acc1[e] * cs : -INFINITY;
      }
      float mx0 = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
      float mx1 = fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const bool mv0 = mx0 > ref0 + kSlack || ref0 == -INFINITY;
      const bool mv1 = mx1 > ref1 + kSlack || ref1 == -INFINITY;
      if (__any_sync(0xffffffffu, mv0 || mv1)) {
        const float f0 = mv0 ? ex2(ref0 - mx0) : 1.f, f1 = mv1 ? ex2(ref1 - mx1) : 1.f;
        if (mv0) ref0 = mx0;
        if (mv1) ref1 = mx1;
        l0 *= f0;
        l1 *= f1;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          o[j][0] *= f0; o[j][1] *= f0; o[j][2] *= f1; o[j][3] *= f1;
        }
      }
      float p[2][4];
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        p[n][0] = ex2(sc[n][0] - ref0);
        p[n][1] = ex2(sc[n][1] - ref0);
        p[n][2] = ex2(sc[n][2] - ref1);
        p[n][3] = ex2(sc[n][3] - ref1);
      }
      l0 += p[0][0] + p[0][1] + p[1][0] + p[1][1];
      l1 += p[0][2] + p[0][3] + p[1][2] + p[1][3];
      uint32_t pa[4] = {pack2(p[0][0], p[0][1]), pack2(p[0][2], p[0][3]),
                        pack2(p[1][0], p[1][1]), pack2(p[1][2], p[1][3])};
      {
        const int row = (jm & 1) * 8 + jr;
#pragma unroll
        for (int jp = 0; jp < 8; ++jp) {
          uint32_t vf[4];
          ldsm4t(vb + blk_off(row, 2 * jp + (jm >> 1)), vf);
          mma16816(o[2 * jp], pa, vf[0], vf[1]);
          mma16816(o[2 * jp + 1], pa, vf[2], vf[3]);
        }
      }
      // every lane has read the slot: the warp's own next copy may overwrite it (the rows
      // zeroed above were written through the generic proxy, the copy goes through the async one)
      if (nv < kBlock) fence_async_smem();
      __syncwarp();
      ++c_done;
    }
    if (!alive) break;
    // ---- this unit's rows: straight from the accumulator fragments
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    if (a.pdl && cur.fin_n > 0 && !waited) {   // the partial results folded below come from
      pdl_wait();                              // earlier kernels of the call
      waited = true;
    }
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int r = g + 8 * half;
      if (r < R) {
        const UserRef ur = s_users[r / G];
        const int head = cur.h * G + r % G;
        float L = half ? l1 : l0, M = half ? ref1 : ref0;
        for (int pj = 0; pj < cur.fin_n; ++pj) {
          const size_t prow = (size_t)(cur.fin_begin + pj) * HQ + head;
          if (a.part_flag && ((cur.fin_flags >> pj) & 1u)) {
            // produced by a plain unit of this very launch: claimed before this unit was (the
            // counter hands out plain units first), so it is running or done - wait for it
            uint32_t spins = 0;
            int ready;
            do {
              asm volatile("ld.acquire.gpu.global.s32 %0, [%1];"
                           : "=r"(ready) : "l"(a.part_flag + prow) : "memory");
              ready = ready == ready_mark;
            } while (!ready && ++spins < kSpin && !((spins & 255) == 255 && *cta_abort));
            if (!ready) {
              if (spins >= kSpin) atomicCAS(a.d_error, 0, 9500 + w);
              *cta_abort = 1;
              alive = false;
            }
          }
          const float2 ml = a.part_ml[prow];
          const float2* src = (const float2*)(a.part_o + prow * kDim) + tq;
          const float mn = fmaxf(M, ml.x);
          const float f0 = M == -INFINITY ? 0.f : ex2(M - mn);
          const float f1 = ml.x == -INFINITY ? 0.f : ex2(ml.x - mn);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 x = src[4 * j];
            o[j][2 * half] = o[j][2 * half] * f0 + x.x * f1;
            o[j][2 * half + 1] = o[j][2 * half + 1] * f0 + x.y * f1;
          }
          L = L * f0 + ml.y * f1;
          M = mn;
        }
        if (ur.slot < 0 || cur.fin_n > 0) {
          const float inv = 1.f / L;
          uint32_t* dst = (uint32_t*)a.out + ((size_t)ur.query * HQ + head) * 64 + tq;
#pragma unroll
          for (int j = 0; j < 16; ++j)
            dst[4 * j] = pack2(o[j][2 * half] * inv, o[j][2 * half + 1] * inv);
        } else {
          const size_t prow = (size_t)(ur.slot + cur.slot_add) * HQ + head;
          float2* dst = (float2*)(a.part_o + prow * kDim) + tq;
#pragma unroll
          for (int j = 0; j < 16; ++j) dst[4 * j] = make_float2(o[j][2 * half], o[j][2 * half + 1]);
          if (tq == 0) a.part_ml[prow] = make_float2(M, L);
        }
      }
    }
    // plain units of a launch that also holds finishing units: publish the partial rows
    if (a.part_flag && cur.fin_n == 0) {
      __syncwarp();
      if (tq == 0) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int r = g + 8 * half;
          if (r < R) {
            const UserRef ur = s_users[r / G];
            if (ur.slot >= 0) {
              __threadfence();
              *(volatile int*)(a.part_flag +
                               (size_t)(ur.slot + cur.slot_add) * HQ + cur.h * G + r % G) =
                  ready_mark;
            }
          }
        }
      }
    }
    if (!alive) break;
    // ---- on to the next unit: whatever of its background work is still open is finished now
    if (!nxt.valid) {
      if (no_more) break;
      fetch_to_end();
      nxt = nn;
      nn_final = false;
      q_phase = 0;
      if (!nxt.valid) break;
    }
    if (q_phase == 0) load_users(nxt);
    if (q_phase <= 1) load_q(nxt, which ^ 1, qn);
    cur = nxt;
    nxt.valid = false;
    which ^= 1;
    q_phase = 0;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
#pragma unroll
      for (int e = 0; e < 4; ++e) qa[ks][e] = qn[ks][e];
    // the load cursor is either already inside this unit or still at the end of the old one
    if (l_in_next) {
      l_in_next = false;
    } else {
      l_blk = 0;
      bid_ready = false;
    }
    if (nn_final) {                    // a fetch that finished in the meantime moves up
      nxt = nn;
      nn_final = false;
    }
  }
  // a warp that gave up still waits (with a limit of its own) for the copies it has in flight
  // before its shared memory goes away
  for (int c = c_done; !alive && c < c_load; ++c) {
    const uint32_t fb = full_bar(c % kSlots), par = (c / kSlots) & 1;
    for (uint32_t i = 0; i < kSpin && !bar_try(fb, par); ++i) {}
  }
  leave();
  if (a.pdl) pdl_wait();               // this grid completes after its predecessor
}

}  // namespace

cudaError_t launch_attention_ws(const AttnArgs& a, int item_begin, int n_items, cudaStream_t st,
                                int ticket_index) {
  if (n_items <= 0) return cudaSuccess;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_ws_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemW);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_ws_persist_kernel,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemWP);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const int hkv = a.shape.num_kv_heads;
  if (a.ws_mode != 1 && a.d_ticket != nullptr) {
    // persistent form: every warp of two resident CTAs per SM claims (item, kv head) units
    // (the counters put themselves back to zero at the end of every launch)
    const long long n_units = (long long)n_items * hkv;
    const int grid = (int)std::min<long long>((n_units + 3) / 4, 2LL * a.num_sms);
    return launch_kernel(attn_ws_persist_kernel, dim3(grid), dim3(128), kSmemWP, st, a.pdl != 0,
                         *a.tm_k, *a.tm_v, a, item_begin, (int)n_units,
                         a.d_ticket + 4 * ticket_index);
  }
  // Whole items per CTA when there are enough of them to fill the machine; otherwise the kv
  // heads are dealt out over several CTAs (in multiples of the four consumer warps).
  const int max_groups = (hkv + 3) / 4;
  const int want = (4 * a.num_sms + n_items - 1) / n_items;
  const int groups = want < 1 ? 1 : (want > max_groups ? max_groups : want);
  const int heads_per_cta = ((hkv + groups - 1) / groups + 3) / 4 * 4;
  const int grid_y = (hkv + heads_per_cta - 1) / heads_per_cta;
  return launch_kernel(attn_ws_kernel, dim3(n_items, grid_y), dim3(160), kSmemW, st, a.pdl != 0,
                       *a.tm_k, *a.tm_v, a, item_begin, heads_per_cta);
}

}  // namespace apar

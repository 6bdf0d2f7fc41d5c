// Tensor-core attention path for work items that carry several query rows (siblings that share
// a run of blocks, and the heads of a GQA group).
//
// One CTA owns one (work item, kv head).  A producer warp walks the block table and brings each
// 16-token block of K and V into shared memory with TMA tensor copies (two 64-dim halves per
// tile, 128-byte swizzle), three 64-token stages deep, handing stages over through mbarriers.
// Four consumer warps hold the query rows as MMA A-fragments (16 rows per warp tile) and run
// S = Q K^T and O += P V with mma.sync m16n8k16 (bf16 in, fp32 accumulate), with the online
// softmax kept in registers.  Work items with fewer than 49 rows split the tokens of a stage
// between warps and fold the partial states in shared memory at the end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "apar_internal.h"

namespace apar {
namespace {

constexpr int kStageTokens = 64;
constexpr int kStageBlocks = kStageTokens / kBlock;            // 4
constexpr int kStages = 3;
constexpr int kHalfBytes = kStageTokens * 128;                 // 64 tokens x 64 dims x 2 B = 8 KiB
constexpr int kKVBytes = 2 * kHalfBytes;                       // K (or V) of a stage: 16 KiB
constexpr int kStageBytes = 2 * kKVBytes;                      // 32 KiB
constexpr int kUsersOff = kStages * kStageBytes + 256;        // the item's UserRef entries (<= 64)
constexpr int kSmemBytes = kUsersOff + 64 * 8 + 1024 /*alignment*/;
constexpr int kOutPitch = kDim + 4;                            // floats per staged output row
constexpr uint32_t kSpinLimit = 1u << 20;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (or as soon as another warp gave up), raises the
// CTA's abort flag and the global error word, and lets the caller unwind.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* cta_abort,
                                          int* err_word) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023) == 1023 && *cta_abort) return false;
  }
  *cta_abort = 1;
  atomicExch(err_word, 1);
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"((uint64_t)map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void consumer_sync() {   // the four consumer warps only
  asm volatile("bar.sync 1, 128;" ::: "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {   // 2^x, flushes to zero, 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&v;
}

// Byte offset of (row, 16-byte chunk c of 16) inside a [2 halves][64 rows][64 dims] bf16 tile
// written by TMA with the 128-byte swizzle: chunk index xor (row mod 8) inside each 128-byte row.
__device__ __forceinline__ uint32_t tile_off(int row, int c) {
  return (uint32_t)((c >> 3) * kHalfBytes + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}

// MT = 16-row query tiles of the item (1..4).  SPLITS warps share one query tile and divide the
// blocks of every stage between them.
template <int MT>
__global__ void __launch_bounds__(160, 2)
attn_mma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                const AttnArgs a, int item_begin) {
  constexpr int SPLITS = MT == 1 ? 4 : (MT == 2 ? 2 : 1);
  constexpr int NBW = kStageBlocks / SPLITS;        // blocks of a stage per warp
  constexpr int ACTIVE = MT * SPLITS;               // consumer warps that compute

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kStages * kStageBytes;      // full[kStages], empty[kStages], q_done
  volatile int* cta_abort = (volatile int*)(base_ptr + kStages * kStageBytes + 128);
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
  const uint32_t q_done_bar = bars + 8u * (2 * kStages);

  const WorkItem it = a.d_items[item_begin + blockIdx.x];
  // an earlier CTA gave up a wait: do not pile up (one reader, so the whole CTA agrees)
  if (threadIdx.x == 0) *cta_abort = *(volatile int*)a.d_error;
  __syncthreads();
  if (*cta_abort) return;
  const int kvh = blockIdx.y;
  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  const int tok_end = it.tok_end < 0 ? a.d_lens[it.table_row] : it.tok_end;
  const int n_tok = tok_end - it.tok_begin;
  const int n_blk = (n_tok + kBlock - 1) / kBlock;
  const int n_tiles = (n_tok + kStageTokens - 1) / kStageTokens;
  const int32_t* table = a.d_tables + (size_t)it.table_row * a.shape.table_stride +
                         it.tok_begin / kBlock;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int R = it.n_users * G;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), ACTIVE);
    }
    mbar_init(q_done_bar, 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == 4) {
    // ------------------------------------------------------------------ producer warp
    // block ids are fetched 32 at a time (eight tiles), one batch ahead of their use, so that
    // no table read sits between two tiles
    int ids_cur = lane < n_blk ? table[lane] : 0;
    int ids_next = 32 + lane < n_blk ? table[32 + lane] : 0;
    for (int t = 0; t < n_tiles; ++t) {
      const int s = t % kStages;
      if (t > 0 && (t & 7) == 0) {
        ids_cur = ids_next;
        const int nxt = (t + 8) * kStageBlocks + lane;
        ids_next = nxt < n_blk ? table[nxt] : 0;
      }
      const int blk = t * kStageBlocks + (lane >> 2);
      const bool mine = lane < 4 * kStageBlocks && blk < n_blk;
      const int bid = __shfl_sync(0xffffffffu, ids_cur, blk & 31);
      if (t >= kStages) {
        if (!mbar_wait(empty_bar(s), ((t / kStages) - 1) & 1, cta_abort, a.d_error)) break;
      } else if (s == kStages - 1) {
        // the last stage first holds the query rows: wait until they sit in registers
        if (!mbar_wait(q_done_bar, 0, cta_abort, a.d_error)) break;
      }
      if (lane == 0) {
        const int nb = min(kStageBlocks, n_blk - t * kStageBlocks);
        mbar_expect_tx(full_bar(s), (uint32_t)nb * 2u * kTileBytes);
      }
      __syncwarp();
      if (mine) {
        const int which = lane & 3;                         // K lo, K hi, V lo, V hi
        const uint32_t dst = base + s * kStageBytes + (which >> 1) * kKVBytes +
                             (which & 1) * kHalfBytes + (lane >> 2) * (kBlock * 128);
        tma_load_2d(dst, (which >> 1) ? &tm_v : &tm_k, (which & 1) * 64,
                    (bid * HKV + kvh) * kBlock, full_bar(s));
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  // query rows -> shared memory (tile layout of a K stage, rows = query rows), zero padded
  UserRef* s_users = (UserRef*)(base_ptr + kUsersOff);
  if (threadIdx.x < it.n_users) s_users[threadIdx.x] = a.d_users[it.user_begin + threadIdx.x];
  consumer_sync();
  {
    const uint32_t qbase = base + (kStages - 1) * kStageBytes;
    uint8_t* qptr = base_ptr + (kStages - 1) * kStageBytes;
#pragma unroll
    for (int i = threadIdx.x; i < MT * 16 * 16; i += 128) {
      const int row = i >> 4, c = i & 15;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (row < R) {
        const int query = s_users[row / G].query;
        v = *((const uint4*)a.q + ((size_t)query * HQ + kvh * G + row % G) * 16 + c);
      }
      *(uint4*)(qptr + tile_off(row, c)) = v;
    }
    (void)qbase;
  }
  consumer_sync();
  const int mt = warp % MT, split = warp / MT;
  const bool active = warp < ACTIVE;
  uint32_t qa[8][4];
  {
    const uint32_t qbase = base + (kStages - 1) * kStageBytes;
    const int j = lane >> 3;
    const int row = mt * 16 + (j & 1) * 8 + (lane & 7);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) ldsm_x4(qbase + tile_off(row, 2 * ks + (j >> 1)), qa[ks]);
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(q_done_bar);

  float o[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const float c = a.scale_log2e;
  const int g = lane >> 2, tq = lane & 3;
  const int jm = lane >> 3, jr = lane & 7;                 // ldmatrix: matrix index, row in it

  if (active) {
    for (int t = 0; t < n_tiles; ++t) {
      const int s = t % kStages;
      if (!mbar_wait(full_bar(s), (t / kStages) & 1, cta_abort, a.d_error)) break;
      const uint32_t kb = base + s * kStageBytes, vb = kb + kKVBytes;
      const int tile_tok = min(kStageTokens, n_tok - t * kStageTokens);
      float sc[NBW * 2][4];
      bool any = false;
#pragma unroll
      for (int i = 0; i < NBW; ++i) {
        const int b = split * NBW + i;                     // block of the stage
        if (b * kBlock < tile_tok) {
          any = true;
          float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
          const int row = b * kBlock + (jm >> 1) * 8 + jr;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint32_t kf[4];
            ldsm_x4(kb + tile_off(row, 2 * ks + (jm & 1)), kf);
            mma_bf16(acc0, qa[ks], kf[0], kf[1]);
            mma_bf16(acc1, qa[ks], kf[2], kf[3]);
          }
          const int t0 = b * kBlock + 2 * tq;              // token of acc0[0] inside the tile
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int tok0 = t0 + (e & 1), tok1 = tok0 + 8;
            sc[2 * i][e] = tok0 < tile_tok ? acc0[e] * c : -INFINITY;
            sc[2 * i + 1][e] = tok1 < tile_tok ? acc1[e] * c : -INFINITY;
          }
          // rows of V past the valid length hold unspecified bits: zero them before P V
          const int nv = tile_tok - b * kBlock;
          if (nv < kBlock) {
            uint8_t* vptr = base_ptr + s * kStageBytes + kKVBytes;
            for (int x = lane; x < (kBlock - nv) * 16; x += 32)
              *(uint4*)(vptr + tile_off(b * kBlock + nv + (x >> 4), x & 15)) =
                  make_uint4(0u, 0u, 0u, 0u);
            __syncwarp();
          }
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) sc[2 * i][e] = sc[2 * i + 1][e] = -INFINITY;
        }
      }
      if (any) {
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < NBW * 2; ++n) {
          mx0 = fmaxf(mx0, fmaxf(sc[n][0], sc[n][1]));
          mx1 = fmaxf(mx1, fmaxf(sc[n][2], sc[n][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);   // finite: token 0 is valid
        const float cr0 = ex2(m0 - mn0), cr1 = ex2(m1 - mn1);
        m0 = mn0; m1 = mn1;
        float ps0 = 0.f, ps1 = 0.f;
        uint32_t pa[NBW][4];
#pragma unroll
        for (int i = 0; i < NBW; ++i) {
          float p[2][4];
#pragma unroll
          for (int n = 0; n < 2; ++n) {
            p[n][0] = ex2(sc[2 * i + n][0] - mn0);
            p[n][1] = ex2(sc[2 * i + n][1] - mn0);
            p[n][2] = ex2(sc[2 * i + n][2] - mn1);
            p[n][3] = ex2(sc[2 * i + n][3] - mn1);
            ps0 += p[n][0] + p[n][1];
            ps1 += p[n][2] + p[n][3];
          }
          pa[i][0] = pack_bf16(p[0][0], p[0][1]);
          pa[i][1] = pack_bf16(p[0][2], p[0][3]);
          pa[i][2] = pack_bf16(p[1][0], p[1][1]);
          pa[i][3] = pack_bf16(p[1][2], p[1][3]);
        }
        l0 = l0 * cr0 + ps0;
        l1 = l1 * cr1 + ps1;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          o[j][0] *= cr0; o[j][1] *= cr0; o[j][2] *= cr1; o[j][3] *= cr1;
        }
#pragma unroll
        for (int i = 0; i < NBW; ++i) {
          const int b = split * NBW + i;
          if (b * kBlock < tile_tok) {
            const int row = b * kBlock + (jm & 1) * 8 + jr;
#pragma unroll
            for (int jp = 0; jp < 8; ++jp) {
              uint32_t vf[4];
              ldsm_x4_trans(vb + tile_off(row, 2 * jp + (jm >> 1)), vf);
              mma_bf16(o[2 * jp], pa[i], vf[0], vf[1]);
              mma_bf16(o[2 * jp + 1], pa[i], vf[2], vf[3]);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(s));
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  }

  // ---- fold the warps that share a query tile and write the rows out
  consumer_sync();                       // every stage has been consumed: reuse it as staging
  float* so = (float*)base_ptr;                              // [4 warps][16][kOutPitch]
  float* sml = so + 4 * 16 * kOutPitch;                      // [4 warps][16][2]
  if (active) {
    float* mine = so + warp * 16 * kOutPitch;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      *(float2*)(mine + g * kOutPitch + 8 * j + 2 * tq) = make_float2(o[j][0], o[j][1]);
      *(float2*)(mine + (g + 8) * kOutPitch + 8 * j + 2 * tq) = make_float2(o[j][2], o[j][3]);
    }
    if (tq == 0) {
      sml[(warp * 16 + g) * 2] = m0;       sml[(warp * 16 + g) * 2 + 1] = l0;
      sml[(warp * 16 + g + 8) * 2] = m1;   sml[(warp * 16 + g + 8) * 2 + 1] = l1;
    }
  }
  consumer_sync();
  const int d = threadIdx.x;                                 // one output dim per thread
#pragma unroll 4
  for (int r = 0; r < R; ++r) {
    const int rmt = r >> 4, ri = r & 15;
    float M = -INFINITY;
#pragma unroll
    for (int sp = 0; sp < SPLITS; ++sp) M = fmaxf(M, sml[((rmt + MT * sp) * 16 + ri) * 2]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int sp = 0; sp < SPLITS; ++sp) {
      const int w = rmt + MT * sp;
      const float mw = sml[(w * 16 + ri) * 2];
      const float wgt = mw == -INFINITY ? 0.f : ex2(mw - M);
      L += sml[(w * 16 + ri) * 2 + 1] * wgt;
      O += so[(w * 16 + ri) * kOutPitch + d] * wgt;
    }
    const UserRef ur = s_users[r / G];
    const int head = kvh * G + r % G;
    if (ur.slot < 0) {
      ((__nv_bfloat16*)a.out)[((size_t)ur.query * HQ + head) * kDim + d] =
          __float2bfloat16_rn(O / L);
    } else {
      const size_t prow = (size_t)(ur.slot + it.slot_add) * HQ + head;
      a.part_o[prow * kDim + d] = O;
      if (d == 0) a.part_ml[prow] = make_float2(M, L);
    }
  }
}

template <int MT>
cudaError_t launch_mt(const AttnArgs& a, int item_begin, int n_items, cudaStream_t st) {
  if (n_items <= 0) return cudaSuccess;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_mma_kernel<MT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  attn_mma_kernel<MT><<<dim3(n_items, a.shape.num_kv_heads), 160, kSmemBytes, st>>>(
      *a.tm_k, *a.tm_v, a, item_begin);
  return cudaGetLastError();
}

}  // namespace

// Items must be grouped by query-tile count: counts[i] items need i+1 tiles of 16 rows.
cudaError_t launch_attention_mma(const AttnArgs& a, int item_begin, const int32_t* counts,
                                 cudaStream_t st) {
  cudaError_t e = cudaSuccess;
  int at = item_begin;
  if (e == cudaSuccess) e = launch_mt<4>(a, at, counts[3], st);
  at += counts[3];
  if (e == cudaSuccess) e = launch_mt<3>(a, at, counts[2], st);
  at += counts[2];
  if (e == cudaSuccess) e = launch_mt<2>(a, at, counts[1], st);
  at += counts[1];
  if (e == cudaSuccess) e = launch_mt<1>(a, at, counts[0], st);
  return e;
}

// Tensor maps over the K and V pools seen as 2-D bf16 arrays [num_blocks*num_kv_heads*16][128];
// a box is one 64-dim half of a 16-token tile, stored with the 128-byte swizzle.
int make_pool_tensor_maps(void* k_pool, void* v_pool, int64_t num_blocks, int num_kv_heads,
                          CUtensorMap* tm_k, CUtensorMap* tm_v) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                               const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                               const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) !=
          cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess)
    return -1;
  const cuuint64_t dims[2] = {(cuuint64_t)kDim, (cuuint64_t)num_blocks * num_kv_heads * kBlock};
  const cuuint64_t strides[1] = {(cuuint64_t)kDim * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)kBlock};
  const cuuint32_t estr[2] = {1, 1};
  void* pools[2] = {k_pool, v_pool};
  CUtensorMap* maps[2] = {tm_k, tm_v};
  for (int i = 0; i < 2; ++i) {
    CUresult r = ((EncodeFn)fn)(maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pools[i], dims,
                                strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return (int)r;
  }
  return 0;
}

}  // namespace apar

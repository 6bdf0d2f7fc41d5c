// CUDA kernels of the APAR decode hot path for sm_100a: copy-on-fork of a partial block,
// KV append scatter, device-table sync, the vectorised CUDA-core attention path for
// work items with few query rows (private tails under MHA), and the cross-item merge.
#include <algorithm>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "apar_internal.h"

namespace apar {

// ------------------------------------------------------------------ fork: copy r rows
// One CTA per (copy, kv head, K|V): the r valid rows of a (block, head) tile are r * 256
// contiguous bytes.
__global__ void __launch_bounds__(128) cow_copy_kernel(uint4* __restrict__ k_pool,
                                                       uint4* __restrict__ v_pool,
                                                       const CowCopy* __restrict__ copies,
                                                       int num_kv_heads) {
  const CowCopy c = copies[blockIdx.x];
  uint4* pool = blockIdx.z ? v_pool : k_pool;
  const size_t tile = kTileBytes / 16;
  const uint4* src = pool + ((size_t)c.src_block * num_kv_heads + blockIdx.y) * tile;
  uint4* dst = pool + ((size_t)c.dst_block * num_kv_heads + blockIdx.y) * tile;
  const int n = c.rows * (kDim * 2 / 16);
  for (int i = threadIdx.x; i < n; i += blockDim.x) dst[i] = src[i];
}

cudaError_t launch_cow_copy(void* k_pool, void* v_pool, const CowCopy* d_copies, int n,
                            int num_kv_heads, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  cow_copy_kernel<<<dim3(n, num_kv_heads, 2), 128, 0, st>>>((uint4*)k_pool, (uint4*)v_pool,
                                                            d_copies, num_kv_heads);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ append: scatter new rows
// One thread per 16 bytes of a new row; blockIdx.y selects K or V.
__global__ void __launch_bounds__(256) append_kernel(uint4* __restrict__ k_pool,
                                                     uint4* __restrict__ v_pool,
                                                     const uint4* __restrict__ k_new,
                                                     const uint4* __restrict__ v_new,
                                                     const int32_t* __restrict__ slots,
                                                     long long first_row, int n_rows,
                                                     int num_kv_heads) {
  const int per_row = num_kv_heads * 16;                 // 16-byte pieces per token row
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_rows * per_row) return;
  const int r = (int)(idx / per_row), rem = (int)(idx % per_row);
  const int h = rem >> 4, c = rem & 15;
  const int slot = slots[r];
  const int block = slot >> 4, off = slot & 15;
  const uint4* src = (blockIdx.y ? v_new : k_new) + (first_row + r) * per_row + rem;
  uint4* dst = (blockIdx.y ? v_pool : k_pool) +
               (((size_t)block * num_kv_heads + h) * kBlock + off) * 16 + c;
  *dst = *src;
}

cudaError_t launch_append(void* k_pool, void* v_pool, const void* k_new, const void* v_new,
                          const int32_t* d_slots, int64_t first_row, int n_rows,
                          int num_kv_heads, cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  const long long total = (long long)n_rows * num_kv_heads * 16;
  const unsigned grid = (unsigned)((total + 255) / 256);
  append_kernel<<<dim3(grid, 2), 256, 0, st>>>((uint4*)k_pool, (uint4*)v_pool,
                                               (const uint4*)k_new, (const uint4*)v_new, d_slots,
                                               (long long)first_row, n_rows, num_kv_heads);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ device table / length sync
__global__ void __launch_bounds__(128) sync_kernel(int32_t* __restrict__ tables, int stride,
                                                   int32_t* __restrict__ lens,
                                                   const TableDelta* __restrict__ deltas,
                                                   const int32_t* __restrict__ data, int n_deltas,
                                                   const int32_t* __restrict__ pairs, int n_pairs) {
  if ((int)blockIdx.x < n_deltas) {
    const TableDelta d = deltas[blockIdx.x];
    int32_t* dst = tables + (size_t)d.row * stride + d.pos;
    const int32_t* src = data + d.data_off;
    for (int i = threadIdx.x; i < d.count; i += blockDim.x) dst[i] = src[i];
  } else {
    const int i = ((int)blockIdx.x - n_deltas) * blockDim.x + threadIdx.x;
    if (i < n_pairs) lens[pairs[2 * i]] = pairs[2 * i + 1];
  }
}

cudaError_t launch_sync(int32_t* d_tables, int table_stride, int32_t* d_lens,
                        const TableDelta* d_deltas, const int32_t* d_data, int n_deltas,
                        const int32_t* d_len_pairs, int n_pairs, cudaStream_t st) {
  const int grid = n_deltas + (n_pairs + 127) / 128;
  if (grid <= 0) return cudaSuccess;
  sync_kernel<<<grid, 128, 0, st>>>(d_tables, table_stride, d_lens, d_deltas, d_data, n_deltas,
                                    d_len_pairs, n_pairs);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ decode step: lengths and slots
// One thread per entry of the step's thread list: the device length of the thread's table row
// goes up by one and the pool slot of its new row (block * 16 + offset) is written to the slot
// map that the scatter kernels of all layers read.  A thread that starts a new block this step
// gets the block from the host: pair j = (list position, table row, table position, block id),
// written into the device table here; its slot is the first row of that block.  The two kinds
// of work touch disjoint words, so one launch does both.
__global__ void __launch_bounds__(256) step_advance_kernel(int32_t* __restrict__ tables, int stride,
                                                           int32_t* __restrict__ lens,
                                                           const int32_t* __restrict__ step_rows,
                                                           int n, const int4* __restrict__ pairs,
                                                           int n_pairs,
                                                           int32_t* __restrict__ slot_map) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    const int row = step_rows[i];
    const int len = lens[row];
    lens[row] = len + 1;
    if (len & (kBlock - 1))
      slot_map[i] = tables[(size_t)row * stride + (len >> 4)] * kBlock + (len & (kBlock - 1));
  }
  if (i < n_pairs) {
    const int4 p = pairs[i];
    tables[(size_t)p.y * stride + p.z] = p.w;
    slot_map[p.x] = p.w * kBlock;
  }
}

cudaError_t launch_step_advance(int32_t* d_tables, int table_stride, int32_t* d_lens,
                                const int32_t* d_step_rows, int n, const void* d_pairs,
                                int n_pairs, int32_t* d_slot_map, cudaStream_t st) {
  const int work = n > n_pairs ? n : n_pairs;
  if (work <= 0) return cudaSuccess;
  step_advance_kernel<<<(work + 255) / 256, 256, 0, st>>>(d_tables, table_stride, d_lens,
                                                          d_step_rows, n, (const int4*)d_pairs,
                                                          n_pairs, d_slot_map);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ attention, vector path
__device__ __forceinline__ void bf16x8_to_float(const uint4& u, float* f) {
  f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
  f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
  f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xffff0000u);
  f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xffff0000u);
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// A CTA of four warps owns one (work item, kv head).  Each warp takes every fourth block of
// the item.  A 16-token tile of K (4 KiB) is fetched with eight coalesced 16-byte loads per
// lane: load j brings tokens 2j (lanes 0-15) and 2j+1 (lanes 16-31), lane c of a half holding
// dims [8c, 8c+8).  Scores are reduced over the 16 lanes of a half with shuffles; the online
// softmax state (m, l) is kept identical in both halves, o is per half and folded at the end.
// ROWS query rows are carried at once; items with more rows loop over groups of ROWS.
template <int ROWS>
__global__ void __launch_bounds__(128) attn_vec_kernel(const AttnArgs a, int item_begin) {
  const WorkItem it = a.d_items[item_begin + blockIdx.x];
  const int kvh = blockIdx.y;
  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  const int tok_end = it.tok_end < 0 ? a.d_lens[it.table_row] : it.tok_end;
  const int n_tok = tok_end - it.tok_begin;
  const int n_blk = (n_tok + kBlock - 1) / kBlock;
  const int32_t* table = a.d_tables + (size_t)it.table_row * a.shape.table_stride +
                         it.tok_begin / kBlock;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, c = lane & 15;
  const int R = it.n_users * G;

  __shared__ float sm_m[4][ROWS], sm_l[4][ROWS];
  __shared__ __align__(16) float sm_o[4][ROWS][kDim];

  for (int r0 = 0; r0 < R; r0 += ROWS) {
    float qf[ROWS][8], o[ROWS][8], m[ROWS], l[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      m[r] = -INFINITY;
      l[r] = 0.f;
#pragma unroll
      for (int d = 0; d < 8; ++d) { o[r][d] = 0.f; qf[r][d] = 0.f; }
      if (r0 + r < R) {
        const int u = (r0 + r) / G, hg = (r0 + r) % G;
        const int query = a.d_users[it.user_begin + u].query;
        const uint4 qv = *((const uint4*)a.q + ((size_t)query * HQ + kvh * G + hg) * 16 + c);
        bf16x8_to_float(qv, qf[r]);
#pragma unroll
        for (int d = 0; d < 8; ++d) qf[r][d] *= a.scale_log2e;
      }
    }
    for (int b = warp; b < n_blk; b += 4) {
      const int bid = table[b];
      const size_t tile = ((size_t)bid * HKV + kvh) * (kTileBytes / 16);
      const uint4* kt = (const uint4*)a.k_pool + tile + half * 16 + c;
      const uint4* vt = (const uint4*)a.v_pool + tile + half * 16 + c;
      const int nv = min(kBlock, n_tok - b * kBlock);
      uint4 kk[8], vv[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) kk[j] = ld_stream(kt + j * 32);
#pragma unroll
      for (int j = 0; j < 8; ++j) vv[j] = ld_stream(vt + j * 32);
      float s[ROWS][8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float kf[8];
        bf16x8_to_float(kk[j], kf);
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
          float acc = 0.f;
#pragma unroll
          for (int d = 0; d < 8; ++d) acc = fmaf(qf[r][d], kf[d], acc);
          s[r][j] = acc;
        }
      }
#pragma unroll
      for (int r = 0; r < ROWS; ++r)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float x = s[r][j];
          x += __shfl_xor_sync(0xffffffffu, x, 8);
          x += __shfl_xor_sync(0xffffffffu, x, 4);
          x += __shfl_xor_sync(0xffffffffu, x, 2);
          x += __shfl_xor_sync(0xffffffffu, x, 1);
          s[r][j] = (2 * j + half < nv) ? x : -INFINITY;   // rows past the length are never used
        }
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        float bm = s[r][0];
#pragma unroll
        for (int j = 1; j < 8; ++j) bm = fmaxf(bm, s[r][j]);
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));   // token 0 is always valid
        const float mn = fmaxf(m[r], bm);
        const float corr = exp2f(m[r] - mn);
        m[r] = mn;
        float ps = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          s[r][j] = exp2f(s[r][j] - mn);
          ps += s[r][j];
        }
        l[r] = l[r] * corr + ps;
#pragma unroll
        for (int d = 0; d < 8; ++d) o[r][d] *= corr;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float vf[8];
        bf16x8_to_float(vv[j], vf);
        if (2 * j + half >= nv) {          // unspecified bits (possibly NaN patterns): drop them
#pragma unroll
          for (int d = 0; d < 8; ++d) vf[d] = 0.f;
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r)
#pragma unroll
          for (int d = 0; d < 8; ++d) o[r][d] = fmaf(s[r][j], vf[d], o[r][d]);
      }
    }
    // fold the two halves of the warp, then the four warps
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      l[r] += __shfl_xor_sync(0xffffffffu, l[r], 16);
#pragma unroll
      for (int d = 0; d < 8; ++d) o[r][d] += __shfl_xor_sync(0xffffffffu, o[r][d], 16);
      if (half == 0) {
#pragma unroll
        for (int d = 0; d < 8; ++d) sm_o[warp][r][8 * c + d] = o[r][d];
      }
      if (lane == 0) { sm_m[warp][r] = m[r]; sm_l[warp][r] = l[r]; }
    }
    __syncthreads();
    const int t = threadIdx.x;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      if (r0 + r < R) {
        const float M = fmaxf(fmaxf(sm_m[0][r], sm_m[1][r]), fmaxf(sm_m[2][r], sm_m[3][r]));
        float L = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const float wgt = sm_m[w][r] == -INFINITY ? 0.f : exp2f(sm_m[w][r] - M);
          L += sm_l[w][r] * wgt;
          O += sm_o[w][r][t] * wgt;
        }
        const int u = (r0 + r) / G, hg = (r0 + r) % G;
        const UserRef ur = a.d_users[it.user_begin + u];
        const int head = kvh * G + hg;
        if (ur.slot < 0) {
          // an empty range (no tokens at all) has L = 0: its output is defined as zero
          ((__nv_bfloat16*)a.out)[((size_t)ur.query * HQ + head) * kDim + t] =
              __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
        } else {
          const size_t prow = (size_t)(ur.slot + it.slot_add) * HQ + head;
          a.part_o[prow * kDim + t] = O;
          if (t == 0) a.part_ml[prow] = make_float2(M, L);
        }
      }
    }
    __syncthreads();
  }
}

// Single-row items (a private tail read by one query, MHA): one CTA per item, and each of its
// four warps walks whole kv heads on its own - warp w takes heads w, w+4, ... of the CTA's
// group - so there is nothing to fold between warps, no shared memory and no CTA barrier, and
// the fixed cost of a CTA is paid once per item instead of once per (item, head).  Loads are
// the same coalesced 16-byte pattern as above; the block id of the next tile is fetched one
// tile ahead.
__global__ void __launch_bounds__(128) attn_vec_heads_kernel(const AttnArgs a, int item_begin,
                                                             int heads_per_cta) {
  const WorkItem it = a.d_items[item_begin + blockIdx.x];
  const int HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;   // equal: group == 1
  const int tok_end = it.tok_end < 0 ? a.d_lens[it.table_row] : it.tok_end;
  const int n_tok = tok_end - it.tok_begin;
  const int n_blk = (n_tok + kBlock - 1) / kBlock;
  const int32_t* table = a.d_tables + (size_t)it.table_row * a.shape.table_stride +
                         it.tok_begin / kBlock;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, c = lane & 15;
  const UserRef ur = a.d_users[it.user_begin];
  const int h_begin = blockIdx.y * heads_per_cta;
  const int h_end = min(HKV, h_begin + heads_per_cta);

  for (int h = h_begin + warp; h < h_end; h += 4) {
    float qf[8], o[8];
    {
      const uint4 qv = __ldg((const uint4*)a.q + ((size_t)ur.query * HQ + h) * 16 + c);
      bf16x8_to_float(qv, qf);
#pragma unroll
      for (int d = 0; d < 8; ++d) { qf[d] *= a.scale_log2e; o[d] = 0.f; }
    }
    float m = -INFINITY, l = 0.f;
    int bid = n_blk > 0 ? table[0] : 0;
    for (int b = 0; b < n_blk; ++b) {
      const int bid_next = b + 1 < n_blk ? table[b + 1] : 0;
      const size_t tile = ((size_t)bid * HKV + h) * (kTileBytes / 16);
      const uint4* kt = (const uint4*)a.k_pool + tile + half * 16 + c;
      const uint4* vt = (const uint4*)a.v_pool + tile + half * 16 + c;
      const int nv = min(kBlock, n_tok - b * kBlock);
      uint4 kk[8], vv[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) kk[j] = ld_stream(kt + j * 32);
#pragma unroll
      for (int j = 0; j < 8; ++j) vv[j] = ld_stream(vt + j * 32);
      float s[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float kf[8];
        bf16x8_to_float(kk[j], kf);
        float acc = 0.f;
#pragma unroll
        for (int d = 0; d < 8; ++d) acc = fmaf(qf[d], kf[d], acc);
        s[j] = acc;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float x = s[j];
        x += __shfl_xor_sync(0xffffffffu, x, 8);
        x += __shfl_xor_sync(0xffffffffu, x, 4);
        x += __shfl_xor_sync(0xffffffffu, x, 2);
        x += __shfl_xor_sync(0xffffffffu, x, 1);
        s[j] = (2 * j + half < nv) ? x : -INFINITY;      // rows past the length are never used
      }
      float bm = s[0];
#pragma unroll
      for (int j = 1; j < 8; ++j) bm = fmaxf(bm, s[j]);
      bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));   // token 0 is always valid
      const float mn = fmaxf(m, bm);
      const float corr = exp2f(m - mn);
      m = mn;
      float ps = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        s[j] = exp2f(s[j] - mn);
        ps += s[j];
      }
      l = l * corr + ps;
#pragma unroll
      for (int d = 0; d < 8; ++d) o[d] *= corr;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float vf[8];
        bf16x8_to_float(vv[j], vf);
        if (2 * j + half >= nv) {          // unspecified bits (possibly NaN patterns): drop them
#pragma unroll
          for (int d = 0; d < 8; ++d) vf[d] = 0.f;
        }
#pragma unroll
        for (int d = 0; d < 8; ++d) o[d] = fmaf(s[j], vf[d], o[d]);
      }
      bid = bid_next;
    }
    l += __shfl_xor_sync(0xffffffffu, l, 16);
#pragma unroll
    for (int d = 0; d < 8; ++d) o[d] += __shfl_xor_sync(0xffffffffu, o[d], 16);
    if (half == 0) {
      // a finishing item folds the partial results of the rest of the chain into its own
      for (int j = 0; j < fin_count(it); ++j) {
        const size_t prow = (size_t)(it.fin_begin + j) * HQ + h;
        const float2 ml = a.part_ml[prow];
        const float4* src = (const float4*)(a.part_o + prow * kDim) + 2 * c;
        const float4 x0 = src[0], x1 = src[1];
        const float mn = fmaxf(m, ml.x);
        const float f0 = m == -INFINITY ? 0.f : exp2f(m - mn);
        const float f1 = ml.x == -INFINITY ? 0.f : exp2f(ml.x - mn);
        o[0] = o[0] * f0 + x0.x * f1; o[1] = o[1] * f0 + x0.y * f1;
        o[2] = o[2] * f0 + x0.z * f1; o[3] = o[3] * f0 + x0.w * f1;
        o[4] = o[4] * f0 + x1.x * f1; o[5] = o[5] * f0 + x1.y * f1;
        o[6] = o[6] * f0 + x1.z * f1; o[7] = o[7] * f0 + x1.w * f1;
        l = l * f0 + ml.y * f1;
        m = mn;
      }
      if (ur.slot < 0 || fin_count(it) > 0) {
        const float inv = l > 0.f ? 1.f / l : 0.f;      // no tokens at all: zeros
        __nv_bfloat162 p0 = __floats2bfloat162_rn(o[0] * inv, o[1] * inv);
        __nv_bfloat162 p1 = __floats2bfloat162_rn(o[2] * inv, o[3] * inv);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(o[4] * inv, o[5] * inv);
        __nv_bfloat162 p3 = __floats2bfloat162_rn(o[6] * inv, o[7] * inv);
        uint4 packed;
        packed.x = *(uint32_t*)&p0; packed.y = *(uint32_t*)&p1;
        packed.z = *(uint32_t*)&p2; packed.w = *(uint32_t*)&p3;
        ((uint4*)((__nv_bfloat16*)a.out + ((size_t)ur.query * HQ + h) * kDim))[c] = packed;
      } else {
        const size_t prow = (size_t)(ur.slot + it.slot_add) * HQ + h;
        float4* dst = (float4*)(a.part_o + prow * kDim) + 2 * c;
        dst[0] = make_float4(o[0], o[1], o[2], o[3]);
        dst[1] = make_float4(o[4], o[5], o[6], o[7]);
        if (c == 0) a.part_ml[prow] = make_float2(m, l);
      }
    }
  }
}

cudaError_t launch_attention_vec(const AttnArgs& a, int item_begin, int n_items, bool single_row,
                                 cudaStream_t st) {
  if (n_items <= 0) return cudaSuccess;
  if (single_row) {
    // whole items per CTA when there are enough of them; otherwise heads are dealt out over
    // several CTAs (multiples of the four warps) until the machine is full
    const int hkv = a.shape.num_kv_heads;
    const int max_groups = (hkv + 3) / 4;
    const int want = (5 * a.num_sms + n_items - 1) / n_items;
    const int groups = want < 1 ? 1 : (want > max_groups ? max_groups : want);
    const int heads_per_cta = ((hkv + groups - 1) / groups + 3) / 4 * 4;
    const dim3 grid(n_items, (hkv + heads_per_cta - 1) / heads_per_cta);
    attn_vec_heads_kernel<<<grid, 128, 0, st>>>(a, item_begin, heads_per_cta);
  } else {
    attn_vec_kernel<4><<<dim3(n_items, a.shape.num_kv_heads), 128, 0, st>>>(a, item_begin);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------ verification: candidate part
// One CTA per (candidate query, kv head); warp w takes the query heads w, w + 4, ... of the
// group.  The candidates are at most 64 rows that were appended a moment ago, so they are read
// straight from global memory, two tokens per step (one per half-warp, lane c of a half
// holding dims [8c, 8c + 8) as in the vector path); a token outside the mask is skipped.
__global__ void __launch_bounds__(128) verify_tail_kernel(const AttnArgs a,
                                                          const VerifyDesc* __restrict__ descs) {
  const VerifyDesc d = descs[blockIdx.x];
  const int kvh = blockIdx.y;
  const int G = a.shape.group, HQ = a.shape.num_q_heads, HKV = a.shape.num_kv_heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, c = lane & 15;
  const int32_t* table = a.d_tables + (size_t)d.row * a.shape.table_stride;
  for (int hg = warp; hg < G; hg += 4) {
    const int head = kvh * G + hg;
    float qf[8], o[8];
    {
      const uint4 qv = __ldg((const uint4*)a.q + ((size_t)d.query * HQ + head) * 16 + c);
      bf16x8_to_float(qv, qf);
#pragma unroll
      for (int x = 0; x < 8; ++x) { qf[x] *= a.scale_log2e; o[x] = 0.f; }
    }
    float m = -INFINITY, l = 0.f;
    for (int i0 = 0; i0 < d.n_cand; i0 += 2) {
      const int i = i0 + half;
      const bool on = i < d.n_cand && ((d.mask >> i) & 1ull);
      float s = -INFINITY;
      uint4 vv = make_uint4(0u, 0u, 0u, 0u);
      if (on) {
        const int pos = d.base + i;
        const size_t rowoff =
            (((size_t)table[pos >> 4] * HKV + kvh) * kBlock + (pos & (kBlock - 1))) * 16 + c;
        const uint4 kk = ld_stream((const uint4*)a.k_pool + rowoff);
        vv = ld_stream((const uint4*)a.v_pool + rowoff);
        float kf[8];
        bf16x8_to_float(kk, kf);
        s = 0.f;
#pragma unroll
        for (int x = 0; x < 8; ++x) s = fmaf(qf[x], kf[x], s);
      }
      // sum over the 16 lanes of a half (both halves shuffle, masked-off ones carry -inf)
      float t = on ? s : 0.f;
      t += __shfl_xor_sync(0xffffffffu, t, 8);
      t += __shfl_xor_sync(0xffffffffu, t, 4);
      t += __shfl_xor_sync(0xffffffffu, t, 2);
      t += __shfl_xor_sync(0xffffffffu, t, 1);
      s = on ? t : -INFINITY;
      const float other = __shfl_xor_sync(0xffffffffu, s, 16);
      const float mn = fmaxf(m, fmaxf(s, other));
      if (mn == -INFINITY) continue;               // both tokens masked, nothing seen yet
      const float corr = exp2f(m - mn);             // m = -inf gives 0
      const float p = on ? exp2f(s - mn) : 0.f;
      const float p_other = other == -INFINITY ? 0.f : exp2f(other - mn);
      m = mn;
      l = l * corr + p + p_other;                   // kept identical in both halves
      float vf[8];
      bf16x8_to_float(vv, vf);
#pragma unroll
      for (int x = 0; x < 8; ++x) o[x] = fmaf(p, vf[x], o[x] * corr);
    }
#pragma unroll
    for (int x = 0; x < 8; ++x) o[x] += __shfl_xor_sync(0xffffffffu, o[x], 16);
    if (half == 0) {
      if (d.slot < 0) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        __nv_bfloat162 p0 = __floats2bfloat162_rn(o[0] * inv, o[1] * inv);
        __nv_bfloat162 p1 = __floats2bfloat162_rn(o[2] * inv, o[3] * inv);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(o[4] * inv, o[5] * inv);
        __nv_bfloat162 p3 = __floats2bfloat162_rn(o[6] * inv, o[7] * inv);
        uint4 packed;
        packed.x = *(uint32_t*)&p0; packed.y = *(uint32_t*)&p1;
        packed.z = *(uint32_t*)&p2; packed.w = *(uint32_t*)&p3;
        ((uint4*)((__nv_bfloat16*)a.out + ((size_t)d.query * HQ + head) * kDim))[c] = packed;
      } else {
        const size_t prow = (size_t)d.slot * HQ + head;
        float4* dst = (float4*)(a.part_o + prow * kDim) + 2 * c;
        dst[0] = make_float4(o[0], o[1], o[2], o[3]);
        dst[1] = make_float4(o[4], o[5], o[6], o[7]);
        if (c == 0) a.part_ml[prow] = make_float2(m, l);
      }
    }
  }
}

cudaError_t launch_verify_tail(const AttnArgs& a, const VerifyDesc* d_desc, int n_desc,
                               cudaStream_t st) {
  if (n_desc <= 0) return cudaSuccess;
  verify_tail_kernel<<<dim3(n_desc, a.shape.num_kv_heads), 128, 0, st>>>(a, d_desc);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ accepted candidates: row moves
// One CTA per (group of moves, kv head, K|V).  A group holds the rows one thread keeps (at
// most 64); sources and destinations of a group may overlap, so every source row is read into
// shared memory before the first destination row is written.
__global__ void __launch_bounds__(256) row_move_kernel(uint4* __restrict__ k_pool,
                                                       uint4* __restrict__ v_pool,
                                                       const RowMove* __restrict__ moves,
                                                       const int32_t* __restrict__ group_begin,
                                                       int num_kv_heads) {
  __shared__ uint4 rows[64 * 16];
  const int m0 = group_begin[blockIdx.x], m1 = group_begin[blockIdx.x + 1];
  uint4* pool = blockIdx.z ? v_pool : k_pool;
  const int h = blockIdx.y;
  for (int x = threadIdx.x; x < (m1 - m0) * 16; x += blockDim.x) {
    const int slot = moves[m0 + (x >> 4)].src_slot;
    rows[x] = pool[(((size_t)(slot >> 4) * num_kv_heads + h) * kBlock + (slot & 15)) * 16 + (x & 15)];
  }
  __syncthreads();
  for (int x = threadIdx.x; x < (m1 - m0) * 16; x += blockDim.x) {
    const int slot = moves[m0 + (x >> 4)].dst_slot;
    pool[(((size_t)(slot >> 4) * num_kv_heads + h) * kBlock + (slot & 15)) * 16 + (x & 15)] = rows[x];
  }
}

cudaError_t launch_row_moves(void* k_pool, void* v_pool, const RowMove* d_moves,
                             const int32_t* d_group_begin, int n_groups, int num_kv_heads,
                             cudaStream_t st) {
  if (n_groups <= 0) return cudaSuccess;
  row_move_kernel<<<dim3(n_groups, num_kv_heads, 2), 256, 0, st>>>(
      (uint4*)k_pool, (uint4*)v_pool, d_moves, d_group_begin, num_kv_heads);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ staging upload
// Moves a staged host buffer (pinned, mapped) into device memory with SM loads over PCIe
// instead of a copy engine.  The library's uploads are small (slot lists, table deltas, plan
// pieces) but sit on the critical path of a step; on a copy engine they queue behind whatever
// large host-to-device copy the application has in flight on another stream.
__global__ void __launch_bounds__(256) stage_copy_kernel(uint32_t* __restrict__ dst,
                                                         const uint32_t* __restrict__ src_mapped,
                                                         size_t n_words) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += stride)
    dst[i] = src_mapped[i];
}

cudaError_t launch_stage_copy(void* dst, const void* src_mapped, size_t bytes, cudaStream_t st) {
  const size_t n = bytes / 4;
  if (n == 0) return cudaSuccess;
  const int blocks = (int)std::min<size_t>((n + 255) / 256, 1024);
  stage_copy_kernel<<<blocks, 256, 0, st>>>((uint32_t*)dst, (const uint32_t*)src_mapped, n);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ read-only streaming probe
// Reads a buffer once with the same 16-byte streaming loads as the attention kernels and folds
// what it read into one word, so that the loads cannot be dropped.  Its rate is the ceiling for
// a kernel that only reads HBM.
__global__ void __launch_bounds__(256) stream_read_kernel(const uint4* __restrict__ src, size_t n16,
                                                          unsigned long long* __restrict__ sink) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t acc = 0;
  for (; i + 7 * stride < n16; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = ld_stream(src + i + k * stride);
#pragma unroll
    for (int k = 0; k < 8; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  for (; i < n16; i += stride) {
    const uint4 v = ld_stream(src + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0 && acc != 0) atomicXor(sink, (unsigned long long)acc);
}

cudaError_t launch_stream_read(const void* src, size_t bytes, void* sink, int num_sms,
                               cudaStream_t st) {
  if (bytes < 16) return cudaSuccess;
  stream_read_kernel<<<num_sms * 8, 256, 0, st>>>((const uint4*)src, bytes / 16,
                                                  (unsigned long long*)sink);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ merge of partial results
// One warp per (query, head): out = sum_j o_j 2^(m_j - M) / sum_j l_j 2^(m_j - M).
__global__ void __launch_bounds__(128) merge_kernel(const AttnArgs a,
                                                    const MergeRef* __restrict__ merges) {
  const MergeRef mr = merges[blockIdx.x];
  const int head = blockIdx.y * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int HQ = a.shape.num_q_heads;
  if (head >= HQ) return;
  // the reference maximum: the lanes share the partial results out among themselves
  float M = -INFINITY;
  for (int j = lane; j < mr.n; j += 32)
    M = fmaxf(M, a.part_ml[(size_t)(mr.slot_begin + j) * HQ + head].x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  // weighted sum in slot order, eight partial results in flight at a time
  float L = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j0 = 0; j0 < mr.n; j0 += 8) {
    float2 ml[8];
    float4 o[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      ml[k] = make_float2(-INFINITY, 0.f);
      o[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (j0 + k < mr.n) {
        const size_t prow = (size_t)(mr.slot_begin + j0 + k) * HQ + head;
        ml[k] = a.part_ml[prow];
        o[k] = ((const float4*)(a.part_o + prow * kDim))[lane];
      }
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float w = ml[k].x == -INFINITY ? 0.f : exp2f(ml[k].x - M);
      L += ml[k].y * w;
      acc.x += o[k].x * w; acc.y += o[k].y * w; acc.z += o[k].z * w; acc.w += o[k].w * w;
    }
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;           // every part empty: zeros
  __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
  __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
  uint2 packed;
  packed.x = *(uint32_t*)&lo;
  packed.y = *(uint32_t*)&hi;
  ((uint2*)((__nv_bfloat16*)a.out + ((size_t)mr.query * HQ + head) * kDim))[lane] = packed;
}

cudaError_t launch_merge(const AttnArgs& a, const MergeRef* d_merge, int n_merge, cudaStream_t st) {
  if (n_merge <= 0) return cudaSuccess;
  merge_kernel<<<dim3(n_merge, (a.shape.num_q_heads + 3) / 4), 128, 0, st>>>(a, d_merge);
  return cudaGetLastError();
}

}  // namespace apar

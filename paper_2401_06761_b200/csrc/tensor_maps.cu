// TMA descriptors.  The KV pools: each layer of a pool is seen as a 2-D bf16 array
// [num_blocks * num_kv_heads * 16 rows][128 dims]; a box is the 64-dim half of one 16-token
// tile (16 rows x 128 bytes), written to shared memory with the 128-byte swizzle.
#include <cuda.h>
#include <cuda_runtime.h>

#include "apar_internal.h"

namespace apar {

namespace {
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                             const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                             const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn encode_fn() {
  static EncodeFn cached = nullptr;
  if (cached) return cached;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) !=
          cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess)
    return nullptr;
  cached = (EncodeFn)fn;
  return cached;
}
}  // namespace

int make_query_tensor_map(const void* q, int64_t n_rows, int num_q_heads, int group,
                          CUtensorMap* tm_q) {
  EncodeFn fn = encode_fn();
  if (!fn) return -1;
  if (((uintptr_t)q & 15) != 0 || group < 1 || group > 128 || n_rows < 1) return -2;
  const cuuint64_t dims[3] = {(cuuint64_t)kDim, (cuuint64_t)num_q_heads, (cuuint64_t)n_rows};
  const cuuint64_t strides[2] = {(cuuint64_t)kDim * 2, (cuuint64_t)num_q_heads * kDim * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)group, (cuuint32_t)(128 / group)};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : (int)r;
}

int make_pool_tensor_maps(void* k_pool, void* v_pool, int64_t num_blocks, int num_kv_heads,
                          CUtensorMap* tm_k, CUtensorMap* tm_v) {
  EncodeFn fn = encode_fn();
  if (!fn) return -1;
  const cuuint64_t dims[2] = {(cuuint64_t)kDim, (cuuint64_t)num_blocks * num_kv_heads * kBlock};
  const cuuint64_t strides[1] = {(cuuint64_t)kDim * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)kBlock};
  const cuuint32_t estr[2] = {1, 1};
  void* pools[2] = {k_pool, v_pool};
  CUtensorMap* maps[2] = {tm_k, tm_v};
  for (int i = 0; i < 2; ++i) {
    CUresult r = fn(maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pools[i], dims,
                                strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return (int)r;
  }
  return 0;
}

}  // namespace apar

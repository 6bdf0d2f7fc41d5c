// apar_tree_decode_attention_static: decode attention over caller-supplied device block
// tables that performs no allocation of any kind.
//
// Who needs it: code that runs where device or pinned-host allocation is off limits - inside
// a serving loop whose memory is fully pre-carved by another allocator, in a plugin that is
// forbidden to touch the CUDA allocator of its host process, or from a thread that must never
// block on the implicit device synchronisation cudaMalloc/cudaFree can cause.  The other
// entry points take a caller-owned workspace but still create pinned staging buffers; this
// one keeps everything it needs (work items, per-split partial results) in one array that is
// part of the library image.
#include <algorithm>
#include <mutex>

#include "../../include/apar.h"
#include "apar_internal.h"

namespace apar {
namespace {

constexpr size_t kStaticScratchBytes = 16u << 20;   // resident on every GPU that loads the library
constexpr int kMaxDevices = 64;
constexpr int kMaxSplits = 8;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; the
// address a kernel can use is obtained once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

struct StaticLayout {
  size_t items, users, merges, part_ml, part_o, total;
};

StaticLayout static_layout(int n, int splits, int num_q_heads) {
  StaticLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return o; };
  const size_t rows = (size_t)n * splits * num_q_heads;
  L.items = take((size_t)n * splits * sizeof(WorkItem));
  L.users = take((size_t)n * sizeof(UserRef));
  L.merges = take((size_t)n * sizeof(MergeRef));
  L.part_ml = take(rows * sizeof(float2));
  L.part_o = take(rows * kDim * sizeof(float));
  L.total = off;
  return L;
}

// One thread per (row, split): every table row is a private chain cut into `splits` equal
// token ranges; the last range absorbs whatever lies beyond max_ctx_len.  Lengths come from
// device memory that the host never sees, so they are clamped here to what a table row can
// hold: the attention kernels then never index past a row's max_blocks entries, and a row of
// length <= 0 gets empty ranges (its output is written as zeros).
__global__ void __launch_bounds__(128) static_plan_kernel(WorkItem* items, UserRef* users,
                                                          MergeRef* merges,
                                                          const int32_t* __restrict__ lens, int n,
                                                          int splits, int chunk, int max_blocks) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n * splits) return;
  const int i = idx / splits, s = idx % splits;
  const int len = max(0, min(lens[i], max_blocks * kBlock));
  WorkItem it;
  it.table_row = i;
  it.tok_begin = s * chunk;
  it.tok_end = (s == splits - 1) ? len : min(len, (s + 1) * chunk);
  if (it.tok_end <= it.tok_begin) it.tok_begin = it.tok_end = 0;   // nothing left for this split
  it.user_begin = i;
  it.n_users = 1;
  it.slot_add = s;
  it.fin_n = it.fin_begin = 0;
  items[idx] = it;
  if (s == 0) {
    users[i] = UserRef{i, splits > 1 ? i * splits : -1};
    merges[i] = MergeRef{i, i * splits, splits, 0};
  }
}

}  // namespace
}  // namespace apar

using namespace apar;

extern "C" apar_status apar_tree_decode_attention_static(
    const void* k_pool, const void* v_pool, int32_t num_q_heads, int32_t num_kv_heads,
    int32_t n_threads, int32_t max_blocks_per_thread, const int32_t* block_tables,
    const int32_t* ctx_lens, int32_t max_ctx_len, const void* q, void* out, float sm_scale,
    void* cuda_stream) {
  if (n_threads < 0 || max_blocks_per_thread <= 0 || max_ctx_len <= 0) return APAR_ERR_INVALID_ARG;
  if (num_kv_heads <= 0 || num_q_heads <= 0 || num_q_heads % num_kv_heads) return APAR_ERR_UNSUPPORTED;
  if (n_threads == 0) return APAR_OK;
  if (!k_pool || !v_pool || !block_tables || !ctx_lens || !q || !out) return APAR_ERR_INVALID_ARG;
  const int splits = std::max(1, std::min(kMaxSplits, (max_ctx_len + 1023) / 1024));
  const StaticLayout lay = static_layout(n_threads, splits, num_q_heads);
  if (lay.total > kStaticScratchBytes) return APAR_ERR_WORKSPACE_TOO_SMALL;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return APAR_ERR_CUDA;
  void* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {     // first call on this device, with this device current
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return APAR_ERR_CUDA;
      g_scratch_ptr[dev] = p;
    }
    base = g_scratch_ptr[dev];
  }
  char* s = (char*)base;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int chunk = ((max_ctx_len + splits - 1) / splits + kBlock - 1) / kBlock * kBlock;
  const int n_items = n_threads * splits;
  static_plan_kernel<<<(n_items + 127) / 128, 128, 0, st>>>(
      (WorkItem*)(s + lay.items), (UserRef*)(s + lay.users), (MergeRef*)(s + lay.merges),
      ctx_lens, n_threads, splits, chunk, max_blocks_per_thread);
  if (cudaGetLastError() != cudaSuccess) return APAR_ERR_CUDA;

  AttnArgs a;
  a.q = q;
  a.out = out;
  a.k_pool = k_pool;
  a.v_pool = v_pool;
  a.d_tables = block_tables;
  a.d_lens = ctx_lens;          // not consulted: every item carries an explicit end
  a.d_items = (const WorkItem*)(s + lay.items);
  a.d_users = (const UserRef*)(s + lay.users);
  a.part_o = (float*)(s + lay.part_o);
  a.part_ml = (float2*)(s + lay.part_ml);
  a.shape = Shape{num_q_heads, num_kv_heads, num_q_heads / num_kv_heads, max_blocks_per_thread};
  a.scale_log2e = sm_scale * 1.4426950408889634f;
  if (launch_attention_vec(a, 0, n_items, a.shape.group == 1, st) != cudaSuccess) return APAR_ERR_CUDA;
  if (splits > 1 &&
      launch_merge(a, (const MergeRef*)(s + lay.merges), n_threads, st) != cudaSuccess)
    return APAR_ERR_CUDA;
  return APAR_OK;
}

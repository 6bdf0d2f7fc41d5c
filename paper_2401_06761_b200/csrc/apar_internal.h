// Internal declarations shared by the host side (bookkeeping, planner) and the kernel
// launchers.  Not part of the public boundary (include/apar.h).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

namespace apar {

constexpr int kBlock = 16;      // tokens per KV block
constexpr int kDim = 128;       // head dimension
constexpr int kTileBytes = kBlock * kDim * 2;   // one (block, kv head) tile of K or of V
constexpr int kMaxRowsPerItem = 64;             // query rows one work item may carry

// One unit of attention work: a run of consecutive blocks of one table row, read once for
// every (query, head-in-group) row that shares it.  The kv head is the second grid dimension.
struct WorkItem {
  int32_t table_row;   // row of the device block table to walk
  int32_t tok_begin;   // first token of the run in chain coordinates (multiple of 16)
  int32_t tok_end;     // one past the last token; < 0: "the current length of table_row"
  int32_t user_begin;  // first entry of this item's users in the UserRef array
  int32_t n_users;     // queries sharing the run (rows = n_users * group)
  int32_t slot_add;    // added to every user's partial slot (chunk ordinal inside the run)
  // fin_n > 0: this is the last item of its (single) query's chain; instead of writing a
  // partial it folds partial slots [fin_begin, fin_begin + fin_n), which earlier launches of
  // the same call completed, into its own state and writes the final output.
  // Bits 8.. of fin_n: bit (8 + j) is set when folded part j is produced by a single-tile
  // item, which a multi-row finishing item may share a kernel launch with; the kernel then
  // waits for that part's ready flag instead of relying on launch order.
  int32_t fin_n, fin_begin;
};
__host__ __device__ inline int fin_count(const WorkItem& w) { return w.fin_n & 0xff; }
__host__ __device__ inline uint32_t fin_same_class(const WorkItem& w) {
  return (uint32_t)w.fin_n >> 8;
}

// A query that reads a work item.  slot < 0: the item covers the query's whole chain and
// writes the final output; otherwise partial row (slot + item.slot_add) receives (m, l, o).
struct UserRef {
  int32_t query;
  int32_t slot;
};

// A query whose chain was covered by n >= 2 items: merge partial slots [slot_begin, +n).
struct MergeRef {
  int32_t query;
  int32_t slot_begin;
  int32_t n;
  int32_t pad;
};

// A contiguous update of the device block table: table[row][pos .. pos+count) = data[...].
struct TableDelta {
  int32_t row, pos, count, data_off;
};

// Copy of the valid rows of a partial block at fork.
struct CowCopy {
  int32_t src_block, dst_block, rows, pad;
};

// One candidate token of a verification step (a query of its own): it sits at chain position
// base + index of thread `row`, which holds n_cand candidates from `base` on, and attends,
// among them, exactly those whose bit is set in `mask` (its own bit included).  The committed
// prefix [0, base) is covered by ordinary work items; `slot` is where this partial result goes
// (-1: there is no prefix, write the output).
struct VerifyDesc {
  int32_t row, base, n_cand, slot;
  uint64_t mask;
  int32_t query, pad;
};

// Rows to move when candidates are accepted: row src of the thread's chain becomes row dst.
struct RowMove {
  int32_t src_slot, dst_slot;     // pool slots (block * 16 + offset)
};

struct Shape {
  int32_t num_q_heads, num_kv_heads, group;
  int32_t table_stride;        // ints per device table row
};

// ---- programmatic dependent launch ------------------------------------------------------
// A warp-stream attention launch that follows another attention kernel of the same call is
// allowed to take the SM slots its predecessor's last wave leaves free.  Rules that keep this
// correct:
//   * the tensor-core and warp-stream kernels call pdl_launch_dependents() early, so that a
//     successor may start as soon as all of their own CTAs have started;
//   * a CTA calls pdl_wait() before it reads what an earlier kernel of the call wrote
//     (partial results) - it returns once the predecessor grid has completed and flushed;
//   * a CTA that reads nothing of the kind still calls pdl_wait() before it exits, so that
//     "this grid has completed" implies "every earlier grid of the call has completed".
// Both are no-ops in a kernel that was launched the ordinary way; all other kernels are
// launched the ordinary way and start after everything before them on the stream.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---- kernel launchers (kernels.cu); all enqueue on `st` and return cudaGetLastError() ----
cudaError_t launch_cow_copy(void* k_pool, void* v_pool, const CowCopy* d_copies, int n,
                            int num_kv_heads, cudaStream_t st);
// dst[0..bytes) = src_mapped[0..bytes) read by the SMs; src_mapped is the device alias of a
// pinned, mapped host buffer; bytes is a multiple of 4.
cudaError_t launch_stage_copy(void* dst, const void* src_mapped, size_t bytes, cudaStream_t st);
// Reads `bytes` (rounded down to 16) once and xors them into *sink (8 bytes, device).
cudaError_t launch_stream_read(const void* src, size_t bytes, void* sink, int num_sms,
                               cudaStream_t st);
// slots[r] = block * 16 + offset for new row r.
cudaError_t launch_append(void* k_pool, void* v_pool, const void* k_new, const void* v_new,
                          const int32_t* d_slots, int64_t first_row, int n_rows,
                          int num_kv_heads, cudaStream_t st);
// Applies table deltas and (row, length) pairs to the device copies in one launch.
cudaError_t launch_sync(int32_t* d_tables, int table_stride, int32_t* d_lens,
                        const TableDelta* d_deltas, const int32_t* d_data, int n_deltas,
                        const int32_t* d_len_pairs, int n_pairs, cudaStream_t st);

// One decode step on the device: lens[row] += 1 for the n rows in d_step_rows, slot of each new
// row into d_slot_map; d_pairs (int4: list position, row, table position, block id) are the
// blocks the host allocated for threads that start a new block this step.
cudaError_t launch_step_advance(int32_t* d_tables, int table_stride, int32_t* d_lens,
                                const int32_t* d_step_rows, int n, const void* d_pairs,
                                int n_pairs, int32_t* d_slot_map, cudaStream_t st);

struct AttnArgs {
  const void* q; void* out;
  const void* k_pool; const void* v_pool;
  const int32_t* d_tables; const int32_t* d_lens;
  const WorkItem* d_items; const UserRef* d_users;
  float* part_o; float2* part_ml;     // [slots][num_q_heads][128], [slots][num_q_heads]
  // [slots][num_q_heads] ready flags, or nullptr: written (after the partial row, with the
  // launch's own mark) by the plain units of a warp-stream launch that also holds finishing units
  int* part_flag = nullptr;
  Shape shape;
  float scale_log2e;                  // sm_scale * log2(e)
  const CUtensorMap* tm_k = nullptr;  // [host] TMA descriptors of the pools (tensor-core path)
  const CUtensorMap* tm_v = nullptr;
  int* d_error = nullptr;             // [device] set to 1 when a bounded wait gave up
  // 1: this launch is allowed to start before the launch before it on the stream has finished
  // (programmatic dependent launch); its kernel then orders itself with pdl_wait()
  int pdl = 0;
  int num_sms = 148;                  // of the device the context lives on
  int umma_heads = 0;                 // > 0: kv heads per CTA of the tcgen05 kernel (testing)
  int umma_mode = 0;                  // tcgen05 kernel: 0 default, 1 one CTA per (item, heads),
                                      // 2 persistent CTAs that claim units from *d_ticket
  int ws_mode = 0;                    // warp-stream kernel: 0 default, 1 one CTA per item, 2 persistent
  int* d_ticket = nullptr;            // [device] counters of the persistent forms, zero when no
                                      // launch is in flight: words 0-2 tcgen05 kernel, 4-6 and
                                      // 8-10 warp-stream launches (unit counter, leavers, launches)
};
// single_row: every item carries exactly one query row.
cudaError_t launch_attention_vec(const AttnArgs& a, int item_begin, int n_items, bool single_row,
                                 cudaStream_t st);
// Blackwell tcgen05/TMEM path for items with up to 64 rows (any number of query tiles).
cudaError_t launch_attention_umma(const AttnArgs& a, int item_begin, int n_items, cudaStream_t st);
// Tree-masked attention of consecutive query tokens with 128-row tiles (tcgen05): item i is
// n_tok (at most 2 * (128 / group)) tokens of the thread in table row table_row, the first at
// chain position pos0; its queries are rows q_first .. q_first + n_tok - 1 of the query
// array, which the kernel reads through tm_q (make_query_tensor_map).  Uses a.out, a.d_tables,
// a.shape, a.scale_log2e, a.tm_k, a.tm_v, a.d_error, a.num_sms and words 0-1 of a.d_ticket.
struct PrefillItem { int32_t table_row, q_first, pos0, n_tok; };
cudaError_t launch_attention_prefill(const AttnArgs& a, const CUtensorMap* tm_q,
                                     const PrefillItem* d_items, int n_items, cudaStream_t st);
// TMA descriptor of a query array [n_rows][num_q_heads][128] bf16 (16-byte aligned): a box is
// the 64-dim half of the rows of `group` consecutive heads of 128 / group consecutive tokens.
// Returns 0 on success.
int make_query_tensor_map(const void* q, int64_t n_rows, int num_q_heads, int group,
                          CUtensorMap* tm_q);
// Warp-stream path for items with at most 16 rows per kv head; one CTA per item, all kv heads.
// ticket_index: which group of four words of a.d_ticket the persistent form uses (1 or 2; group
// 0 belongs to the tcgen05 kernel).
cudaError_t launch_attention_ws(const AttnArgs& a, int item_begin, int n_items, cudaStream_t st,
                                int ticket_index);
// Returns 0 on success.
int make_pool_tensor_maps(void* k_pool, void* v_pool, int64_t num_blocks, int num_kv_heads,
                          CUtensorMap* tm_k, CUtensorMap* tm_v);
// Candidate part of a verification step: one partial result (or the output) per VerifyDesc.
cudaError_t launch_verify_tail(const AttnArgs& a, const VerifyDesc* d_desc, int n_desc,
                               cudaStream_t st);
// Moves token rows inside one layer of the pools (K and V, all kv heads); moves are grouped:
// group g is moves [begin[g], begin[g+1]) and is carried out as "read all, then write all".
cudaError_t launch_row_moves(void* k_pool, void* v_pool, const RowMove* d_moves,
                             const int32_t* d_group_begin, int n_groups, int num_kv_heads,
                             cudaStream_t st);
cudaError_t launch_merge(const AttnArgs& a, const MergeRef* d_merge, int n_merge, cudaStream_t st);

// ---- planner (planner.cpp) ----
// A run of consecutive table positions whose blocks are held by the same set of threads
// ("group"): blocks become shared only through fork, so the host keeps, per thread, its table
// as a short list of such runs (see apar_api.cu) and the planner can count per group instead
// of per block.
struct BlockRun {
  int32_t gid;            // group id (dense, recycled)
  int32_t pos;            // first table position
  int32_t n;              // blocks
};

struct PlanQuery {
  const int32_t* table;   // host block ids of the query's thread
  int32_t table_row;      // row in the device table
  int32_t len;            // tokens
  // optional: the same table as runs of groups; when every query of a call has them (and no
  // query is listed twice or cut short), the planner walks these instead of the block ids
  const BlockRun* runs = nullptr;
  int32_t n_runs = 0;
  // 1: one more partial result of this query is produced outside the plan's items (the
  // candidate tokens of a verification step); a slot is reserved for it (Plan::extra_slot)
  // and the query is merged.  len may then be 0 (nothing but that result).
  int32_t extra_parts = 0;
};

struct Plan {
  // vec items (finishing ones last), then mma items by tile count 4, 3, 2, 1 (in the 1-tile
  // class the finishing ones last); each group longest first
  std::vector<WorkItem> items;
  int32_t n_vec = 0, n_mma = 0;
  int32_t n_vec_final = 0, n_mma1_final = 0;   // finishing items at the end of their class
  int32_t n_mma_tiles[4] = {0, 0, 0, 0};   // mma items needing 1, 2, 3, 4 query tiles
  std::vector<UserRef> users;
  std::vector<MergeRef> merges;
  std::vector<int32_t> extra_slot;   // per query with extra_parts: its slot, -1 = writes the output
  int64_t total_slots = 0;         // partial rows (before the head dimension)
  int64_t unique_tokens = 0, attended_tokens = 0;
  int32_t chunk_tokens = 0;
};

class Planner {
 public:
  void init(int num_blocks, int group, int num_kv_heads);
  // open_tails: the last chunk of a private tail run gets tok_end < 0 (resolved on the device
  // from the length array), so the plan stays valid while threads only grow.
  // Items with at least mma_min_rows query rows go to the tensor-core kernel.
  // Returns false if the partial rows cannot fit `slot_capacity` even without splitting.
  // fuse_final: the last item of a query whose chain ends in a private run of at most 16 rows
  // finishes the query itself (see WorkItem::fin_n); such queries need no merge entry.
  // by_runs: walk the queries' group runs (keys are group ids) instead of their block ids.
  bool build(const PlanQuery* q, int n, int64_t slot_capacity, bool open_tails,
             int mma_min_rows, bool fuse_final, Plan* out, bool by_runs = false);
  void set_num_sms(int n) { num_sms_ = n > 0 ? n : 148; }

 private:
  template <bool kRuns>
  void find_segments(const PlanQuery* q, int n, bool open_tails, int64_t* unique,
                     int64_t* attended);
  void ensure_keys(size_t n);
  int num_blocks_ = 0, group_ = 1, hint_kv_heads_ = 1, num_sms_ = 148;
  uint32_t epoch_ = 0;
  std::vector<uint32_t> stamp_;
  std::vector<int32_t> cnt_, seg_of_;
  std::vector<uint8_t> partial_;
  struct Seg { int32_t table_row, tok_begin, tok_end, n_blocks, n_users, user_off, priv, open; };
  struct SegUser { int32_t seg, query, ord; };
  std::vector<Seg> segs_;
  std::vector<SegUser> seg_users_;
  std::vector<int32_t> n_parts_, qbeg_, part_off_;
  std::vector<WorkItem> vec_items_, mma_items_[4], vec_final_, mma1_final_;
  std::vector<uint8_t> fused_;
};

}  // namespace apar

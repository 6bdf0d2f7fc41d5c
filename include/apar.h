/*
 * apar.h - C ABI of the APAR decode hot path on one NVIDIA B200 (sm_100a).
 *
 * APAR (Auto-Parallel Auto-Regressive decoding) lets a model fork generation threads.
 * A forked thread shares its parent's prefix; with a paged KV cache the fork shares all
 * full blocks of the parent and duplicates no more than one block (paper, Section 2.3 "Decoding").
 * A new token attends only to the tokens on its path to the root of the paragraph tree,
 * itself included (Section 2.2 "Training attention"; Section 2.4 feature 3).  When a
 * thread finishes, whatever cache no other thread still uses is freed (Section 2.3; feature 2).
 *
 * This library owns the host-side bookkeeping (block tables, reference counts, free list)
 * and launches the CUDA kernels for: the copy of the partial last block at fork, the
 * scatter of new K/V rows into the pool, and the batched decode attention in which every
 * shared block is read once for all threads and query heads that see it.
 *
 * Conventions
 *   - Every pointer is tagged [host] or [device].  The caller owns all device memory (pool,
 *     q, out, k_new, v_new, workspace) and the stream; the library owns host tables and
 *     its pinned staging buffers.
 *   - Calls return after enqueueing their kernels on `cuda_stream` (a cudaStream_t passed
 *     as void*; NULL = the default stream).  Host bookkeeping is complete on return.  All
 *     calls on one context must use streams that are ordered with respect to each other
 *     (normally one stream); a context is not thread-safe.
 *   - The library's own uploads (slot lists, table deltas, plans: KBs per step) are read from
 *     its pinned, mapped staging buffers by kernels on `cuda_stream`, not by a copy engine,
 *     so they never wait behind the caller's host-to-device copies on other streams.
 *   - Batched calls process their entries in index order and are all-or-nothing: on any
 *     error other than APAR_ERR_CUDA no host state changes and nothing is launched.
 *     APAR_ERR_CUDA means a CUDA runtime call (an event wait, a launch) failed part-way
 *     through a call: the host tables may then already describe rows or forks whose kernels
 *     were never enqueued.  Such errors are sticky in the CUDA runtime; the context must not
 *     be used further except for apar_last_cuda_error and apar_destroy.
 *   - No exceptions, aborts or device traps cross this boundary; errors are status codes.
 *     There is no CPU fallback: without a usable CUDA device calls fail with APAR_ERR_CUDA.
 *
 * Layout of the KV pool (fixed): K pool and V pool are each
 *       bf16 [num_layers][num_blocks][num_kv_heads][block_size = 16][head_dim = 128],
 *   so the rows of one (layer, block, kv head) form a contiguous 4 KiB tile.  All layers share
 *   one set of block tables: block b of layer l is the same logical block in every layer.  Q, out:
 *   bf16 [n][num_q_heads][128].  k_new, v_new: bf16 [rows][num_kv_heads][128].
 *   Query head h reads KV head h / (num_q_heads / num_kv_heads).
 *
 * Deterministic policy (the paper is silent; stated so that block ids are reproducible)
 *   - Thread ids are handed out 0, 1, 2, ... and never reused.
 *   - The free list is a stack.  A fresh pool hands out blocks 0, 1, 2, ...; released
 *     blocks are pushed in table order and reused last-in first-out.
 *   - Fork is eager: the CHILD receives a newly allocated block holding a copy of the
 *     r = len mod 16 valid rows of the parent's partial last block; the parent keeps its
 *     block and continues to append in place.  r = 0 copies nothing.  Rows r..15 of the
 *     new block are unspecified and never read.
 */
#ifndef APAR_H_
#define APAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct apar_ctx apar_ctx;   /* opaque; host state owned by the library */
typedef int32_t apar_status;

enum {
  APAR_OK = 0,
  APAR_ERR_INVALID_ARG = -1,          /* null pointer, negative count, duplicate id, bad shape   */
  APAR_ERR_BAD_THREAD = -2,           /* unknown, released or (in release) repeated thread id     */
  APAR_ERR_NO_BLOCKS = -3,            /* the pool cannot supply the blocks the whole call needs   */
  APAR_ERR_NO_THREADS = -4,           /* more than max_threads live threads                       */
  APAR_ERR_TABLE_FULL = -5,           /* a thread would exceed max_blocks_per_thread              */
  APAR_ERR_EMPTY_CONTEXT = -6,        /* attention requested for a thread with no tokens          */
  APAR_ERR_WORKSPACE_TOO_SMALL = -7,  /* workspace_bytes < apar_workspace_bytes(), or a plan that
                                         does not fit the partial-result area                     */
  APAR_ERR_CUDA = -8,                 /* a CUDA runtime call failed; see apar_last_cuda_error     */
  APAR_ERR_UNSUPPORTED = -9           /* block_size != 16, head_dim != 128, heads not divisible,
                                         more than 64 query heads per kv head                     */
};

typedef struct {
  int32_t num_blocks;             /* blocks in each of k_pool and v_pool                         */
  int32_t block_size;             /* must be 16                                                  */
  int32_t num_q_heads;
  int32_t num_kv_heads;           /* must divide num_q_heads; num_q_heads / num_kv_heads <= 64   */
  int32_t head_dim;               /* must be 128                                                 */
  int32_t max_threads;            /* live generation threads at any time                         */
  int32_t max_blocks_per_thread;  /* longest chain, in blocks                                    */
  int32_t num_layers;             /* attention layers that share the block tables; 0 means 1     */
  void*   k_pool;                 /* [device] caller-owned, 256-byte aligned                     */
  void*   v_pool;                 /* [device] caller-owned, 256-byte aligned                     */
  void*   workspace;              /* [device] caller-owned scratch, 256-byte aligned             */
  size_t  workspace_bytes;        /* >= apar_workspace_bytes(cfg)                                */
} apar_config;

typedef struct {
  int64_t live_threads;
  int64_t free_blocks;
  int64_t used_blocks;
  int64_t forks;                  /* threads created by apar_fork so far                         */
  int64_t cow_blocks;             /* blocks copied by forks so far (<= forks)                    */
  int64_t cow_rows;               /* token rows copied by forks so far                           */
  /* the most recent attention call: */
  int64_t attn_threads;           /* queries                                                     */
  int64_t attn_attended_tokens;   /* sum of chain lengths ("attended tokens", Section 3.4)       */
  int64_t attn_unique_tokens;     /* distinct KV token rows read (each shared row counted once)  */
  int64_t attn_work_items;        /* (segment chunk) items, before the kv-head dimension         */
  int64_t attn_partials;          /* partial (m, l, o) rows per query head written and merged    */
  int64_t attn_kernels;           /* kernels launched by the call                                */
  int64_t attn_plan_reused;       /* 1 if the cached plan of the previous call was reused        */
  int64_t attn_vec_items;         /* items on the CUDA-core vector path                          */
  int64_t attn_mma_items;         /* items on the tensor-core path                               */
  int64_t kernels_total;          /* kernels launched by this context since creation             */
  int64_t peak_used_blocks;       /* most blocks ever in use at once (x16 = "max cached tokens",
                                     Section 3.4, in block granularity)                           */
  int64_t device_wait_timeouts;   /* non-zero once a kernel gave up a bounded wait (results of
                                     that call are invalid); reading it synchronises the device   */
  int64_t attn_plan_host_us;      /* host time the most recent attention call spent planning
                                     (0 when it reused the cached plan), microseconds            */
  int64_t attn_upload_bytes;      /* bytes that call staged for the device (plan, table deltas)  */
} apar_stats;

/* Bytes of device scratch a context with this configuration needs (pool pointers and the
 * workspace fields are ignored).  Returns 0 for an unsupported configuration. */
size_t apar_workspace_bytes(const apar_config* cfg /*[host]*/);

/* Creates a context over an empty pool.  Allocates host memory and pinned staging only.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_create(const apar_config* cfg /*[host]*/, apar_ctx** out /*[host]*/);
/* The same bookkeeping without a device (the paper has no counterpart): k_pool, v_pool and
 * workspace are ignored, no CUDA call is made, nothing is ever launched.  apar_new_threads,
 * apar_fork, apar_append_kv (row pointers may be NULL), apar_release, the paragraph calls and
 * all introspection work as documented and hand out the same ids as a device context would;
 * every attention call and apar_decode_step return APAR_ERR_UNSUPPORTED.  For schedulers that
 * want to try an admission decision (will this fork or append fit?) on a copy of the state,
 * and for checking the bookkeeping on a machine without a GPU. */
apar_status apar_create_host_only(const apar_config* cfg /*[host]*/, apar_ctx** out /*[host]*/);
apar_status apar_destroy(apar_ctx* ctx);

/* n new prompt sequences (roots of paragraph trees; the initial sequence group of Algorithm 1): empty block
 * tables, length 0.  tid_out [host] receives n ids.  Errors: NO_THREADS. */
apar_status apar_new_threads(apar_ctx* ctx, int32_t n, int32_t* tid_out /*[host]*/);

/* Fork (Algorithm 1, the step that duplicates a sequence; Section 2.3: the child maps the
 * parent's blocks and at most a single block is physically duplicated).  For each parent, in order: the child's table is the parent's first
 * floor(len/16) block ids (their reference counts go up by one); if r = len mod 16 != 0 a
 * block is taken from the free list and the r valid rows of the parent's last block (K and V,
 * all KV heads) are copied into it by a kernel enqueued on the stream.  Child length = len.
 * The same parent may appear several times.  child_tid_out [host] receives n ids.
 * Errors: BAD_THREAD, NO_THREADS, NO_BLOCKS (needs one block per parent with r != 0),
 * WORKSPACE_TOO_SMALL (more copies in one call than the staging area holds), CUDA. */
apar_status apar_fork(apar_ctx* ctx, int32_t n, const int32_t* parent_tid /*[host]*/,
                      int32_t* child_tid_out /*[host]*/, void* cuda_stream);

/* KV append (the token append of Algorithm 1, i.e. the K, V rows the model writes for it).
 * Thread tid[i] receives n_tok[i] rows (n_tok NULL = one row each), taken consecutively from
 * k_new / v_new [device] bf16 [sum n_tok][num_kv_heads][128].  A row at position p goes to
 * slot p mod 16 of the thread's block p / 16; a block is allocated whenever p mod 16 == 0.
 * Blocks are allocated in (entry, position) order.  Thread ids must be distinct.
 * Errors: BAD_THREAD, INVALID_ARG, TABLE_FULL, NO_BLOCKS. */
apar_status apar_append_kv(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/,
                           const int32_t* n_tok /*[host] or NULL*/,
                           const void* k_new /*[device]*/, const void* v_new /*[device]*/,
                           void* cuda_stream);

/* Tree decode attention (Section 2.2 "Training attention", Section 2.4 feature 3): for
 * query i, owned by thread tid[i], and every query head h,
 *     out[i][h] = softmax_j(sm_scale * <q[i][h], K_j>) . V_j
 * over the len(tid[i]) tokens of that thread's chain (everything it inherited at its forks
 * plus its own rows, the newest row included), KV head h / group.  bf16 in, fp32
 * accumulation, bf16 out (round to nearest even).  Each physical block is read once per
 * call for all queries and heads that share it.  A thread may be listed more than once;
 * n <= max_threads.
 * q [device] bf16 [n][num_q_heads][128]; out [device] same shape.
 * Errors: INVALID_ARG, BAD_THREAD, EMPTY_CONTEXT, WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_tree_decode_attention(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/,
                                       const void* q /*[device]*/, void* out /*[device]*/,
                                       float sm_scale, void* cuda_stream);

/* Tree-masked attention for queries at arbitrary positions (the training / prefill mask of
 * Section 2.2: a token attends the tokens of its ancestors and, causally, those of its own
 * node).  Query i sits on the chain of thread tid[i] and sees its first attend_len[i] tokens,
 * 1 <= attend_len[i] <= len(tid[i]); a thread may be listed many times (all positions of a
 * prompt, several candidate positions of one thread).  Blocks that several queries see in full
 * are still read once for all of them.  Same shapes, arithmetic and errors as
 * apar_tree_decode_attention, plus INVALID_ARG for a length out of range; n <= max_threads. */
apar_status apar_tree_prefix_attention(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/,
                                       const int32_t* attend_len /*[host]*/,
                                       const void* q /*[device]*/, void* out /*[device]*/,
                                       float sm_scale, void* cuda_stream);

/* Verification of speculated tokens with tree attention (Section 3.2 "Implementation": the
 * Medusa setting predicts the next few tokens with extra heads and verifies them in one pass
 * with a tree mask among the candidates).  Thread tid[i] holds n_cand[i] candidate tokens as the
 * LAST n_cand[i] rows of its chain (put there with apar_append_kv, n_tok = n_cand[i]).
 * Candidate j of that thread is one query; it attends every committed token of the chain
 * (positions below len - n_cand[i], through the shared blocks exactly as in decode attention,
 * so candidates of sibling threads still read a shared prompt once) and, among the candidates,
 * exactly those whose bit is set in its mask: bit x of anc_mask means "sees candidate x of the
 * same thread".  Bit j (itself) must be set; bits >= n_cand[i] must be clear.  A chain of
 * candidates is a lower-triangular mask, a tree of them sets for each node the bits of its
 * ancestors.  q, out [device] bf16 [sum n_cand][num_q_heads][128], candidates of tid[0] first.
 *   n_cand [host] [n], 1..64 each and <= len(tid[i]); anc_mask [host] uint64 [sum n_cand];
 *   tids distinct; sum n_cand <= max_threads.
 * Layer 0; apar_tree_decode_attention_layer replays the same verification on other layers.
 * Errors: INVALID_ARG (also a bad mask), BAD_THREAD, WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_tree_verify_attention(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/,
                                       const int32_t* n_cand /*[host]*/,
                                       const uint64_t* anc_mask /*[host]*/,
                                       const void* q /*[device]*/, void* out /*[device]*/,
                                       float sm_scale, void* cuda_stream);
/* Outcome of a verification: of the n_cand[i] candidate rows at the end of thread tid[i], the
 * n_keep[i] rows keep_idx (indices into the candidates, strictly increasing; all threads'
 * lists one after the other) stay, moved up so that they follow the committed rows in order
 * (K and V, all kv heads, every layer; by a kernel on the stream), and the thread ends after
 * them.  Blocks that hold no remaining row go back to the free list in table order.  The
 * paper's own Medusa path keeps one contiguous cache for a whole batch and therefore masks
 * mispredicted slots in later attention (Appendix C.1); with a block table per thread every
 * thread simply keeps its own accepted length, so nothing is ever masked afterwards.
 * The blocks from the first candidate on must be held by this thread alone (INVALID_ARG if a
 * fork has shared them since).  tids distinct.
 * Errors: INVALID_ARG, BAD_THREAD, WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_accept_candidates(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/,
                                   const int32_t* n_cand /*[host]*/,
                                   const int32_t* n_keep /*[host]*/,
                                   const int32_t* keep_idx /*[host] [sum n_keep]*/,
                                   void* cuda_stream);

/* Tree-masked attention for whole runs of consecutive tokens: prompt prefill into the paged
 * pool and the training mask of Section 2.2 (Fig. 2: a token attends the tokens of its
 * ancestors and, causally, those of its own node).  Segment i is the q_count[i] tokens of
 * thread tid[i] at chain positions q_begin[i] .. q_begin[i] + q_count[i] - 1 (their K, V rows
 * must already be in the pool: append first); the query at position p attends positions
 * 0 .. p of that thread's chain.  A prompt is one segment from position 0; every node of a
 * paragraph tree is one segment of its thread that starts where the node's own tokens start.
 * q, out [device] bf16 [sum q_count][num_q_heads][128], segments in order, q 16-byte aligned
 * (it is read by TMA).  The queries of a segment are processed 256 rows at a time
 * (2 * (128 / group) tokens x group heads) on the tensor cores; a tile reads its chain once
 * for all of its rows and masks every row at its own position.  Any number of queries per
 * call; `layer` selects the pool layer.  Invalidates the cached decode plan.
 * Errors: INVALID_ARG (also a range outside the thread, or a misaligned q), BAD_THREAD, CUDA. */
apar_status apar_tree_prefill_attention(apar_ctx* ctx, int32_t layer, int32_t n,
                                        const int32_t* tid /*[host]*/,
                                        const int32_t* q_begin /*[host]*/,
                                        const int32_t* q_count /*[host]*/,
                                        const void* q /*[device]*/, void* out /*[device]*/,
                                        float sm_scale, void* cuda_stream);

/* The same decode step for the other attention layers of a model (Algorithm 1's Sample runs
 * every layer over the same sequences; the paper states nothing per layer).  Both calls reuse
 * what the most recent apar_append_kv / apar_tree_decode_attention of this context prepared on
 * the device - the slot of every new row, the work plan - and do no bookkeeping, no planning
 * and no host-to-device copy: they only launch kernels on layer `layer` (0 <= layer <
 * num_layers) of the pools.
 *   apar_append_kv_layer: k_new / v_new [device] hold the same rows, in the same order, as in
 *     that apar_append_kv call (which itself wrote layer 0).  At most 262144 rows are retained
 *     per call; a larger call cannot be replayed (APAR_ERR_WORKSPACE_TOO_SMALL).
 *   apar_tree_decode_attention_layer: same queries, in the same order, as in that attention
 *     call (which itself ran on layer 0).  Fails with APAR_ERR_INVALID_ARG if any bookkeeping
 *     call (new_threads, fork, append, release) came after it.
 * apar_fork copies the partial block in every layer.
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_append_kv_layer(apar_ctx* ctx, int32_t layer, const void* k_new /*[device]*/,
                                 const void* v_new /*[device]*/, void* cuda_stream);
apar_status apar_tree_decode_attention_layer(apar_ctx* ctx, int32_t layer,
                                             const void* q /*[device]*/, void* out /*[device]*/,
                                             float sm_scale, void* cuda_stream);

/* One decode step of Algorithm 1 for the threads tid[0..n) in a single call: every thread gains
 * one token (the Sample / append pair of the algorithm's loop; Section 2.3 "Decoding"), then
 * attends over its chain, the new token included.  Equivalent to apar_append_kv (one row each)
 * followed by apar_tree_decode_attention on the same list, with the same block ids, and built
 * so that a steady step costs the host almost nothing: while the list stays the same from one
 * step to the next (no release, no apar_append_kv in between), the device keeps the list, the
 * tables and the lengths; one small kernel bumps the lengths and derives the pool slot of every
 * new row from the device tables, and the host only handles the threads that start a new block
 * in this step (one in sixteen) plus a counter per thread.  The work plan is reused as in
 * apar_tree_decode_attention.  Layer 0 of the pools is written and read; other layers follow
 * with apar_append_kv_layer / apar_tree_decode_attention_layer.
 *   tid [host] distinct ids; k_new, v_new [device] bf16 [n][num_kv_heads][128], row i for tid[i];
 *   q, out [device] bf16 [n][num_q_heads][128].
 * CUDA graphs: a step whose list is unchanged and in which no thread starts a new block
 * (apar_steps_before_new_block() > 0) launches kernels only and uses no staging buffer, so it
 * can be captured (together with the layer calls that follow it) and replayed.  The capturing
 * call does the host bookkeeping of the first replay; before every further replay call
 * apar_note_step_replay.  While a stream is capturing, a step that would need staging is refused
 * with APAR_ERR_INVALID_ARG and changes nothing.
 * Errors: INVALID_ARG (also duplicate ids), BAD_THREAD, TABLE_FULL, NO_BLOCKS,
 * WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_decode_step(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/,
                             const void* k_new /*[device]*/, const void* v_new /*[device]*/,
                             const void* q /*[device]*/, void* out /*[device]*/, float sm_scale,
                             void* cuda_stream);
/* How many more steps the thread list of the most recent apar_decode_step can take before one
 * of its threads starts a new block (0: the next step allocates).  Errors: INVALID_ARG if there
 * is no such list or a release / apar_append_kv came after it. */
apar_status apar_steps_before_new_block(apar_ctx* ctx, int32_t* steps_out /*[host]*/);
/* Host side of one replay of a captured apar_decode_step: every thread of the list is one token
 * longer, exactly what the replayed kernels do on the device.  Launches nothing.
 * Errors: INVALID_ARG if the step list or the plan is no longer the captured one (any
 * bookkeeping call since), or if a thread of the list would start a new block - make an
 * ordinary apar_decode_step then, and capture again afterwards if block ids matter to the
 * graph (they do not: the captured kernels read tables and lengths from the device). */
apar_status apar_note_step_replay(apar_ctx* ctx);

/* ReleaseCache (Algorithm 1; Section 2.3: a finished sequence gives back the cache that no
 * other sequence holds):
 * one reference is dropped per table entry, in table order; blocks reaching zero go back to
 * the free list; the ids become invalid.  Errors: BAD_THREAD (also for a repeated id). */
apar_status apar_release(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/);

/* The same attention for a caller that keeps its own block tables (an external scheduler):
 * block_tables [host] int32 [n_threads][max_blocks_per_thread] (row stride from cfg),
 * ctx_lens [host] int32 [n_threads] tokens per query; n_threads <= cfg->max_threads.  Uses
 * cfg->workspace for the whole call; no state survives it, and it returns only after its own
 * host-to-device copies have completed (it synchronises the stream).  Blocks that appear in
 * several rows are read once, provided they are full for every row that lists them.
 * Errors: INVALID_ARG, UNSUPPORTED, EMPTY_CONTEXT, WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_tree_decode_attention_tables(const apar_config* cfg /*[host]*/, int32_t n_threads,
                                              const int32_t* block_tables /*[host]*/,
                                              const int32_t* ctx_lens /*[host]*/,
                                              const void* q /*[device]*/, void* out /*[device]*/,
                                              float sm_scale, void* cuda_stream);

/* Decode attention for callers that must not allocate.  (The paper has no counterpart: this
 * is a packaging variant of the attention above, not a step of the method.)
 *
 * Some callers cannot let a library call cudaMalloc, cudaMallocHost or cudaFree on their
 * behalf: a serving process whose GPU memory is entirely pre-carved by its own allocator, a
 * plugin barred from the CUDA allocator of its host, or a latency-critical thread that must
 * not hit the device-wide synchronisation those calls can imply.  Every other attention entry
 * point of this library creates pinned staging buffers; this one allocates nothing at all.
 * Its work-item list and its per-split partial results live in a 16 MiB array that is part
 * of the library image, so every GPU that loads the library carries that array until exit.
 *
 * Semantics: row i of block_tables [device] int32 [n_threads][max_blocks_per_thread] with
 * ctx_lens[i] [device] tokens, 1 <= ctx_lens[i] <= 16 * max_blocks_per_thread, is one private
 * chain; out[i][h] is the same softmax attention as above over that chain.  The host never
 * reads the lengths, so it cannot refuse bad ones: a length above 16 * max_blocks_per_thread
 * is treated as that bound (the kernels never walk past a table row), and a row of length
 * <= 0 attends nothing and receives zeros.  The first ceil(len / 16) ids of every row must be
 * valid block ids of the pools; they are not checked.  Rows are not de-duplicated: a block listed by several
 * rows is read once per row.  Chains are cut into ceil(max_ctx_len / 1024) (at most 8) token
 * ranges whose partial results are merged; max_ctx_len [host] is an upper bound of ctx_lens
 * (a longer row is still computed correctly, only less evenly split).  k_pool, v_pool, q, out
 * as in apar_config / apar_tree_decode_attention, all [device].
 *
 * Limits and sharing: the request is refused with APAR_ERR_WORKSPACE_TOO_SMALL when
 * n_threads * splits * (32 + num_q_heads * 520) + n_threads * 24 bytes (each part rounded to
 * 256) exceed 16 MiB - e.g. 64 rows x 32 heads x 8 splits fit, 512 rows x 64 heads x 8 do not.
 * All calls on a device share the one array and it keeps the previous call's contents; every
 * entry a call reads is written by that same call first, so nothing needs clearing, but two
 * calls that overlap on the GPU (different streams, no ordering) race on it.
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call before any stream capture begins.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL, CUDA. */
apar_status apar_tree_decode_attention_static(const void* k_pool /*[device]*/,
                                              const void* v_pool /*[device]*/,
                                              int32_t num_q_heads, int32_t num_kv_heads,
                                              int32_t n_threads, int32_t max_blocks_per_thread,
                                              const int32_t* block_tables /*[device]*/,
                                              const int32_t* ctx_lens /*[device]*/,
                                              int32_t max_ctx_len, const void* q /*[device]*/,
                                              void* out /*[device]*/, float sm_scale,
                                              void* cuda_stream);

/* Paragraph tree of Algorithm 1 (host only): which slice of which sequence belongs where in the
 * final text.  apar_paragraph_root makes thread tid (a prompt sequence, already holding its
 * prompt) the root: its node starts at the thread's current length.  From then on every
 * apar_fork of a tracked thread s at length L closes s's current node at L, opens the
 * next-sibling node (s, start L) and the first-child node (child, start L + 1: the child's
 * first appended row is taken to be the forced child token, which is not part of the text),
 * as the algorithm does when the last token of s is the fork token.  apar_restore writes the
 * slices (tid, start, end) in the order root, first child, next sibling; an open node ends at
 * its thread's current length (or at its length when it was released).  n receives the
 * number of slices; at most cap triples are written.
 * Errors: BAD_THREAD (unknown thread / not a root), INVALID_ARG. */
apar_status apar_paragraph_root(apar_ctx* ctx, int32_t tid);
apar_status apar_restore(apar_ctx* ctx, int32_t root_tid, int32_t* slices /*[host] 3 x cap*/,
                         int32_t cap, int32_t* n /*[host]*/);

/* Introspection (host state only; used to compare bookkeeping entry by entry). */
apar_status apar_get_thread(apar_ctx* ctx, int32_t tid, int32_t* len, int32_t* n_blocks,
                            int32_t* blocks /*[host] cap entries, may be NULL*/, int32_t cap);
apar_status apar_get_refcounts(apar_ctx* ctx, int32_t* refcnt /*[host] [num_blocks]*/);
/* ids in the order they will be handed out; n receives the count (<= cap are written). */
apar_status apar_get_free_list(apar_ctx* ctx, int32_t* ids /*[host]*/, int32_t cap, int32_t* n);
apar_status apar_get_stats(apar_ctx* ctx, apar_stats* out /*[host]*/);

/* Debug aid: checks the host tables against each other - every table entry is a valid block,
 * reference counts equal the number of table entries that name the block, free list and used
 * blocks partition the pool without repeats, table lengths match thread lengths.
 * Returns APAR_OK, or APAR_ERR_INVALID_ARG if an invariant is broken (a library bug). */
apar_status apar_check_invariants(apar_ctx* ctx);

/* Debug aid, host only (makes no CUDA call, needs no GPU): plans one attention call over
 * explicit block tables exactly as apar_tree_decode_attention_tables would and returns the
 * plan, so that the planner can be checked without a device.  The planner is the library's
 * own part of the path (the paper reads shared blocks once per thread; Section 2.3 only says
 * which blocks are shared).
 *   block_tables [host] [n_threads][max_blocks] block ids, ctx_lens [host] [n_threads] > 0
 *   mma_min_rows: items with at least this many query rows are classed for the tensor-core
 *                 kernels; fuse_final != 0: the last item of a chain that ends in a private
 *                 run finishes its query (folds the other partial results)
 *   items_out [host] [cap_items][8] int32: table_row, tok_begin, tok_end, user_begin, n_users,
 *             slot_add, fin_n, fin_begin (the fields of a work item; table_row = index of the
 *             thread whose table the item walks; fin_n holds the number of folded partial
 *             results in its low 8 bits and, from bit 8 on, one bit per folded part that is
 *             set when that part comes from an item of 2..16 rows)
 *   users_out [host] [cap_users][2] int32: query (thread index), partial slot or -1
 *   merges_out [host] [cap_merges][3] int32: query, first partial slot, number of slots
 *   counts_out [host] [6] int64: items, users, merges, partial slots, unique tokens,
 *              attended tokens
 * Returns APAR_ERR_WORKSPACE_TOO_SMALL if a cap is too small (counts_out is still filled),
 * APAR_ERR_INVALID_ARG for bad shapes, lengths or block ids, APAR_ERR_UNSUPPORTED for more
 * than 64 query heads per kv head. */
apar_status apar_debug_plan(int32_t num_blocks, int32_t num_q_heads, int32_t num_kv_heads,
                            int32_t n_threads, int32_t max_blocks, const int32_t* block_tables,
                            const int32_t* ctx_lens, int32_t mma_min_rows, int32_t fuse_final,
                            int32_t* items_out, int32_t cap_items, int32_t* users_out,
                            int32_t cap_users, int32_t* merges_out, int32_t cap_merges,
                            int64_t* counts_out);

/* Debug aid, host only: the plan apar_tree_decode_attention would make for the threads
 * tid[0..n) of this context (closed tails: token ranges are written out in full), in the same
 * output arrays as apar_debug_plan; table_row of an item is the library's internal row of the
 * thread.  by_groups != 0: the planner counts per group of blocks that the same threads hold
 * (what the library does when no thread is listed twice), which needs distinct ids;
 * by_groups == 0: it counts per block id, as apar_debug_plan does.  Both must give the same
 * plan.  Drops the context's cached plan.
 * Errors: INVALID_ARG, BAD_THREAD, EMPTY_CONTEXT, WORKSPACE_TOO_SMALL (counts_out filled). */
apar_status apar_debug_plan_threads(apar_ctx* ctx, int32_t n, const int32_t* tid /*[host]*/,
                                    int32_t by_groups, int32_t mma_min_rows, int32_t fuse_final,
                                    int32_t* items_out, int32_t cap_items, int32_t* users_out,
                                    int32_t cap_users, int32_t* merges_out, int32_t cap_merges,
                                    int64_t* counts_out);

/* Measurement aid (the paper has no counterpart): enqueues one kernel that reads `bytes` bytes
 * (rounded down to a multiple of 16) at `src` once, with the 16-byte streaming loads the
 * attention kernels use, and xors them into the 8-byte word at `sink`.  Timing it over a buffer
 * much larger than the L2 cache gives the read-only HBM rate, the ceiling for attention, which
 * reads far more than it writes.
 *   src   [device] 16-byte aligned, caller-owned, not modified
 *   sink  [device] 8-byte aligned word, caller-owned; its old value is xor-ed into, not cleared
 * Returns APAR_ERR_INVALID_ARG for NULL or misaligned pointers, APAR_ERR_CUDA if the launch
 * failed (no context, so the CUDA error is read with cudaGetLastError by the caller). */
apar_status apar_stream_read(const void* src, size_t bytes, void* sink, void* cuda_stream);

/* Measurement aid (the paper has no counterpart): from now on every attention call of this
 * context (apar_tree_decode_attention, apar_decode_step, the prefix and layer forms) records
 * `start` on its stream just before its attention kernels and `stop` just after them, so that
 * the caller can time those kernels alone inside a larger call.  Both are cudaEvent_t handles
 * created by the caller with timing enabled; the library does not own them.  NULL, NULL turns
 * it off.  Errors: INVALID_ARG if only one of the two is NULL. */
apar_status apar_set_timing_events(apar_ctx* ctx, void* start, void* stop);

/* cudaError_t value of the most recent failing CUDA call of this context (0 if none). */
int32_t     apar_last_cuda_error(apar_ctx* ctx);
const char* apar_status_string(apar_status s);

#ifdef __cplusplus
}
#endif
#endif  /* APAR_H_ */

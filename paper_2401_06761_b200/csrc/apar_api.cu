// C-ABI entry points (include/apar.h): host bookkeeping of the paged pool, staging of
// per-call metadata, and the launch sequence of each call.
#include <algorithm>
#include <chrono>
#include <climits>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/apar.h"
#include "apar_internal.h"

using namespace apar;

namespace {

constexpr int kRing = 12;             // pinned staging buffers in flight: enough for the uploads of
                                      // two whole steps, so that the host can prepare a step
                                      // while the GPU still runs the one before
constexpr int kFewQueries = 768;      // up to here single-row items go to the warp-stream kernel
constexpr int kSlotsPerThread = 6;    // partial-result rows provisioned per live thread
constexpr int kMinSlots = 1184;       // and never fewer than this (8 per SM of a 148-SM part), so
                                      // that a few very long threads still spread over the machine
constexpr int kSlotMapRows = 262144;  // new-row slots of the last append kept for other layers

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {            // partition of the caller's workspace
  size_t err, ticket, tables, lens, stage, slot_map, step_rows, verify, plan_items, plan_users, plan_merges, part_ml, part_flag, part_o, total;
  size_t stage_cap;        // bytes of the transient staging area
  int64_t slot_capacity;   // partial rows (before the head dimension)
  int64_t entry_capacity;  // (item, user) pairs a plan may hold
};

bool supported(const apar_config* c) {
  return c && c->block_size == kBlock && c->head_dim == kDim && c->num_blocks > 0 &&
         c->num_kv_heads > 0 && c->num_q_heads > 0 && c->num_q_heads % c->num_kv_heads == 0 &&
         // one work item carries all query heads of a kv head for at least one thread
         c->num_q_heads / c->num_kv_heads <= kMaxRowsPerItem &&
         c->max_threads > 0 && c->max_blocks_per_thread > 0 && c->num_layers >= 0 &&
         (int64_t)c->num_blocks * kBlock < INT32_MAX &&
         (int64_t)std::max(1, c->num_layers) * c->num_blocks * c->num_kv_heads * kBlock < INT32_MAX;
}

Layout make_layout(const apar_config* c) {
  Layout L;
  const size_t table_bytes = (size_t)c->max_threads * c->max_blocks_per_thread * 4;
  L.slot_capacity = std::max<int64_t>((int64_t)c->max_threads * kSlotsPerThread, kMinSlots);
  L.entry_capacity = L.slot_capacity + c->max_threads;
  L.stage_cap = std::min<size_t>(std::max<size_t>(table_bytes / 4 + (64 << 10), 1 << 20), 64 << 20);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.err = take(256);
  L.ticket = take(256);
  L.tables = take(table_bytes);
  L.lens = take((size_t)c->max_threads * 4);
  L.stage = take(L.stage_cap);
  L.slot_map = take((size_t)std::max(kSlotMapRows, c->max_threads) * 4);
  L.step_rows = take((size_t)c->max_threads * 4);
  L.verify = take((size_t)c->max_threads * sizeof(VerifyDesc));
  L.plan_items = take((size_t)L.entry_capacity * sizeof(WorkItem));
  L.plan_users = take((size_t)L.entry_capacity * sizeof(UserRef));
  L.plan_merges = take((size_t)c->max_threads * sizeof(MergeRef));
  L.part_ml = take((size_t)L.slot_capacity * c->num_q_heads * sizeof(float2));
  L.part_flag = take((size_t)L.slot_capacity * c->num_q_heads * sizeof(int32_t));
  L.part_o = take((size_t)L.slot_capacity * c->num_q_heads * kDim * sizeof(float));
  L.total = off;
  return L;
}

struct ThreadRec {
  int32_t tid = -1;       // -1: slot free
  int32_t len = 0;
  int32_t n_blocks = 0;
  int32_t synced = 0;     // table entries already on the device
  int32_t dev_len = -1;   // length the device array holds for this slot
};

struct Staging {
  char* host = nullptr;
  char* mapped = nullptr;   // the same buffer as the device sees it
  cudaEvent_t done = nullptr;
  bool in_flight = false;
};

}  // namespace

struct apar_ctx {
  apar_config cfg;
  Shape shape;
  Layout lay;
  // ---- host bookkeeping
  std::vector<int32_t> free_stack;     // top of the stack at the back
  std::vector<int32_t> refcnt;
  std::vector<int32_t> tables;         // [max_threads][max_blocks_per_thread] by slot
  std::vector<ThreadRec> slots;
  std::vector<int32_t> free_slots;
  std::vector<int32_t> tid_slot;       // tid -> slot or -1
  int32_t next_tid = 0;
  int64_t live = 0;
  int64_t forks = 0, cow_blocks = 0, cow_rows = 0, kernels_total = 0, peak_used = 0;
  apar_stats last = {};
  std::vector<uint32_t> mark;          // per slot, duplicate detection
  uint32_t mark_epoch = 0;
  // ---- staging
  Staging ring[kRing];
  size_t ring_bytes = 0;
  int ring_next = 0, ring_n = kRing;   // buffers in use (a one-call context needs few)
  // ---- planning
  Planner planner;
  Plan plan;
  std::vector<PlanQuery> pq;
  std::vector<int32_t> plan_tids;
  uint64_t struct_epoch = 1, plan_epoch = 0;
  int64_t plan_attended = 0;
  int plan_age = 0;
  int mma_min_rows = INT_MAX;
  int plan_min_rows = INT_MAX;          // the value the current plan was built with
  bool auto_path = true;                // no kernel family forced
  int umma_heads = 0;                   // > 0: kv heads per CTA of the tcgen05 kernel (testing)
  int umma_mode = 0;                    // 1: one CTA per (item, heads); 2: persistent CTAs
  int ws_mode = 0;                      // 1: one CTA per item; 2: persistent warps
  int64_t prefill_batch = INT64_MAX;    // tree-masked attention: work items per launch, at most
                                        // (testing)
  int num_sms = 148;
  int use_pdl = 1;                      // warp-stream launches may start before the kernel before
                                        // them has finished (0: ordinary launches only)
  bool use_ws = true;                   // single-tile items use the warp-stream kernel
  std::vector<CUtensorMap> tm_k, tm_v;   // one pair per layer
  size_t layer_bytes = 0;                // bytes of one layer of a pool
  int num_layers = 1;
  uint64_t book_seq = 1, attn_book_seq = 0;   // bookkeeping calls so far / at the last plan
  int64_t last_append_rows = -1;              // rows of the last append kept in the slot map
  int plan_verify_n = 0;                      // candidate descriptors that belong to the plan
  int32_t last_cuda = 0;
  bool host_only = false;                     // bookkeeping only: no device, nothing is launched
  // Every thread's table as runs of groups (blocks held by the same set of threads).  A
  // thread's blocks since it was last forked form its own, open group; a fork closes the full
  // blocks of that group (the child lists them from then on) and opens a new one.
  std::vector<std::vector<BlockRun>> runs;    // by slot
  std::vector<uint8_t> own_open;              // by slot: the last run is the open group
  std::vector<int32_t> gid_ref, gid_free;     // threads listing each group; ids to reuse
  bool track_runs = true;                     // false: tables were filled in directly
  bool plan_by_runs = true;                   // APAR_PLANNER=tables (testing): walk block ids
  cudaEvent_t time_start = nullptr, time_stop = nullptr;   // caller's events around the kernels
  // thread list of the most recent apar_decode_step; its table rows are resident on the device
  std::vector<int32_t> step_tids, step_slots, tmp_slots;
  bool step_valid = false;
  uint64_t life_seq = 1, mod_seq = 1;         // releases so far / appends outside apar_decode_step
  uint64_t step_life = 0, step_mod = 0;       // their values when the list was last brought in sync
  // paragraph tree of Algorithm 1 (host only)
  struct PNodeRec { int32_t tid, start, end, first_child, next_sibling; };
  std::vector<PNodeRec> pnodes;
  std::vector<int32_t> cur_node, root_node;   // by thread id; -1: not tracked / not a root

  int32_t* row(int slot) { return tables.data() + (size_t)slot * cfg.max_blocks_per_thread; }
  char* ws(size_t off) { return (char*)cfg.workspace + off; }
};

namespace {

#define APAR_CUDA(ctx, expr)                         \
  do {                                               \
    cudaError_t e_ = (expr);                         \
    if (e_ != cudaSuccess) {                         \
      (ctx)->last_cuda = (int32_t)e_;                \
      return APAR_ERR_CUDA;                          \
    }                                                \
  } while (0)

// Next pinned buffer, once the copy that last used it has completed.
apar_status acquire(apar_ctx* c, Staging** out) {
  Staging* s = &c->ring[c->ring_next];
  c->ring_next = (c->ring_next + 1) % c->ring_n;
  if (s->in_flight) {
    APAR_CUDA(c, cudaEventSynchronize(s->done));
    s->in_flight = false;
  }
  *out = s;
  return APAR_OK;
}

apar_status send(apar_ctx* c, Staging* s, void* dst, size_t bytes, cudaStream_t st) {
  // By a kernel, not a copy engine: these uploads gate the step's kernels and must not wait
  // behind an application's large host-to-device copy on another stream.
  if (bytes % 4 == 0 && s->mapped) {
    if (bytes) {
      APAR_CUDA(c, launch_stage_copy(dst, s->mapped, bytes, st));
      ++c->kernels_total;
    }
  } else if (bytes) {
    APAR_CUDA(c, cudaMemcpyAsync(dst, s->host, bytes, cudaMemcpyHostToDevice, st));
  }
  APAR_CUDA(c, cudaEventRecord(s->done, st));
  s->in_flight = true;
  return APAR_OK;
}

int slot_of(apar_ctx* c, int32_t tid) {
  if (tid < 0 || tid >= (int32_t)c->tid_slot.size()) return -1;
  return c->tid_slot[tid];
}

uint32_t next_mark(apar_ctx* c) {
  if (++c->mark_epoch == 0) {
    std::fill(c->mark.begin(), c->mark.end(), 0u);
    c->mark_epoch = 1;
  }
  return c->mark_epoch;
}

int32_t new_slot(apar_ctx* c) {
  const int32_t s = c->free_slots.back();
  c->free_slots.pop_back();
  ThreadRec& t = c->slots[s];
  t = ThreadRec();
  t.tid = c->next_tid++;
  c->tid_slot.push_back(s);
  c->cur_node.push_back(-1);
  c->root_node.push_back(-1);
  ++c->live;
  return s;
}

int32_t alloc_block(apar_ctx* c) {
  const int32_t b = c->free_stack.back();
  c->free_stack.pop_back();
  c->refcnt[b] = 1;
  c->peak_used = std::max<int64_t>(c->peak_used, c->cfg.num_blocks - (int64_t)c->free_stack.size());
  return b;
}

int32_t new_gid(apar_ctx* c) {
  int32_t g;
  if (!c->gid_free.empty()) {
    g = c->gid_free.back();
    c->gid_free.pop_back();
  } else {
    g = (int32_t)c->gid_ref.size();
    c->gid_ref.push_back(0);
  }
  c->gid_ref[g] = 1;
  return g;
}

// The thread in `slot` gained a block at table position `pos` (its new last block).
void run_add_block(apar_ctx* c, int slot, int32_t pos) {
  std::vector<BlockRun>& r = c->runs[slot];
  if (c->own_open[slot]) {
    ++r.back().n;
  } else {
    r.push_back(BlockRun{new_gid(c), pos, 1});
    c->own_open[slot] = 1;
  }
}

// Fork of the thread in slot `ps`, which holds `full` full blocks, into the fresh slot `cs`:
// the full blocks of the parent's open group become a group of their own, shared from now
// on, and the child lists every run below `full`.
void run_fork(apar_ctx* c, int ps, int cs, int32_t full) {
  std::vector<BlockRun>& pr = c->runs[ps];
  if (c->own_open[ps]) {
    BlockRun& last = pr.back();
    if (full > last.pos) {
      if (last.pos + last.n > full) {           // the partial block stays the parent's own
        const int32_t rest = last.pos + last.n - full;
        last.n = full - last.pos;
        pr.push_back(BlockRun{new_gid(c), full, rest});
      } else {
        c->own_open[ps] = 0;                    // all of it full: the next block opens a group
      }
    }
  }
  std::vector<BlockRun>& cr = c->runs[cs];
  cr.clear();
  for (const BlockRun& r : pr) {
    if (r.pos + r.n > full) break;
    cr.push_back(r);
    ++c->gid_ref[r.gid];
  }
  c->own_open[cs] = 0;
}

void run_release(apar_ctx* c, int slot) {
  for (const BlockRun& r : c->runs[slot])
    if (--c->gid_ref[r.gid] == 0) c->gid_free.push_back(r.gid);
  c->runs[slot].clear();
  c->own_open[slot] = 0;
}

// Brings the device copies of block tables and lengths up to date for the given slots.
apar_status sync_device_tables(apar_ctx* c, const int32_t* slots, int n, cudaStream_t st) {
  int i = 0;
  while (i < n) {
    Staging* s;
    apar_status rc = acquire(c, &s);
    if (rc) return rc;
    // layout inside the staging area: [deltas][pairs][data]; sized so that all three fit
    const size_t cap = c->lay.stage_cap;
    const int max_entries = (int)std::min<size_t>(cap / 4 / sizeof(TableDelta), 1 << 20);
    TableDelta* deltas = (TableDelta*)s->host;
    int32_t* pairs = (int32_t*)(s->host + (size_t)max_entries * sizeof(TableDelta));
    int32_t* data = pairs + 2 * (size_t)max_entries;
    const size_t data_cap = (cap - ((char*)data - s->host)) / 4;
    int nd = 0, np = 0;
    size_t used = 0;
    const uint32_t mk = next_mark(c);
    for (; i < n; ++i) {
      ThreadRec& t = c->slots[slots[i]];
      if (c->mark[slots[i]] == mk) continue;           // listed twice in this round
      const int need = t.n_blocks - t.synced;
      if (need > 0 && (nd >= max_entries || used + need > data_cap)) break;
      if (t.dev_len != t.len && np >= max_entries) break;
      c->mark[slots[i]] = mk;
      if (need > 0) {
        deltas[nd++] = TableDelta{slots[i], t.synced, need, (int32_t)used};
        memcpy(data + used, c->row(slots[i]) + t.synced, (size_t)need * 4);
        used += need;
        t.synced = t.n_blocks;
      }
      if (t.dev_len != t.len) {
        pairs[2 * np] = slots[i];
        pairs[2 * np + 1] = t.len;
        ++np;
        t.dev_len = t.len;
      }
    }
    if (nd == 0 && np == 0) {
      if (i < n) return APAR_ERR_WORKSPACE_TOO_SMALL;   // one row larger than the staging area
      break;
    }
    // close the gaps between the three arrays, so that only what was filled crosses PCIe
    const size_t off_pairs = (size_t)nd * sizeof(TableDelta);
    const size_t off_data = off_pairs + (size_t)np * 8;
    c->last.attn_upload_bytes += (int64_t)(off_data + used * 4);
    memmove(s->host + off_pairs, pairs, (size_t)np * 8);
    memmove(s->host + off_data, data, used * 4);
    // Every entry is read exactly once, so the kernel takes them straight from the pinned
    // buffer (mapped into the device's address space) instead of from a device copy.
    const char* src = s->mapped;
    if (!src) {
      src = c->ws(c->lay.stage);
      rc = send(c, s, c->ws(c->lay.stage), off_data + used * 4, st);
      if (rc) return rc;
    }
    APAR_CUDA(c, launch_sync((int32_t*)c->ws(c->lay.tables), c->cfg.max_blocks_per_thread,
                             (int32_t*)c->ws(c->lay.lens), (const TableDelta*)src,
                             (const int32_t*)(src + off_data), nd,
                             (const int32_t*)(src + off_pairs), np, st));
    if (s->mapped) {
      rc = send(c, s, nullptr, 0, st);      // nothing to copy: only marks the buffer in flight
      if (rc) return rc;
    }
    ++c->kernels_total;
    ++c->last.attn_kernels;
  }
  return APAR_OK;
}

// Launch sequence of the current plan on one layer of the pools.
apar_status launch_plan(apar_ctx* c, int layer, const void* q, void* out, float sm_scale,
                        cudaStream_t st, int* launches_out) {
  const Plan& p = c->plan;
  AttnArgs a;
  a.q = q;
  a.out = out;
  a.k_pool = (const char*)c->cfg.k_pool + (size_t)layer * c->layer_bytes;
  a.v_pool = (const char*)c->cfg.v_pool + (size_t)layer * c->layer_bytes;
  a.d_tables = (const int32_t*)c->ws(c->lay.tables);
  a.d_lens = (const int32_t*)c->ws(c->lay.lens);
  a.d_items = (const WorkItem*)c->ws(c->lay.plan_items);
  a.d_users = (const UserRef*)c->ws(c->lay.plan_users);
  a.part_o = (float*)c->ws(c->lay.part_o);
  a.part_ml = (float2*)c->ws(c->lay.part_ml);
  a.shape = c->shape;
  a.scale_log2e = sm_scale * 1.4426950408889634f;
  a.tm_k = &c->tm_k[layer];
  a.tm_v = &c->tm_v[layer];
  a.d_error = (int*)c->ws(c->lay.err);
  a.num_sms = c->num_sms;
  a.umma_heads = c->umma_heads;
  a.umma_mode = c->umma_mode;
  a.ws_mode = c->ws_mode;
  a.d_ticket = (int*)c->ws(c->lay.ticket);
  // The first attention kernel of the call is launched the ordinary way (it starts after the
  // table sync and the append have completed).  A warp-stream launch that follows another
  // attention kernel may start while that kernel is still in its last wave, and orders itself
  // where it has to (pdl_wait).  Measured: worth 2 % where tensor-core and warp-stream
  // kernels follow each other (config 5), nothing on config 4; the single-row kernel lost
  // 10-25 % when its finishing items started early (configs 2 and 3), so it and the merge are
  // launched the ordinary way, which also orders them after everything before them.
  const int chain = c->use_pdl ? 1 : 0;
  bool first = true;
  // Single-tile items go to the warp-stream kernel (unless the tcgen05 kernel is forced for
  // everything).  Its persistent form takes plain and finishing items in ONE launch: the unit
  // counter hands out the plain ones first, and a finishing unit waits for the ready flag of
  // each partial result that a plain unit of the same launch produces.
  const int n_ws = (c->use_ws && p.n_mma) ? p.n_mma_tiles[0] : 0;
  const int n_ws_final = c->use_ws ? p.n_mma1_final : 0;
  const bool ws_merged = c->ws_mode != 1 && n_ws_final > 0 && n_ws > n_ws_final;
  // (flags and unit counters look after themselves: the flags carry the number of the launch
  // that wrote them, the counters are put back to zero by the last warp of a launch)
  if (ws_merged) a.part_flag = (int*)c->ws(c->lay.part_flag);
  if (p.n_mma) {
    // items are ordered 4, 3, 2, 1 query tiles, finishing items last
    const int n_umma = p.n_mma - n_ws;
    if (n_umma) {
      a.pdl = 0;
      APAR_CUDA(c, launch_attention_umma(a, p.n_vec, n_umma, st));
      ++*launches_out;
      first = false;
    }
    const int n_now = ws_merged ? n_ws : n_ws - n_ws_final;
    if (n_now > 0) {
      a.pdl = first ? 0 : chain;
      APAR_CUDA(c, launch_attention_ws(a, p.n_vec + n_umma, n_now, st, 1));
      ++*launches_out;
      first = false;
    }
  }
  a.part_flag = nullptr;
  const bool single_row = c->shape.group == 1 && c->plan_min_rows <= 2;
  a.pdl = 0;
  if (p.n_vec - p.n_vec_final > 0) {
    APAR_CUDA(c, launch_attention_vec(a, 0, p.n_vec - p.n_vec_final, single_row, st));
    ++*launches_out;
    first = false;
  }
  // finishing items: everything they fold has been enqueued before them on this stream
  if (p.n_mma1_final > 0 && !ws_merged) {
    a.pdl = first ? 0 : chain;
    APAR_CUDA(c, launch_attention_ws(a, p.n_vec + p.n_mma - p.n_mma1_final, p.n_mma1_final, st, 2));
    ++*launches_out;
    first = false;
  }
  a.pdl = 0;
  if (p.n_vec_final > 0) {
    APAR_CUDA(c, launch_attention_vec(a, p.n_vec - p.n_vec_final, p.n_vec_final, single_row, st));
    ++*launches_out;
  }
  // candidate tokens of a verification step: their own partial result per query
  if (c->plan_verify_n > 0) {
    APAR_CUDA(c, launch_verify_tail(a, (const VerifyDesc*)c->ws(c->lay.verify), c->plan_verify_n,
                                    st));
    ++*launches_out;
  }
  if (!p.merges.empty()) {
    APAR_CUDA(c, launch_merge(a, (const MergeRef*)c->ws(c->lay.plan_merges),
                              (int)p.merges.size(), st));
    ++*launches_out;
  }
  return APAR_OK;
}

// A plan is kept while the tree is unchanged and the same threads are queried; it is rebuilt
// now and then only because the longest-first order of its items drifts as tails grow.
bool plan_reusable(const apar_ctx* c, int n, const int32_t* tids, int64_t attended) {
  return c->plan_epoch == c->struct_epoch && c->plan_age < 1024 &&
         (int)c->plan_tids.size() == n &&
         memcmp(c->plan_tids.data(), tids, (size_t)n * 4) == 0 &&
         attended - c->plan_attended < c->plan_attended / 4 + 64;
}

// The attention launch sequence for queries given as slots (already validated, len > 0).
// qlens (optional): tokens query i attends, counted from the root; default the thread's length.
apar_status run_attention(apar_ctx* c, int n, const int32_t* qslots, const int32_t* tids,
                          bool has_dups, const void* q, void* out, float sm_scale,
                          cudaStream_t st, const int32_t* qlens = nullptr,
                          bool tables_in_sync = false, std::vector<VerifyDesc>* verify = nullptr) {
  c->last.attn_kernels = 0;
  int64_t attended = 0;
  for (int i = 0; i < n; ++i) attended += qlens ? qlens[i] : c->slots[qslots[i]].len;

  const bool cacheable = tids != nullptr && !has_dups && !qlens;
  bool reuse = cacheable && plan_reusable(c, n, tids, attended);
  c->last.attn_plan_host_us = 0;
  if (!tables_in_sync) c->last.attn_upload_bytes = 0;   // (else the caller's uploads count too)
  if (!reuse) {
    const auto t_plan = std::chrono::steady_clock::now();
    c->pq.resize(n);
    // every query attends its thread's whole chain and no thread is listed twice: the planner
    // may count per group of blocks instead of per block
    const bool by_runs = cacheable && c->track_runs && c->plan_by_runs;
    for (int i = 0; i < n; ++i) {
      c->pq[i] = PlanQuery{c->row(qslots[i]), qslots[i],
                           qlens ? qlens[i] : c->slots[qslots[i]].len};
      if (by_runs) {
        c->pq[i].runs = c->runs[qslots[i]].data();
        c->pq[i].n_runs = (int32_t)c->runs[qslots[i]].size();
      }
      if (verify) c->pq[i].extra_parts = 1;
    }
    c->plan_verify_n = 0;
    // Single-row items (no GQA group, private tail): the vector kernel keeps up to 16 CTAs per
    // SM in flight and wins when there are many of them; with few, the warp-stream kernel's
    // deeper per-warp rings do better (measured crossover near 900 queries).
    c->plan_min_rows = c->mma_min_rows;
    if (c->auto_path && c->shape.group == 1 && n <= kFewQueries) c->plan_min_rows = 1;
    // finishing items land in the single-row vector kernel or the warp-stream kernel
    const bool fuse_final = c->use_ws && c->plan_min_rows <= 2 && !verify;
    if (!c->planner.build(c->pq.data(), n, c->lay.slot_capacity, cacheable, c->plan_min_rows,
                          fuse_final, &c->plan, by_runs))
      return APAR_ERR_WORKSPACE_TOO_SMALL;
    if ((int64_t)c->plan.users.size() > c->lay.entry_capacity ||
        (int64_t)c->plan.items.size() > c->lay.entry_capacity)
      return APAR_ERR_WORKSPACE_TOO_SMALL;
    c->last.attn_plan_host_us = std::chrono::duration_cast<std::chrono::microseconds>(
                                    std::chrono::steady_clock::now() - t_plan).count();
  }
  apar_status rc = tables_in_sync ? APAR_OK : sync_device_tables(c, qslots, n, st);
  if (rc) return rc;

  const Plan& p = c->plan;
  if (!reuse) {
    const size_t b_items = p.items.size() * sizeof(WorkItem);
    const size_t b_users = p.users.size() * sizeof(UserRef);
    const size_t b_merges = p.merges.size() * sizeof(MergeRef);
    struct Part { const void* src; size_t bytes, dst; } parts[3] = {
        {p.items.data(), b_items, c->lay.plan_items},
        {p.users.data(), b_users, c->lay.plan_users},
        {p.merges.data(), b_merges, c->lay.plan_merges}};
    for (const Part& part : parts) {
      size_t done = 0;
      while (done < part.bytes) {
        Staging* s;
        rc = acquire(c, &s);
        if (rc) return rc;
        const size_t chunk = std::min(part.bytes - done, c->ring_bytes);
        memcpy(s->host, (const char*)part.src + done, chunk);
        rc = send(c, s, c->ws(part.dst) + done, chunk, st);
        if (rc) return rc;
        c->last.attn_upload_bytes += (int64_t)chunk;
        done += chunk;
      }
    }
    if (verify) {
      // every candidate's descriptor learns where its partial result goes
      if ((size_t)n * sizeof(VerifyDesc) > c->ring_bytes) return APAR_ERR_WORKSPACE_TOO_SMALL;
      for (int i = 0; i < n; ++i) (*verify)[i].slot = p.extra_slot[i];
      Staging* s;
      rc = acquire(c, &s);
      if (rc) return rc;
      memcpy(s->host, verify->data(), (size_t)n * sizeof(VerifyDesc));
      rc = send(c, s, c->ws(c->lay.verify), (size_t)n * sizeof(VerifyDesc), st);
      if (rc) return rc;
      c->last.attn_upload_bytes += (int64_t)n * sizeof(VerifyDesc);
      c->plan_verify_n = n;
    }
    if (cacheable) {
      c->plan_tids.assign(tids, tids + n);
      c->plan_epoch = c->struct_epoch;
      c->plan_attended = attended;
      c->plan_age = 0;
    } else {
      c->plan_epoch = 0;
    }
  } else {
    ++c->plan_age;
  }

  int launches = 0;
  if (c->time_start) APAR_CUDA(c, cudaEventRecord(c->time_start, st));
  rc = launch_plan(c, 0, q, out, sm_scale, st, &launches);
  if (rc) return rc;
  if (c->time_stop) APAR_CUDA(c, cudaEventRecord(c->time_stop, st));
  c->attn_book_seq = c->book_seq;
  c->kernels_total += launches;
  c->last.attn_kernels += launches;
  c->last.attn_threads = n;
  c->last.attn_attended_tokens = attended;
  c->last.attn_unique_tokens = p.unique_tokens + (reuse ? attended - c->plan_attended : 0);
  c->last.attn_work_items = (int64_t)p.items.size();
  c->last.attn_partials = p.total_slots * c->shape.num_q_heads;
  c->last.attn_plan_reused = reuse ? 1 : 0;
  c->last.attn_vec_items = p.n_vec;
  c->last.attn_mma_items = p.n_mma;
  return APAR_OK;
}

apar_status create_impl(const apar_config* cfg, bool external, bool host_only, apar_ctx** out) {
  if (!cfg || !out) return APAR_ERR_INVALID_ARG;
  if (!supported(cfg)) return APAR_ERR_UNSUPPORTED;
  const Layout lay = make_layout(cfg);
  if (!host_only) {
    if (!cfg->k_pool || !cfg->v_pool || !cfg->workspace) return APAR_ERR_INVALID_ARG;
    if (((uintptr_t)cfg->k_pool | (uintptr_t)cfg->v_pool) & 255) return APAR_ERR_INVALID_ARG;
    if ((uintptr_t)cfg->workspace & 255) return APAR_ERR_INVALID_ARG;
    if (cfg->workspace_bytes < lay.total) return APAR_ERR_WORKSPACE_TOO_SMALL;
  }
  apar_ctx* c = new (std::nothrow) apar_ctx();
  if (!c) return APAR_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->host_only = host_only;
  c->track_runs = !external;
  c->runs.resize(cfg->max_threads);
  c->own_open.assign(cfg->max_threads, 0);
  c->lay = lay;
  c->shape = Shape{cfg->num_q_heads, cfg->num_kv_heads, cfg->num_q_heads / cfg->num_kv_heads,
                   cfg->max_blocks_per_thread};
  c->refcnt.assign(cfg->num_blocks, 0);
  c->free_stack.resize(cfg->num_blocks);
  for (int i = 0; i < cfg->num_blocks; ++i) c->free_stack[i] = cfg->num_blocks - 1 - i;
  c->tables.assign((size_t)cfg->max_threads * cfg->max_blocks_per_thread, 0);
  c->slots.assign(cfg->max_threads, ThreadRec());
  c->free_slots.resize(cfg->max_threads);
  for (int i = 0; i < cfg->max_threads; ++i) c->free_slots[i] = cfg->max_threads - 1 - i;
  c->mark.assign(cfg->max_threads, 0);
  c->planner.init(cfg->num_blocks, c->shape.group, cfg->num_kv_heads);
  // Testing switches, read once here.  APAR_ATTN_PATH forces one kernel family for every item
  // it can take: "vec" CUDA cores only, "umma" tcgen05 for every multi-row item, "ws" the
  // warp-stream kernel also for single rows.  Default ("auto"): 1 row vector kernel (warp-
  // stream when the call has few queries), up to 16 rows warp-stream, more rows tcgen05.
  const char* path = getenv("APAR_ATTN_PATH");
  c->mma_min_rows = (path && !strcmp(path, "vec")) ? INT_MAX : (path && !strcmp(path, "ws")) ? 1 : 2;
  const char* pdl = getenv("APAR_PDL");                  // 0 = ordinary launches only
  c->use_pdl = pdl ? atoi(pdl) : 1;
  c->use_ws = !(path && !strcmp(path, "umma"));
  const char* heads = getenv("APAR_UMMA_HEADS");         // kv heads per CTA of the tcgen05 kernel
  c->umma_heads = heads ? atoi(heads) : 0;
  const char* mode = getenv("APAR_UMMA_MODE");           // "grid" | "persist"
  c->umma_mode = (mode && !strcmp(mode, "grid")) ? 1 : (mode && !strcmp(mode, "persist")) ? 2 : 0;
  mode = getenv("APAR_WS_MODE");                         // "grid" | "persist"
  c->ws_mode = (mode && !strcmp(mode, "grid")) ? 1 : (mode && !strcmp(mode, "persist")) ? 2 : 0;
  mode = getenv("APAR_PREFILL_BATCH");                   // tree-masked attention: work items per
                                                         // launch, at most
  if (mode && atoll(mode) > 0) c->prefill_batch = atoll(mode);
  c->auto_path = !path || !strcmp(path, "auto") || !*path;
  const char* planner = getenv("APAR_PLANNER");          // testing: "tables" = per-block walk
  c->plan_by_runs = !(planner && !strcmp(planner, "tables"));
  c->ring_bytes = lay.stage_cap;
  c->num_layers = std::max(1, cfg->num_layers);
  c->layer_bytes = (size_t)cfg->num_blocks * cfg->num_kv_heads * kTileBytes;
  if (host_only) {
    *out = c;
    return APAR_OK;
  }
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      c->num_sms = sms;
    c->planner.set_num_sms(c->num_sms);
  }
  c->tm_k.resize(c->num_layers);
  c->tm_v.resize(c->num_layers);
  bool maps_ok = true;
  for (int l = 0; l < c->num_layers && maps_ok; ++l)
    maps_ok = make_pool_tensor_maps((char*)cfg->k_pool + l * c->layer_bytes,
                                    (char*)cfg->v_pool + l * c->layer_bytes, cfg->num_blocks,
                                    cfg->num_kv_heads, &c->tm_k[l], &c->tm_v[l]) == 0;
  if (!maps_ok || cudaMemset(c->ws(lay.err), 0, 256) != cudaSuccess ||
      cudaMemset(c->ws(lay.ticket), 0, 256) != cudaSuccess ||
      cudaMemset(c->ws(lay.part_flag), 0,
                 (size_t)lay.slot_capacity * cfg->num_q_heads * sizeof(int32_t)) != cudaSuccess) {
    c->last_cuda = (int32_t)cudaGetLastError();
    delete c;
    return APAR_ERR_CUDA;
  }
  c->ring_n = external ? 2 : kRing;
  for (int i = 0; i < c->ring_n; ++i) {
    cudaError_t e = cudaHostAlloc((void**)&c->ring[i].host, c->ring_bytes, cudaHostAllocMapped);
    if (e == cudaSuccess)
      e = cudaHostGetDevicePointer((void**)&c->ring[i].mapped, c->ring[i].host, 0);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ring[i].done, cudaEventDisableTiming);
    if (e != cudaSuccess) {
      apar_destroy(c);
      return APAR_ERR_CUDA;
    }
  }
  *out = c;
  return APAR_OK;
}

}  // namespace

extern "C" {

size_t apar_workspace_bytes(const apar_config* cfg) {
  if (!supported(cfg)) return 0;
  return make_layout(cfg).total;
}

apar_status apar_create(const apar_config* cfg, apar_ctx** out) {
  return create_impl(cfg, false, false, out);
}

apar_status apar_create_host_only(const apar_config* cfg, apar_ctx** out) {
  return create_impl(cfg, false, true, out);
}

apar_status apar_destroy(apar_ctx* c) {
  if (!c) return APAR_ERR_INVALID_ARG;
  for (int i = 0; i < kRing; ++i) {
    if (c->ring[i].in_flight) cudaEventSynchronize(c->ring[i].done);
    if (c->ring[i].done) cudaEventDestroy(c->ring[i].done);
    if (c->ring[i].host) cudaFreeHost(c->ring[i].host);
  }
  delete c;
  return APAR_OK;
}

apar_status apar_new_threads(apar_ctx* c, int32_t n, int32_t* tid_out) {
  if (!c || n < 0 || (n > 0 && !tid_out)) return APAR_ERR_INVALID_ARG;
  if (c->live + n > c->cfg.max_threads) return APAR_ERR_NO_THREADS;
  for (int i = 0; i < n; ++i) tid_out[i] = c->slots[new_slot(c)].tid;
  if (n) ++c->struct_epoch;
  ++c->book_seq;
  return APAR_OK;
}

apar_status apar_fork(apar_ctx* c, int32_t n, const int32_t* parent_tid, int32_t* child_tid_out,
                      void* cuda_stream) {
  if (!c || n < 0 || (n > 0 && (!parent_tid || !child_tid_out))) return APAR_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int need = 0;
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, parent_tid[i]);
    if (s < 0) return APAR_ERR_BAD_THREAD;
    if (c->slots[s].len % kBlock) ++need;
  }
  if (c->live + n > c->cfg.max_threads) return APAR_ERR_NO_THREADS;
  if (need > (int)c->free_stack.size()) return APAR_ERR_NO_BLOCKS;
  if ((size_t)need * sizeof(CowCopy) > c->lay.stage_cap) return APAR_ERR_WORKSPACE_TOO_SMALL;
  Staging* stg = nullptr;
  if (need && !c->host_only) {
    apar_status rc = acquire(c, &stg);
    if (rc) return rc;
  }
  CowCopy* copies = stg ? (CowCopy*)stg->host : nullptr;
  int nc = 0;
  for (int i = 0; i < n; ++i) {
    const int ps = slot_of(c, parent_tid[i]);
    const int32_t L = c->slots[ps].len, full = L / kBlock, r = L % kBlock;
    const int cs = new_slot(c);
    ThreadRec& ch = c->slots[cs];
    int32_t* ct = c->row(cs);
    const int32_t* pt = c->row(ps);
    for (int b = 0; b < full; ++b) {
      ct[b] = pt[b];
      ++c->refcnt[pt[b]];
    }
    ch.n_blocks = full;
    run_fork(c, ps, cs, full);
    if (r) {
      const int32_t dst = alloc_block(c);
      if (copies) copies[nc] = CowCopy{pt[full], dst, r, 0};
      ++nc;
      ct[full] = dst;
      ch.n_blocks = full + 1;
      run_add_block(c, cs, full);
      ++c->cow_blocks;
      c->cow_rows += r;
    }
    ch.len = L;
    child_tid_out[i] = ch.tid;
    ++c->forks;
    const int32_t cur = c->cur_node[parent_tid[i]];
    if (cur >= 0) {   // the parent is tracked: close its node, open sibling and child nodes
      const int32_t sib = (int32_t)c->pnodes.size();
      c->pnodes.push_back({parent_tid[i], L, -1, -1, -1});
      c->pnodes.push_back({ch.tid, L + 1, -1, -1, -1});
      c->pnodes[cur].end = L;
      c->pnodes[cur].next_sibling = sib;
      c->pnodes[cur].first_child = sib + 1;
      c->cur_node[parent_tid[i]] = sib;
      c->cur_node[ch.tid] = sib + 1;
    }
  }
  if (n) ++c->struct_epoch;
  ++c->book_seq;
  if (nc && !c->host_only) {
    char* d_stage = c->ws(c->lay.stage);
    apar_status rc = send(c, stg, d_stage, (size_t)nc * sizeof(CowCopy), st);
    if (rc) return rc;
    for (int l = 0; l < c->num_layers; ++l) {
      APAR_CUDA(c, launch_cow_copy((char*)c->cfg.k_pool + l * c->layer_bytes,
                                   (char*)c->cfg.v_pool + l * c->layer_bytes,
                                   (const CowCopy*)d_stage, nc, c->cfg.num_kv_heads, st));
      ++c->kernels_total;
    }
  }
  return APAR_OK;
}

apar_status apar_append_kv(apar_ctx* c, int32_t n, const int32_t* tid, const int32_t* n_tok,
                           const void* k_new, const void* v_new, void* cuda_stream) {
  if (!c || n < 0 || (n > 0 && (!tid || ((!k_new || !v_new) && !c->host_only))))
    return APAR_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  for (int i = 0; i < n; ++i)
    if (slot_of(c, tid[i]) < 0) return APAR_ERR_BAD_THREAD;
  const uint32_t mk = next_mark(c);
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (c->mark[s] == mk || (n_tok && n_tok[i] < 0)) return APAR_ERR_INVALID_ARG;
    c->mark[s] = mk;
  }
  int64_t need = 0, rows = 0;
  for (int i = 0; i < n; ++i) {
    const ThreadRec& t = c->slots[slot_of(c, tid[i])];
    const int64_t cnt = n_tok ? n_tok[i] : 1;
    const int64_t after = (t.len + cnt + kBlock - 1) / kBlock;
    if (after > c->cfg.max_blocks_per_thread) return APAR_ERR_TABLE_FULL;
    need += after - t.n_blocks;
    rows += cnt;
  }
  if (need > (int64_t)c->free_stack.size()) return APAR_ERR_NO_BLOCKS;
  if (rows > INT32_MAX) return APAR_ERR_INVALID_ARG;
  // bookkeeping and slot list, streamed to the device in staging-sized pieces; calls that fit
  // leave their slots in the slot map so that the other layers can replay the scatter
  const bool keep = rows <= kSlotMapRows;
  c->last_append_rows = keep ? rows : -1;
  ++c->book_seq;
  ++c->mod_seq;
  const size_t cap_rows = c->lay.stage_cap / 4;
  Staging* stg = nullptr;
  int32_t* slots = nullptr;
  size_t filled = 0;
  int64_t first_row = 0;
  auto flush = [&]() -> apar_status {
    if (!filled) return APAR_OK;
    char* d_stage = keep ? c->ws(c->lay.slot_map) + (size_t)first_row * 4 : c->ws(c->lay.stage);
    apar_status rc = send(c, stg, d_stage, filled * 4, st);
    if (rc) return rc;
    APAR_CUDA(c, launch_append(c->cfg.k_pool, c->cfg.v_pool, k_new, v_new,
                               (const int32_t*)d_stage, first_row, (int)filled,
                               c->cfg.num_kv_heads, st));
    ++c->kernels_total;
    first_row += (int64_t)filled;
    filled = 0;
    stg = nullptr;
    return APAR_OK;
  };
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    ThreadRec& t = c->slots[s];
    int32_t* tab = c->row(s);
    const int cnt = n_tok ? n_tok[i] : 1;
    for (int k = 0; k < cnt; ++k) {
      const int32_t pos = t.len;
      if (pos % kBlock == 0) {
        // a thread without a private tail gains one: cached plans no longer describe it
        if (t.n_blocks == 0 || c->refcnt[tab[t.n_blocks - 1]] > 1) ++c->struct_epoch;
        run_add_block(c, s, t.n_blocks);
        tab[t.n_blocks++] = alloc_block(c);
      }
      if (c->host_only) {
        t.len = pos + 1;
        continue;
      }
      if (!stg) {
        apar_status rc = acquire(c, &stg);
        if (rc) return rc;   // APAR_ERR_CUDA: the context is unusable from here on (apar.h)
        slots = (int32_t*)stg->host;
      }
      slots[filled++] = tab[pos / kBlock] * kBlock + pos % kBlock;
      t.len = pos + 1;
      if (filled == cap_rows) {
        apar_status rc = flush();
        if (rc) return rc;
      }
    }
  }
  return flush();
}

// True while the cached step list still describes live threads whose device rows are current.
static bool step_list_current(const apar_ctx* c) {
  return c->step_valid && c->step_life == c->life_seq && c->step_mod == c->mod_seq;
}

apar_status apar_decode_step(apar_ctx* c, int32_t n, const int32_t* tid, const void* k_new,
                             const void* v_new, const void* q, void* out, float sm_scale,
                             void* cuda_stream) {
  if (!c || n < 0 || n > c->cfg.max_threads ||
      (n > 0 && (!tid || !k_new || !v_new || !q || !out)))
    return APAR_ERR_INVALID_ARG;
  if (c->host_only) return APAR_ERR_UNSUPPORTED;
  if (n == 0) return APAR_OK;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool same = step_list_current(c) && (int)c->step_tids.size() == n &&
                    memcmp(c->step_tids.data(), tid, (size_t)n * 4) == 0;
  // ---- every check comes before the first change
  if (!same) {
    c->tmp_slots.resize(n);
    for (int i = 0; i < n; ++i) {
      const int s = slot_of(c, tid[i]);
      if (s < 0) return APAR_ERR_BAD_THREAD;
      c->tmp_slots[i] = s;
    }
    const uint32_t mk = next_mark(c);
    for (int i = 0; i < n; ++i) {
      if (c->mark[c->tmp_slots[i]] == mk) return APAR_ERR_INVALID_ARG;
      c->mark[c->tmp_slots[i]] = mk;
    }
  }
  const int32_t* sl = same ? c->step_slots.data() : c->tmp_slots.data();
  int need = 0;
  for (int i = 0; i < n; ++i) {
    const int32_t len = c->slots[sl[i]].len;
    if ((len & (kBlock - 1)) == 0) {
      if (len / kBlock >= c->cfg.max_blocks_per_thread) return APAR_ERR_TABLE_FULL;
      ++need;
    }
  }
  if (need > (int)c->free_stack.size()) return APAR_ERR_NO_BLOCKS;
  if ((size_t)need * sizeof(int4) > c->lay.stage_cap) return APAR_ERR_WORKSPACE_TOO_SMALL;
  {
    // a step that has to use the staging buffers (new list, new blocks) cannot be captured
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    APAR_CUDA(c, cudaStreamIsCapturing(st, &cap));
    if (cap != cudaStreamCaptureStatusNone) {
      if (!same || need) return APAR_ERR_INVALID_ARG;
      int64_t attended = n;                       // chain lengths after this step
      for (int i = 0; i < n; ++i) attended += c->slots[sl[i]].len;
      if (!plan_reusable(c, n, tid, attended)) return APAR_ERR_INVALID_ARG;
    }
  }
  apar_status rc;
  c->last.attn_upload_bytes = (same ? 0 : (int64_t)n * 4) + (int64_t)need * sizeof(int4);
  if (!same) {
    // a new list: its table rows go to the device, and the device tables and lengths of its
    // threads are brought up to date once; from then on the step kernel keeps them current
    c->step_valid = false;
    c->step_slots.swap(c->tmp_slots);
    c->step_tids.assign(tid, tid + n);
    size_t done = 0;
    const size_t bytes = (size_t)n * 4;
    while (done < bytes) {
      Staging* s;
      rc = acquire(c, &s);
      if (rc) return rc;
      const size_t chunk = std::min(bytes - done, c->ring_bytes);
      memcpy(s->host, (const char*)c->step_slots.data() + done, chunk);
      rc = send(c, s, c->ws(c->lay.step_rows) + done, chunk, st);
      if (rc) return rc;
      done += chunk;
    }
    rc = sync_device_tables(c, c->step_slots.data(), n, st);
    if (rc) return rc;
    c->step_valid = true;
    c->step_life = c->life_seq;
    c->step_mod = c->mod_seq;
    sl = c->step_slots.data();
  }
  // ---- bookkeeping: only a thread that starts a new block needs more than a counter
  Staging* stg = nullptr;
  int4* pairs = nullptr;
  int np = 0;
  if (need) {
    rc = acquire(c, &stg);
    if (rc) return rc;
    pairs = (int4*)stg->host;
  }
  for (int i = 0; i < n; ++i) {
    ThreadRec& t = c->slots[sl[i]];
    if ((t.len & (kBlock - 1)) == 0) {
      int32_t* tab = c->row(sl[i]);
      // a thread without a private tail gains one: cached plans no longer describe it
      if (t.n_blocks == 0 || c->refcnt[tab[t.n_blocks - 1]] > 1) ++c->struct_epoch;
      const int32_t b = alloc_block(c);
      run_add_block(c, sl[i], t.n_blocks);
      pairs[np++] = make_int4(i, sl[i], t.n_blocks, b);
      tab[t.n_blocks++] = b;
      t.synced = t.n_blocks;
    }
    ++t.len;
    t.dev_len = t.len;
  }
  ++c->book_seq;
  c->last_append_rows = n;
  const void* d_pairs = nullptr;
  if (np) {
    if (stg->mapped) {
      d_pairs = stg->mapped;              // read once, straight from the pinned buffer
    } else {
      d_pairs = c->ws(c->lay.stage);
      rc = send(c, stg, c->ws(c->lay.stage), (size_t)np * sizeof(int4), st);
      if (rc) return rc;
    }
  }
  APAR_CUDA(c, launch_step_advance((int32_t*)c->ws(c->lay.tables), c->cfg.max_blocks_per_thread,
                                   (int32_t*)c->ws(c->lay.lens),
                                   (const int32_t*)c->ws(c->lay.step_rows), n, d_pairs, np,
                                   (int32_t*)c->ws(c->lay.slot_map), st));
  if (np && stg->mapped) {
    rc = send(c, stg, nullptr, 0, st);    // nothing to copy: only marks the buffer in flight
    if (rc) return rc;
  }
  APAR_CUDA(c, launch_append(c->cfg.k_pool, c->cfg.v_pool, k_new, v_new,
                             (const int32_t*)c->ws(c->lay.slot_map), 0, n, c->cfg.num_kv_heads,
                             st));
  c->kernels_total += 2;
  return run_attention(c, n, sl, tid, false, q, out, sm_scale, st, nullptr, true);
}

apar_status apar_steps_before_new_block(apar_ctx* c, int32_t* steps_out) {
  if (!c || !steps_out) return APAR_ERR_INVALID_ARG;
  if (!step_list_current(c)) return APAR_ERR_INVALID_ARG;
  int32_t steps = INT32_MAX;
  for (int32_t s : c->step_slots) {
    const int32_t r = c->slots[s].len & (kBlock - 1);
    steps = std::min(steps, r ? kBlock - r : 0);
  }
  *steps_out = steps;
  return APAR_OK;
}

apar_status apar_note_step_replay(apar_ctx* c) {
  if (!c) return APAR_ERR_INVALID_ARG;
  // the device-resident plan and step list must be the ones the replayed kernels were
  // captured with, and no thread may need a block (the captured step carries none)
  if (!step_list_current(c) || c->attn_book_seq != c->book_seq || c->plan.items.empty() ||
      c->plan_tids != c->step_tids)
    return APAR_ERR_INVALID_ARG;
  for (int32_t s : c->step_slots)
    if ((c->slots[s].len & (kBlock - 1)) == 0) return APAR_ERR_INVALID_ARG;
  for (int32_t s : c->step_slots) {
    ThreadRec& t = c->slots[s];
    ++t.len;
    t.dev_len = t.len;
  }
  const int64_t n = (int64_t)c->step_slots.size();
  c->last.attn_attended_tokens += n;
  c->last.attn_unique_tokens += n;
  return APAR_OK;
}

apar_status apar_tree_decode_attention(apar_ctx* c, int32_t n, const int32_t* tid, const void* q,
                                       void* out, float sm_scale, void* cuda_stream) {
  if (!c || n < 0 || n > c->cfg.max_threads || (n > 0 && (!tid || !q || !out)))
    return APAR_ERR_INVALID_ARG;
  if (c->host_only) return APAR_ERR_UNSUPPORTED;
  if (n == 0) return APAR_OK;
  std::vector<int32_t> qslots(n);
  const uint32_t mk = next_mark(c);
  bool dups = false;
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (s < 0) return APAR_ERR_BAD_THREAD;
    qslots[i] = s;
  }
  for (int i = 0; i < n; ++i) {
    if (c->slots[qslots[i]].len == 0) return APAR_ERR_EMPTY_CONTEXT;
    if (c->mark[qslots[i]] == mk) dups = true;
    c->mark[qslots[i]] = mk;
  }
  return run_attention(c, n, qslots.data(), tid, dups, q, out, sm_scale,
                       (cudaStream_t)cuda_stream);
}

apar_status apar_tree_prefix_attention(apar_ctx* c, int32_t n, const int32_t* tid,
                                       const int32_t* attend_len, const void* q, void* out,
                                       float sm_scale, void* cuda_stream) {
  if (!c || n < 0 || n > c->cfg.max_threads || (n > 0 && (!tid || !attend_len || !q || !out)))
    return APAR_ERR_INVALID_ARG;
  if (c->host_only) return APAR_ERR_UNSUPPORTED;
  if (n == 0) return APAR_OK;
  std::vector<int32_t> qslots(n);
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (s < 0) return APAR_ERR_BAD_THREAD;
    qslots[i] = s;
  }
  for (int i = 0; i < n; ++i) {
    if (attend_len[i] == 0) return APAR_ERR_EMPTY_CONTEXT;
    if (attend_len[i] < 0 || attend_len[i] > c->slots[qslots[i]].len) return APAR_ERR_INVALID_ARG;
  }
  return run_attention(c, n, qslots.data(), tid, true, q, out, sm_scale,
                       (cudaStream_t)cuda_stream, attend_len);
}

apar_status apar_tree_verify_attention(apar_ctx* c, int32_t n, const int32_t* tid,
                                       const int32_t* n_cand, const uint64_t* anc_mask,
                                       const void* q, void* out, float sm_scale,
                                       void* cuda_stream) {
  if (!c || n < 0 || (n > 0 && (!tid || !n_cand || !anc_mask || !q || !out)))
    return APAR_ERR_INVALID_ARG;
  if (c->host_only) return APAR_ERR_UNSUPPORTED;
  if (n == 0) return APAR_OK;
  int64_t total = 0;
  for (int i = 0; i < n; ++i) {
    if (slot_of(c, tid[i]) < 0) return APAR_ERR_BAD_THREAD;
    if (n_cand[i] < 1 || n_cand[i] > 64) return APAR_ERR_INVALID_ARG;
    total += n_cand[i];
  }
  if (total > c->cfg.max_threads) return APAR_ERR_INVALID_ARG;
  const uint32_t mk = next_mark(c);
  std::vector<int32_t> qslots((size_t)total), qlens((size_t)total);
  std::vector<VerifyDesc> descs((size_t)total);
  int64_t seen = 0, k0 = 0;
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (c->mark[s] == mk) return APAR_ERR_INVALID_ARG;          // a thread listed twice
    c->mark[s] = mk;
    const int32_t k = n_cand[i], len = c->slots[s].len;
    if (k > len) return APAR_ERR_INVALID_ARG;                   // candidates are appended rows
    const uint64_t valid = k == 64 ? ~0ull : ((1ull << k) - 1);
    for (int j = 0; j < k; ++j) {
      const uint64_t m = anc_mask[k0 + j];
      if ((m & ~valid) || !((m >> j) & 1ull)) return APAR_ERR_INVALID_ARG;
      qslots[k0 + j] = s;
      qlens[k0 + j] = len - k;
      descs[k0 + j] = VerifyDesc{s, len - k, k, -1, m, (int32_t)(k0 + j), 0};
      seen += __builtin_popcountll(m);
    }
    k0 += k;
  }
  apar_status rc = run_attention(c, (int)total, qslots.data(), nullptr, true, q, out, sm_scale,
                                 (cudaStream_t)cuda_stream, qlens.data(), false, &descs);
  if (rc == APAR_OK) {
    c->last.attn_attended_tokens += seen;
    c->last.attn_unique_tokens += total;
  }
  return rc;
}

apar_status apar_accept_candidates(apar_ctx* c, int32_t n, const int32_t* tid,
                                   const int32_t* n_cand, const int32_t* n_keep,
                                   const int32_t* keep_idx, void* cuda_stream) {
  if (!c || n < 0 || (n > 0 && (!tid || !n_cand || !n_keep))) return APAR_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  for (int i = 0; i < n; ++i)
    if (slot_of(c, tid[i]) < 0) return APAR_ERR_BAD_THREAD;
  const uint32_t mk = next_mark(c);
  int64_t n_moves = 0, n_groups = 0, kofs = 0;
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (c->mark[s] == mk) return APAR_ERR_INVALID_ARG;
    c->mark[s] = mk;
    const ThreadRec& t = c->slots[s];
    const int32_t k = n_cand[i], keep = n_keep[i];
    if (k < 1 || k > 64 || k > t.len || keep < 0 || keep > k || (keep > 0 && !keep_idx))
      return APAR_ERR_INVALID_ARG;
    int moved = 0;
    for (int j = 0; j < keep; ++j) {
      const int32_t x = keep_idx[kofs + j];
      if (x < j || x >= k || (j > 0 && x <= keep_idx[kofs + j - 1])) return APAR_ERR_INVALID_ARG;
      if (x != j) ++moved;
    }
    // rows are moved and blocks are given back inside the thread's own tail only
    const int32_t* tab = c->row(s);
    for (int b = (t.len - k) / kBlock; b < t.n_blocks; ++b)
      if (c->refcnt[tab[b]] != 1) return APAR_ERR_INVALID_ARG;
    n_moves += moved;
    if (moved) ++n_groups;
    kofs += keep;
  }
  const size_t bytes = (size_t)n_moves * sizeof(RowMove) + (size_t)(n_groups + 1) * 4;
  if (bytes > c->lay.stage_cap) return APAR_ERR_WORKSPACE_TOO_SMALL;
  Staging* stg = nullptr;
  RowMove* moves = nullptr;
  int32_t* gbeg = nullptr;
  if (n_moves && !c->host_only) {
    apar_status rc = acquire(c, &stg);
    if (rc) return rc;
    moves = (RowMove*)stg->host;
    gbeg = (int32_t*)(stg->host + (size_t)n_moves * sizeof(RowMove));
  }
  int64_t nm = 0, ng = 0;
  kofs = 0;
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    ThreadRec& t = c->slots[s];
    int32_t* tab = c->row(s);
    const int32_t k = n_cand[i], keep = n_keep[i], base = t.len - k;
    bool opened = false;
    for (int j = 0; j < keep; ++j) {
      const int32_t x = keep_idx[kofs + j];
      if (x == j) continue;
      if (moves) {
        if (!opened) gbeg[ng++] = (int32_t)nm;
        const int32_t ps = base + x, pd = base + j;
        moves[nm] = RowMove{tab[ps / kBlock] * kBlock + ps % kBlock,
                            tab[pd / kBlock] * kBlock + pd % kBlock};
      }
      opened = true;
      ++nm;
    }
    kofs += keep;
    // the thread ends after its last kept row; blocks past that go back to the pool
    const int32_t new_len = base + keep, new_nb = (new_len + kBlock - 1) / kBlock;
    for (int b = new_nb; b < t.n_blocks; ++b) {
      c->refcnt[tab[b]] = 0;
      c->free_stack.push_back(tab[b]);
    }
    std::vector<BlockRun>& rs = c->runs[s];
    const int32_t open_gid = c->own_open[s] ? rs.back().gid : -1;
    while (!rs.empty() && rs.back().pos >= new_nb) {
      if (--c->gid_ref[rs.back().gid] == 0) c->gid_free.push_back(rs.back().gid);
      rs.pop_back();
    }
    if (!rs.empty() && rs.back().pos + rs.back().n > new_nb) rs.back().n = new_nb - rs.back().pos;
    c->own_open[s] = (open_gid >= 0 && !rs.empty() && rs.back().gid == open_gid) ? 1 : 0;
    t.len = new_len;
    t.n_blocks = new_nb;
    t.synced = std::min(t.synced, new_nb);
    t.dev_len = -1;
  }
  if (n) ++c->struct_epoch;
  ++c->book_seq;
  ++c->mod_seq;
  if (nm && moves) {
    gbeg[ng] = (int32_t)nm;
    char* d_stage = c->ws(c->lay.stage);
    apar_status rc = send(c, stg, d_stage, bytes, st);
    if (rc) return rc;
    for (int l = 0; l < c->num_layers; ++l) {
      APAR_CUDA(c, launch_row_moves((char*)c->cfg.k_pool + l * c->layer_bytes,
                                    (char*)c->cfg.v_pool + l * c->layer_bytes,
                                    (const RowMove*)d_stage,
                                    (const int32_t*)(d_stage + (size_t)n_moves * sizeof(RowMove)),
                                    (int)ng, c->cfg.num_kv_heads, st));
      ++c->kernels_total;
    }
  }
  return APAR_OK;
}

apar_status apar_tree_prefill_attention(apar_ctx* c, int32_t layer, int32_t n,
                                        const int32_t* tid, const int32_t* q_begin,
                                        const int32_t* q_count, const void* q, void* out,
                                        float sm_scale, void* cuda_stream) {
  if (!c || n < 0 || layer < 0 || layer >= c->num_layers ||
      (n > 0 && (!tid || !q_begin || !q_count || !q || !out)))
    return APAR_ERR_INVALID_ARG;
  if (c->host_only) return APAR_ERR_UNSUPPORTED;
  if (n == 0) return APAR_OK;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  std::vector<int32_t> seg_slot(n);
  int64_t total_q = 0, attended = 0;
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (s < 0) return APAR_ERR_BAD_THREAD;
    if (q_begin[i] < 0 || q_count[i] < 1 ||
        (int64_t)q_begin[i] + q_count[i] > c->slots[s].len)
      return APAR_ERR_INVALID_ARG;
    seg_slot[i] = s;
    total_q += q_count[i];
    attended += (int64_t)q_count[i] * q_begin[i] + (int64_t)q_count[i] * (q_count[i] + 1) / 2;
  }
  if (total_q > INT32_MAX) return APAR_ERR_INVALID_ARG;
  apar_status rc = sync_device_tables(c, seg_slot.data(), n, st);
  if (rc) return rc;
  c->attn_book_seq = 0;                 // layer replays of a decode plan need a decode call

  // Work items: the queries of a segment in tiles of 256 rows (2 * (128 / group) tokens); a
  // tile reads the chain from its start to the tile's last token once, for all of its rows,
  // and every row stops at its own position (the mask is applied by the kernel).
  const int G = c->shape.group;
  const int per_tile = 2 * (128 / G);
  struct Tile { int32_t seg, first, count; };
  std::vector<Tile> tiles;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < q_count[i]; j += per_tile)
      tiles.push_back(Tile{i, j, std::min(per_tile, q_count[i] - j)});
  // Order: segments by how far they reach (longest first), the tiles of a segment together,
  // longest first.  The kernel walks this list once per kv head, so the CTAs that run at the
  // same time work on a few segments of one head and find their K and V in the L2 cache.
  std::vector<int32_t> seg_rank(n);
  {
    std::vector<int32_t> order(n);
    for (int i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) {
      return q_begin[x] + q_count[x] > q_begin[y] + q_count[y];
    });
    for (int i = 0; i < n; ++i) seg_rank[order[i]] = i;
  }
  std::stable_sort(tiles.begin(), tiles.end(), [&](const Tile& x, const Tile& y) {
    if (x.seg != y.seg) return seg_rank[x.seg] < seg_rank[y.seg];
    return x.first > y.first;
  });
  std::vector<int64_t> seg_qbase(n);
  {
    int64_t b = 0;
    for (int i = 0; i < n; ++i) { seg_qbase[i] = b; b += q_count[i]; }
  }
  AttnArgs a;
  a.q = q;
  a.out = out;
  a.k_pool = (const char*)c->cfg.k_pool + (size_t)layer * c->layer_bytes;
  a.v_pool = (const char*)c->cfg.v_pool + (size_t)layer * c->layer_bytes;
  a.d_tables = (const int32_t*)c->ws(c->lay.tables);
  a.d_lens = (const int32_t*)c->ws(c->lay.lens);
  // Every tile covers its rows' whole chains, so no partial results are written: the area
  // that holds them in decode calls (by far the largest part of the workspace) takes this
  // call's work items instead.
  const size_t area = (size_t)c->lay.slot_capacity * c->shape.num_q_heads * kDim * sizeof(float);
  const int64_t cap = std::min<int64_t>(c->prefill_batch, (int64_t)(area / sizeof(PrefillItem)));
  char* d_items = c->ws(c->lay.part_o);
  a.part_o = nullptr;
  a.part_ml = nullptr;
  a.shape = c->shape;
  a.scale_log2e = sm_scale * 1.4426950408889634f;
  a.tm_k = &c->tm_k[layer];
  a.tm_v = &c->tm_v[layer];
  a.d_error = (int*)c->ws(c->lay.err);
  a.num_sms = c->num_sms;
  a.d_ticket = (int*)c->ws(c->lay.ticket);
  CUtensorMap tm_q;
  if (make_query_tensor_map(q, total_q, c->shape.num_q_heads, G, &tm_q) != 0)
    return APAR_ERR_INVALID_ARG;        // (a query array that is not 16-byte aligned)

  auto upload = [&](const void* src, size_t bytes, char* dst) -> apar_status {
    size_t done = 0;
    while (done < bytes) {
      Staging* s;
      apar_status r = acquire(c, &s);
      if (r) return r;
      const size_t chunk = std::min(bytes - done, c->ring_bytes);
      memcpy(s->host, (const char*)src + done, chunk);
      r = send(c, s, dst + done, chunk, st);
      if (r) return r;
      done += chunk;
    }
    return APAR_OK;
  };
  std::vector<PrefillItem> items;
  int launches = 0;
  c->last.attn_work_items = 0;
  size_t t0 = 0;
  while (t0 < tiles.size()) {           // (one launch unless the list outgrows its area)
    const size_t t1 = (size_t)std::min<int64_t>((int64_t)tiles.size(), (int64_t)t0 + cap);
    items.clear();
    for (size_t i = t0; i < t1; ++i) {
      const Tile& t = tiles[i];
      items.push_back(PrefillItem{seg_slot[t.seg], (int32_t)(seg_qbase[t.seg] + t.first),
                                  q_begin[t.seg] + t.first, t.count});
    }
    rc = upload(items.data(), items.size() * sizeof(PrefillItem), d_items);
    if (rc) return rc;
    if (c->time_start && t0 == 0) APAR_CUDA(c, cudaEventRecord(c->time_start, st));
    APAR_CUDA(c, launch_attention_prefill(a, &tm_q, (const PrefillItem*)d_items, (int)items.size(),
                                          st));
    ++launches;
    c->last.attn_work_items += (int64_t)items.size();
    t0 = t1;
  }
  if (c->time_stop) APAR_CUDA(c, cudaEventRecord(c->time_stop, st));
  c->kernels_total += launches;
  c->last.attn_kernels = launches;
  c->last.attn_threads = total_q;
  c->last.attn_attended_tokens = attended;
  int64_t unique = 0;                   // rows of the pools that are read: per listed thread,
  {                                     // its chain up to the last query position
    const uint32_t mk = next_mark(c);
    std::vector<int32_t> reach(c->slots.size(), 0);
    for (int i = 0; i < n; ++i)
      reach[seg_slot[i]] = std::max(reach[seg_slot[i]], q_begin[i] + q_count[i]);
    for (int i = 0; i < n; ++i)
      if (c->mark[seg_slot[i]] != mk) {
        c->mark[seg_slot[i]] = mk;
        unique += reach[seg_slot[i]];
      }
  }
  c->last.attn_unique_tokens = unique;
  c->last.attn_partials = 0;
  c->last.attn_plan_reused = 0;
  c->last.attn_vec_items = 0;
  c->last.attn_mma_items = c->last.attn_work_items;
  return APAR_OK;
}

apar_status apar_append_kv_layer(apar_ctx* c, int32_t layer, const void* k_new, const void* v_new,
                                 void* cuda_stream) {
  if (!c || layer < 0 || layer >= c->num_layers || !k_new || !v_new) return APAR_ERR_INVALID_ARG;
  if (c->host_only) return APAR_ERR_UNSUPPORTED;
  if (c->last_append_rows < 0) return APAR_ERR_WORKSPACE_TOO_SMALL;
  if (c->last_append_rows == 0) return APAR_OK;
  APAR_CUDA(c, launch_append((char*)c->cfg.k_pool + layer * c->layer_bytes,
                             (char*)c->cfg.v_pool + layer * c->layer_bytes, k_new, v_new,
                             (const int32_t*)c->ws(c->lay.slot_map), 0, (int)c->last_append_rows,
                             c->cfg.num_kv_heads, (cudaStream_t)cuda_stream));
  ++c->kernels_total;
  return APAR_OK;
}

apar_status apar_tree_decode_attention_layer(apar_ctx* c, int32_t layer, const void* q, void* out,
                                             float sm_scale, void* cuda_stream) {
  if (!c || layer < 0 || layer >= c->num_layers || !q || !out) return APAR_ERR_INVALID_ARG;
  if (c->host_only) return APAR_ERR_UNSUPPORTED;
  // the device-resident plan, tables and lengths must still describe the pool
  if (c->attn_book_seq != c->book_seq || c->plan.items.empty()) return APAR_ERR_INVALID_ARG;
  int launches = 0;
  if (c->time_start) APAR_CUDA(c, cudaEventRecord(c->time_start, (cudaStream_t)cuda_stream));
  apar_status rc = launch_plan(c, layer, q, out, sm_scale, (cudaStream_t)cuda_stream, &launches);
  c->kernels_total += launches;
  if (rc == APAR_OK && c->time_stop)
    APAR_CUDA(c, cudaEventRecord(c->time_stop, (cudaStream_t)cuda_stream));
  return rc;
}

apar_status apar_release(apar_ctx* c, int32_t n, const int32_t* tid) {
  if (!c || n < 0 || (n > 0 && !tid)) return APAR_ERR_INVALID_ARG;
  const uint32_t mk = next_mark(c);
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (s < 0 || c->mark[s] == mk) return APAR_ERR_BAD_THREAD;
    c->mark[s] = mk;
  }
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    ThreadRec& t = c->slots[s];
    const int32_t* tab = c->row(s);
    for (int b = 0; b < t.n_blocks; ++b)
      if (--c->refcnt[tab[b]] == 0) c->free_stack.push_back(tab[b]);
    if (c->cur_node[tid[i]] >= 0) c->pnodes[c->cur_node[tid[i]]].end = t.len;
    run_release(c, s);
    c->tid_slot[tid[i]] = -1;
    t = ThreadRec();
    c->free_slots.push_back(s);
    --c->live;
  }
  if (n) ++c->struct_epoch;
  ++c->book_seq;
  ++c->life_seq;
  return APAR_OK;
}

apar_status apar_tree_decode_attention_tables(const apar_config* cfg, int32_t n,
                                              const int32_t* block_tables, const int32_t* ctx_lens,
                                              const void* q, void* out, float sm_scale,
                                              void* cuda_stream) {
  if (!cfg || n < 0 || (n > 0 && (!block_tables || !ctx_lens || !q || !out)))
    return APAR_ERR_INVALID_ARG;
  if (!supported(cfg)) return APAR_ERR_UNSUPPORTED;
  if (n > cfg->max_threads) return APAR_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (ctx_lens[i] < 0) return APAR_ERR_INVALID_ARG;
    if (ctx_lens[i] == 0) return APAR_ERR_EMPTY_CONTEXT;
    const int nb = (ctx_lens[i] + kBlock - 1) / kBlock;
    if (nb > cfg->max_blocks_per_thread) return APAR_ERR_INVALID_ARG;
    for (int b = 0; b < nb; ++b) {
      const int32_t id = block_tables[(size_t)i * cfg->max_blocks_per_thread + b];
      if (id < 0 || id >= cfg->num_blocks) return APAR_ERR_INVALID_ARG;
    }
  }
  if (n == 0) return APAR_OK;
  apar_ctx* c = nullptr;
  apar_status rc = create_impl(cfg, true, false, &c);
  if (rc) return rc;
  std::vector<int32_t> qslots(n);
  for (int i = 0; i < n; ++i) {
    ThreadRec& t = c->slots[i];
    t.tid = i;
    t.len = ctx_lens[i];
    t.n_blocks = (t.len + kBlock - 1) / kBlock;
    memcpy(c->row(i), block_tables + (size_t)i * cfg->max_blocks_per_thread,
           (size_t)t.n_blocks * 4);
    qslots[i] = i;
  }
  rc = run_attention(c, n, qslots.data(), nullptr, false, q, out, sm_scale,
                     (cudaStream_t)cuda_stream);
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess && rc == APAR_OK)
    rc = APAR_ERR_CUDA;
  apar_destroy(c);
  return rc;
}

apar_status apar_paragraph_root(apar_ctx* c, int32_t tid) {
  if (!c) return APAR_ERR_INVALID_ARG;
  const int s = slot_of(c, tid);
  if (s < 0) return APAR_ERR_BAD_THREAD;
  if (c->cur_node[tid] >= 0) return APAR_ERR_INVALID_ARG;   // already part of a tree
  c->root_node[tid] = c->cur_node[tid] = (int32_t)c->pnodes.size();
  c->pnodes.push_back({tid, c->slots[s].len, -1, -1, -1});
  return APAR_OK;
}

apar_status apar_restore(apar_ctx* c, int32_t root_tid, int32_t* slices, int32_t cap, int32_t* n) {
  if (!c || !n || cap < 0 || (cap > 0 && !slices)) return APAR_ERR_INVALID_ARG;
  if (root_tid < 0 || root_tid >= (int32_t)c->root_node.size() || c->root_node[root_tid] < 0)
    return APAR_ERR_BAD_THREAD;
  std::vector<int32_t> stack{c->root_node[root_tid]};
  int32_t count = 0;
  while (!stack.empty()) {
    const apar_ctx::PNodeRec& nd = c->pnodes[stack.back()];
    stack.pop_back();
    int32_t end = nd.end;
    if (end < 0) {                       // open: the thread is alive, the node runs to its end
      const int s = slot_of(c, nd.tid);
      end = s >= 0 ? c->slots[s].len : nd.start;
    }
    if (count < cap) {
      slices[3 * count] = nd.tid;
      slices[3 * count + 1] = nd.start;
      slices[3 * count + 2] = end;
    }
    ++count;
    if (nd.next_sibling >= 0) stack.push_back(nd.next_sibling);   // visited after the child
    if (nd.first_child >= 0) stack.push_back(nd.first_child);
  }
  *n = count;
  return APAR_OK;
}

apar_status apar_get_thread(apar_ctx* c, int32_t tid, int32_t* len, int32_t* n_blocks,
                            int32_t* blocks, int32_t cap) {
  if (!c) return APAR_ERR_INVALID_ARG;
  const int s = slot_of(c, tid);
  if (s < 0) return APAR_ERR_BAD_THREAD;
  const ThreadRec& t = c->slots[s];
  if (len) *len = t.len;
  if (n_blocks) *n_blocks = t.n_blocks;
  if (blocks) memcpy(blocks, c->row(s), (size_t)std::max(0, std::min(cap, t.n_blocks)) * 4);
  return APAR_OK;
}

apar_status apar_get_refcounts(apar_ctx* c, int32_t* refcnt) {
  if (!c || !refcnt) return APAR_ERR_INVALID_ARG;
  memcpy(refcnt, c->refcnt.data(), c->refcnt.size() * 4);
  return APAR_OK;
}

apar_status apar_get_free_list(apar_ctx* c, int32_t* ids, int32_t cap, int32_t* n) {
  if (!c || !n || cap < 0 || (cap > 0 && !ids)) return APAR_ERR_INVALID_ARG;
  const int32_t total = (int32_t)c->free_stack.size();
  *n = total;
  for (int i = 0; i < std::min(cap, total); ++i) ids[i] = c->free_stack[total - 1 - i];
  return APAR_OK;
}

apar_status apar_get_stats(apar_ctx* c, apar_stats* out) {
  if (!c || !out) return APAR_ERR_INVALID_ARG;
  *out = c->last;
  out->live_threads = c->live;
  out->free_blocks = (int64_t)c->free_stack.size();
  out->used_blocks = c->cfg.num_blocks - out->free_blocks;
  out->forks = c->forks;
  out->cow_blocks = c->cow_blocks;
  out->cow_rows = c->cow_rows;
  out->kernels_total = c->kernels_total;
  out->peak_used_blocks = c->peak_used;
  int32_t flag = 0;   // synchronises with the device: introspection only
  if (!c->host_only && cudaMemcpy(&flag, c->ws(c->lay.err), 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    c->last_cuda = (int32_t)cudaGetLastError();
    return APAR_ERR_CUDA;
  }
  out->device_wait_timeouts = flag;
  return APAR_OK;
}

apar_status apar_check_invariants(apar_ctx* c) {
  if (!c) return APAR_ERR_INVALID_ARG;
  const int32_t nb = c->cfg.num_blocks;
  std::vector<int32_t> count(nb, 0);
  int64_t live = 0;
  for (size_t s = 0; s < c->slots.size(); ++s) {
    const ThreadRec& t = c->slots[s];
    if (t.tid < 0) continue;
    ++live;
    if (slot_of(c, t.tid) != (int)s) return APAR_ERR_INVALID_ARG;
    if (t.n_blocks != (t.len + kBlock - 1) / kBlock) return APAR_ERR_INVALID_ARG;
    if (t.synced > t.n_blocks) return APAR_ERR_INVALID_ARG;
    for (int b = 0; b < t.n_blocks; ++b) {
      const int32_t id = c->row((int)s)[b];
      if (id < 0 || id >= nb) return APAR_ERR_INVALID_ARG;
      ++count[id];
    }
  }
  if (live != c->live) return APAR_ERR_INVALID_ARG;
  if (c->track_runs) {
    // group runs: they tile each table exactly; every thread that lists a group sees it at the
    // same positions with the same blocks; only a thread's own open group may be longer than
    // nobody else's view of it (nobody else lists it); reference counts add up
    struct Seen { int32_t pos, n, first_block, refs; };
    std::vector<Seen> seen(c->gid_ref.size(), Seen{-1, 0, 0, 0});
    for (size_t s = 0; s < c->slots.size(); ++s) {
      const ThreadRec& t = c->slots[s];
      const std::vector<BlockRun>& rs = c->runs[s];
      if (t.tid < 0) {
        if (!rs.empty() || c->own_open[s]) return APAR_ERR_INVALID_ARG;
        continue;
      }
      int32_t pos = 0;
      for (size_t k = 0; k < rs.size(); ++k) {
        const BlockRun& r = rs[k];
        if (r.pos != pos || r.n <= 0 || r.gid < 0 || r.gid >= (int32_t)seen.size())
          return APAR_ERR_INVALID_ARG;
        Seen& g = seen[r.gid];
        const int32_t* tab = c->row((int)s) + r.pos;
        if (g.refs == 0) {
          g = Seen{r.pos, r.n, tab[0], 1};
        } else {
          if (g.pos != r.pos || g.n != r.n || g.first_block != tab[0]) return APAR_ERR_INVALID_ARG;
          ++g.refs;
        }
        pos += r.n;
      }
      if (pos != t.n_blocks) return APAR_ERR_INVALID_ARG;
      if (c->own_open[s] && (rs.empty() || c->gid_ref[rs.back().gid] != 1))
        return APAR_ERR_INVALID_ARG;
      // a partial last block is never shared: it sits in the open group
      if (t.len % kBlock && !c->own_open[s]) return APAR_ERR_INVALID_ARG;
    }
    for (size_t g = 0; g < seen.size(); ++g)
      if (seen[g].refs != c->gid_ref[g]) return APAR_ERR_INVALID_ARG;
    for (int32_t g : c->gid_free)
      if (g < 0 || g >= (int32_t)seen.size() || c->gid_ref[g] != 0) return APAR_ERR_INVALID_ARG;
  }
  for (int32_t id : c->free_stack) {
    if (id < 0 || id >= nb || count[id] != 0) return APAR_ERR_INVALID_ARG;
    count[id] = -1;                                   // seen in the free list
  }
  for (int32_t b = 0; b < nb; ++b) {
    if (count[b] == -1) { if (c->refcnt[b] != 0) return APAR_ERR_INVALID_ARG; }
    else if (count[b] == 0 || count[b] != c->refcnt[b]) return APAR_ERR_INVALID_ARG;
  }
  return APAR_OK;
}

apar_status apar_debug_plan(int32_t num_blocks, int32_t num_q_heads, int32_t num_kv_heads,
                            int32_t n_threads, int32_t max_blocks, const int32_t* block_tables,
                            const int32_t* ctx_lens, int32_t mma_min_rows, int32_t fuse_final,
                            int32_t* items_out, int32_t cap_items, int32_t* users_out,
                            int32_t cap_users, int32_t* merges_out, int32_t cap_merges,
                            int64_t* counts_out) {
  if (num_blocks <= 0 || num_kv_heads <= 0 || num_q_heads <= 0 || num_q_heads % num_kv_heads ||
      n_threads <= 0 || max_blocks <= 0 || !block_tables || !ctx_lens || !counts_out ||
      cap_items < 0 || cap_users < 0 || cap_merges < 0 || (cap_items && !items_out) ||
      (cap_users && !users_out) || (cap_merges && !merges_out))
    return APAR_ERR_INVALID_ARG;
  if (num_q_heads / num_kv_heads > kMaxRowsPerItem) return APAR_ERR_UNSUPPORTED;
  std::vector<PlanQuery> pq(n_threads);
  for (int i = 0; i < n_threads; ++i) {
    const int32_t len = ctx_lens[i];
    if (len <= 0 || (len + kBlock - 1) / kBlock > max_blocks) return APAR_ERR_INVALID_ARG;
    const int32_t* tab = block_tables + (size_t)i * max_blocks;
    for (int b = 0; b < (len + kBlock - 1) / kBlock; ++b)
      if (tab[b] < 0 || tab[b] >= num_blocks) return APAR_ERR_INVALID_ARG;
    pq[i] = PlanQuery{tab, i, len};
  }
  Planner planner;
  planner.init(num_blocks, num_q_heads / num_kv_heads, num_kv_heads);
  Plan plan;
  if (!planner.build(pq.data(), n_threads,
                     std::max<int64_t>((int64_t)kSlotsPerThread * n_threads, kMinSlots), false,
                     mma_min_rows, fuse_final != 0, &plan))
    return APAR_ERR_WORKSPACE_TOO_SMALL;
  counts_out[0] = (int64_t)plan.items.size();
  counts_out[1] = (int64_t)plan.users.size();
  counts_out[2] = (int64_t)plan.merges.size();
  counts_out[3] = plan.total_slots;
  counts_out[4] = plan.unique_tokens;
  counts_out[5] = plan.attended_tokens;
  if ((int64_t)cap_items < counts_out[0] || (int64_t)cap_users < counts_out[1] ||
      (int64_t)cap_merges < counts_out[2])
    return APAR_ERR_WORKSPACE_TOO_SMALL;
  static_assert(sizeof(WorkItem) == 32 && sizeof(UserRef) == 8, "export layout");
  if (!plan.items.empty()) memcpy(items_out, plan.items.data(), plan.items.size() * sizeof(WorkItem));
  if (!plan.users.empty()) memcpy(users_out, plan.users.data(), plan.users.size() * sizeof(UserRef));
  for (size_t i = 0; i < plan.merges.size(); ++i) {
    merges_out[3 * i] = plan.merges[i].query;
    merges_out[3 * i + 1] = plan.merges[i].slot_begin;
    merges_out[3 * i + 2] = plan.merges[i].n;
  }
  return APAR_OK;
}

apar_status apar_debug_plan_threads(apar_ctx* c, int32_t n, const int32_t* tid, int32_t by_groups,
                                    int32_t mma_min_rows, int32_t fuse_final, int32_t* items_out,
                                    int32_t cap_items, int32_t* users_out, int32_t cap_users,
                                    int32_t* merges_out, int32_t cap_merges, int64_t* counts_out) {
  if (!c || n <= 0 || !tid || !counts_out || cap_items < 0 || cap_users < 0 || cap_merges < 0 ||
      (cap_items && !items_out) || (cap_users && !users_out) || (cap_merges && !merges_out))
    return APAR_ERR_INVALID_ARG;
  std::vector<PlanQuery> pq(n);
  const uint32_t mk = next_mark(c);
  for (int i = 0; i < n; ++i) {
    const int s = slot_of(c, tid[i]);
    if (s < 0) return APAR_ERR_BAD_THREAD;
    if (c->slots[s].len == 0) return APAR_ERR_EMPTY_CONTEXT;
    if (c->mark[s] == mk && by_groups) return APAR_ERR_INVALID_ARG;   // needs distinct threads
    c->mark[s] = mk;
    pq[i] = PlanQuery{c->row(s), s, c->slots[s].len};
    if (by_groups) {
      pq[i].runs = c->runs[s].data();
      pq[i].n_runs = (int32_t)c->runs[s].size();
    }
  }
  if (by_groups && !c->track_runs) return APAR_ERR_INVALID_ARG;
  Plan plan;
  if (!c->planner.build(pq.data(), n, c->lay.slot_capacity, false, mma_min_rows, fuse_final != 0,
                        &plan, by_groups != 0))
    return APAR_ERR_WORKSPACE_TOO_SMALL;
  c->plan_epoch = 0;            // the planner's scratch was reused: drop the cached plan
  counts_out[0] = (int64_t)plan.items.size();
  counts_out[1] = (int64_t)plan.users.size();
  counts_out[2] = (int64_t)plan.merges.size();
  counts_out[3] = plan.total_slots;
  counts_out[4] = plan.unique_tokens;
  counts_out[5] = plan.attended_tokens;
  if ((int64_t)cap_items < counts_out[0] || (int64_t)cap_users < counts_out[1] ||
      (int64_t)cap_merges < counts_out[2])
    return APAR_ERR_WORKSPACE_TOO_SMALL;
  if (!plan.items.empty()) memcpy(items_out, plan.items.data(), plan.items.size() * sizeof(WorkItem));
  if (!plan.users.empty()) memcpy(users_out, plan.users.data(), plan.users.size() * sizeof(UserRef));
  for (size_t i = 0; i < plan.merges.size(); ++i) {
    merges_out[3 * i] = plan.merges[i].query;
    merges_out[3 * i + 1] = plan.merges[i].slot_begin;
    merges_out[3 * i + 2] = plan.merges[i].n;
  }
  return APAR_OK;
}

apar_status apar_stream_read(const void* src, size_t bytes, void* sink, void* stream) {
  if (!src || !sink || (reinterpret_cast<uintptr_t>(src) & 15) ||
      (reinterpret_cast<uintptr_t>(sink) & 7))
    return APAR_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return APAR_ERR_CUDA;
  return launch_stream_read(src, bytes, sink, sms, (cudaStream_t)stream) == cudaSuccess
             ? APAR_OK : APAR_ERR_CUDA;
}

apar_status apar_set_timing_events(apar_ctx* c, void* start, void* stop) {
  if (!c || (start == nullptr) != (stop == nullptr)) return APAR_ERR_INVALID_ARG;
  c->time_start = (cudaEvent_t)start;
  c->time_stop = (cudaEvent_t)stop;
  return APAR_OK;
}

int32_t apar_last_cuda_error(apar_ctx* c) { return c ? c->last_cuda : 0; }

const char* apar_status_string(apar_status s) {
  switch (s) {
    case APAR_OK: return "APAR_OK";
    case APAR_ERR_INVALID_ARG: return "APAR_ERR_INVALID_ARG";
    case APAR_ERR_BAD_THREAD: return "APAR_ERR_BAD_THREAD";
    case APAR_ERR_NO_BLOCKS: return "APAR_ERR_NO_BLOCKS";
    case APAR_ERR_NO_THREADS: return "APAR_ERR_NO_THREADS";
    case APAR_ERR_TABLE_FULL: return "APAR_ERR_TABLE_FULL";
    case APAR_ERR_EMPTY_CONTEXT: return "APAR_ERR_EMPTY_CONTEXT";
    case APAR_ERR_WORKSPACE_TOO_SMALL: return "APAR_ERR_WORKSPACE_TOO_SMALL";
    case APAR_ERR_CUDA: return "APAR_ERR_CUDA";
    case APAR_ERR_UNSUPPORTED: return "APAR_ERR_UNSUPPORTED";
    default: return "APAR_ERR_UNKNOWN";
  }
}

}  // extern "C"

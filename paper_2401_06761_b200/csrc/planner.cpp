// Host planner: turns the block tables of the queried threads into work items in which every
// physical block is read once for all queries that share it.
//
// Sharing only arises through fork (paper, Section 2.3: the child shares the parent's full
// blocks), so the sets of threads that hold a block are nested along a chain and a block id
// identifies the whole prefix before it.  The planner therefore needs no tree: it counts, per
// block id, how many queries list it, and cuts each query's table into runs of equal count.
// A run listed by several queries becomes one shared work item; runs are found again through
// the id of their first block.  A block that is ragged (not full) for some query is never
// shared: each query that lists it reads it on its own.
#include <algorithm>
#include <climits>
#include <cstring>

#include "apar_internal.h"

namespace apar {

void Planner::init(int num_blocks, int group, int num_kv_heads) {
  num_blocks_ = num_blocks;
  group_ = group;
  hint_kv_heads_ = num_kv_heads;
  epoch_ = 0;
  stamp_.assign(num_blocks, 0);
  cnt_.assign(num_blocks, 0);
  seg_of_.assign(num_blocks, -1);
  partial_.assign(num_blocks, 0);
}

static inline int64_t round_up16(int64_t x) { return (x + 15) / 16 * 16; }
constexpr int kMaxFoldedParts = 8;   // partial results a finishing item may fold by itself

void Planner::ensure_keys(size_t n) {
  if (stamp_.size() >= n) return;
  n = std::max(n, stamp_.size() * 2);
  stamp_.resize(n, 0);
  cnt_.resize(n, 0);
  seg_of_.resize(n, -1);
  partial_.resize(n, 0);
}

// Passes 1 and 2: how many queries list each key, then each query's table cut into runs of
// equal count (segments).  kRuns = false: a key is a block id and an entry one table position.
// kRuns = true: a key is a group id and an entry one BlockRun; the caller guarantees that no
// query is listed twice and every query attends its thread's whole chain, so the only ragged
// block of a query is the last one of its own, unshared group.
template <bool kRuns>
void Planner::find_segments(const PlanQuery* q, int n, bool open_tails, int64_t* unique_out,
                            int64_t* attended_out) {
  auto n_entries = [&](int i) {
    return kRuns ? q[i].n_runs : (q[i].len + kBlock - 1) / kBlock;
  };
  auto key_of = [&](int i, int e) { return kRuns ? q[i].runs[e].gid : q[i].table[e]; };
  auto pos_of = [&](int i, int e) { return kRuns ? q[i].runs[e].pos : e; };
  auto end_of = [&](int i, int e) { return kRuns ? q[i].runs[e].pos + q[i].runs[e].n : e + 1; };
  // ---- pass 1: how many queries list each key; which blocks are ragged for someone
  int64_t attended = 0;
  for (int i = 0; i < n; ++i) {
    const int ne = n_entries(i);
    attended += q[i].len;
    for (int e = 0; e < ne; ++e) {
      const int32_t b = key_of(i, e);
      if (kRuns) ensure_keys((size_t)b + 1);
      if (stamp_[b] != epoch_) {
        stamp_[b] = epoch_;
        cnt_[b] = 0;
        partial_[b] = 0;
        seg_of_[b] = -1;
      }
      ++cnt_[b];
    }
    if (!kRuns && q[i].len % kBlock) partial_[q[i].table[ne - 1]] = 1;
  }
  // ---- pass 2: runs -> segments; a query's SegUser entries are contiguous, in chain order
  segs_.clear();
  seg_users_.clear();
  qbeg_.assign(n + 1, 0);
  int64_t unique = 0;
  for (int i = 0; i < n; ++i) {
    qbeg_[i] = (int32_t)seg_users_.size();
    const int32_t len = q[i].len, nb = (len + kBlock - 1) / kBlock;
    const int ne = n_entries(i);
    int e0 = 0;
    while (e0 < ne) {
      const int32_t b0 = key_of(i, e0);
      const bool priv0 = partial_[b0] || cnt_[b0] == 1;
      const int32_t key0 = priv0 ? 0 : cnt_[b0];
      int e1 = e0 + 1;
      while (e1 < ne) {
        const int32_t b = key_of(i, e1);
        const int32_t key = (partial_[b] || cnt_[b] == 1) ? 0 : cnt_[b];
        if (key != key0) break;
        ++e1;
      }
      const int32_t p0 = pos_of(i, e0), p1 = end_of(i, e1 - 1);
      const int32_t t0 = p0 * kBlock, t1 = std::min(p1 * kBlock, len);
      int32_t s = -1;
      if (!priv0) {
        s = seg_of_[b0];
        // tables that do not come from forks could disagree on where the run ends
        if (s >= 0 && (segs_[s].n_blocks != p1 - p0 || segs_[s].tok_begin != t0)) s = -1;
      }
      if (s < 0) {
        Seg g;
        g.table_row = q[i].table_row;
        g.tok_begin = t0;
        g.tok_end = t1;
        g.n_blocks = p1 - p0;
        g.n_users = 0;
        g.user_off = 0;
        g.priv = priv0;
        g.open = (priv0 && p1 == nb && open_tails) ? 1 : 0;
        s = (int32_t)segs_.size();
        segs_.push_back(g);
        if (!priv0 && seg_of_[b0] < 0) seg_of_[b0] = s;
        unique += t1 - t0;
      }
      ++segs_[s].n_users;
      seg_users_.push_back(SegUser{s, i, 0});
      e0 = e1;
    }
  }
  qbeg_[n] = (int32_t)seg_users_.size();
  *unique_out = unique;
  *attended_out = attended;
}

bool Planner::build(const PlanQuery* q, int n, int64_t slot_capacity, bool open_tails,
                    int mma_min_rows, bool fuse_final, Plan* out, bool by_runs) {
  if (++epoch_ == 0) {
    std::fill(stamp_.begin(), stamp_.end(), 0u);
    epoch_ = 1;
  }
  int64_t unique = 0, attended = 0;
  if (by_runs) find_segments<true>(q, n, open_tails, &unique, &attended);
  else find_segments<false>(q, n, open_tails, &unique, &attended);

  // ---- chunk length: enough items to fill the machine, never below 128 tokens
  const int64_t kInf = (int64_t)1 << 40;
  int64_t chunk = std::max<int64_t>(128, round_up16(unique * hint_kv_heads_ / (num_sms_ * 8)));
  // `chunk` is sized for the kernels that keep a CTA's loads in flight through TMA rings.  The
  // single-row kernel has no such staging and needs several CTAs per SM to cover the latency:
  // when its runs, dealt out four kv heads to a CTA, would give fewer than four CTAs per SM,
  // they are cut finer (up to eight times).  This only happens with a few very long threads.
  const int max_users = std::max(1, kMaxRowsPerItem / group_);
  auto single_row = [&](const Seg& g) {
    return std::min(g.n_users, max_users) * group_ < mma_min_rows;
  };
  int64_t vec_div = 1;
  {
    int64_t vec_chunks = 0;
    for (const Seg& g : segs_)
      if (single_row(g))
        vec_chunks += (g.tok_end - g.tok_begin + chunk - 1) / chunk * ((g.n_users + max_users - 1) / max_users);
    const int64_t head_groups = (hint_kv_heads_ + 3) / 4;
    while (vec_chunks > 0 && vec_div < 8 && vec_chunks * vec_div * head_groups < 4 * num_sms_) vec_div *= 2;
  }
  auto seg_chunk = [&](const Seg& g) -> int64_t {
    if (chunk >= kInf) return kInf;
    if (vec_div == 1 || !single_row(g)) return chunk;
    return std::max<int64_t>(128, round_up16(chunk / vec_div));
  };
  n_parts_.assign(n, 0);
  int64_t total_slots = 0;
  for (int attempt = 0;; ++attempt) {
    total_slots = 0;
    for (int i = 0; i < n; ++i) {
      int32_t ord = 0;
      for (int k = qbeg_[i]; k < qbeg_[i + 1]; ++k) {
        const Seg& g = segs_[seg_users_[k].seg];
        const int64_t ck = seg_chunk(g);
        seg_users_[k].ord = ord;
        ord += (int32_t)((g.tok_end - g.tok_begin + ck - 1) / ck);
      }
      ord += q[i].extra_parts;        // results the caller computes itself (see PlanQuery)
      n_parts_[i] = ord;
      if (ord >= 2) total_slots += ord;
    }
    if (total_slots <= slot_capacity) break;
    if (chunk >= kInf) return false;
    chunk = attempt >= 3 ? kInf : chunk * 4;
  }

  // ---- partial slots and merges
  out->merges.clear();
  out->extra_slot.assign(n, -1);
  part_off_.assign(n, -1);
  int32_t off = 0;
  fused_.assign(n, 0);
  for (int i = 0; i < n; ++i) {
    if (n_parts_[i] >= 2) {
      part_off_[i] = off;
      // the chain ends in a private run: its last item can finish the query on its own
      const Seg& last = segs_[seg_users_[qbeg_[i + 1] - 1].seg];
      // (folding is serial work of one CTA: chains cut into many pieces go to the merge kernel)
      if (fuse_final && last.priv && group_ <= 16 && n_parts_[i] - 1 <= kMaxFoldedParts &&
          q[i].extra_parts == 0)
        fused_[i] = 1;
      // the caller's own partial result takes the last slot of the query
      if (q[i].extra_parts) out->extra_slot[i] = off + n_parts_[i] - 1;
      if (!fused_[i]) out->merges.push_back(MergeRef{i, off, n_parts_[i], 0});
      off += n_parts_[i];
    }
  }
  // ---- users grouped by segment
  int32_t uo = 0;
  for (Seg& g : segs_) {
    g.user_off = uo;
    uo += g.n_users;
    g.n_users = 0;
  }
  out->users.resize(seg_users_.size());
  for (const SegUser& su : seg_users_) {
    Seg& g = segs_[su.seg];
    out->users[g.user_off + g.n_users++] =
        UserRef{su.query, part_off_[su.query] >= 0 ? part_off_[su.query] + su.ord : -1};
  }
  // ---- items
  vec_items_.clear();
  vec_final_.clear();
  mma1_final_.clear();
  for (auto& v : mma_items_) v.clear();
  for (const Seg& g : segs_) {
    const int64_t chunk = seg_chunk(g);        // this run's own chunk length
    const int32_t n_chunks = (int32_t)((g.tok_end - g.tok_begin + chunk - 1) / chunk);
    for (int u0 = 0; u0 < g.n_users; u0 += max_users) {
      const int nu = std::min(max_users, g.n_users - u0);
      for (int c = 0; c < n_chunks; ++c) {
        WorkItem it;
        it.table_row = g.table_row;
        it.tok_begin = g.tok_begin + (int32_t)(c * chunk);
        it.tok_end = (int32_t)std::min<int64_t>(g.tok_end, it.tok_begin + chunk);
        // An open tail keeps its planned token count, sign-folded, for sorting; the kernels
        // only test the sign and then read the device length array.
        if (g.open && c == n_chunks - 1) it.tok_end = -(it.tok_end - it.tok_begin) - 1;
        it.user_begin = g.user_off + u0;
        it.n_users = nu;
        it.slot_add = c;
        it.fin_n = it.fin_begin = 0;
        const int rows = nu * group_;
        const bool to_mma = rows >= mma_min_rows;
        if (g.priv && g.n_users == 1 && c == n_chunks - 1) {
          // private runs hold exactly one query; is this the end of a fused query's chain?
          const int qi = out->users[g.user_off].query;
          if (fused_[qi] && g.tok_end == q[qi].len) {
            // which of the folded parts come from single-tile items (same kernel class as a
            // multi-row finishing item, hence possibly the same launch): bit = part ordinal
            uint32_t same_class = 0;
            for (int k = qbeg_[qi]; k < qbeg_[qi + 1]; ++k) {
              const Seg& sg = segs_[seg_users_[k].seg];
              int nu_k = sg.n_users;
              if (sg.n_users > max_users) {           // wide run: the user group that holds qi
                int j = 0;
                while (j < sg.n_users && out->users[sg.user_off + j].query != qi) ++j;
                nu_k = std::min(max_users, sg.n_users - j / max_users * max_users);
              }
              const int rows_k = nu_k * group_;
              if (rows_k < mma_min_rows || rows_k > 16) continue;
              const int32_t nck = (int32_t)((sg.tok_end - sg.tok_begin + seg_chunk(sg) - 1) /
                                            seg_chunk(sg));
              for (int x = 0; x < nck; ++x) {
                const int part = seg_users_[k].ord + x;
                if (part < n_parts_[qi] - 1) same_class |= 1u << part;
              }
            }
            it.fin_n = (n_parts_[qi] - 1) | (int32_t)(same_class << 8);
            it.fin_begin = part_off_[qi];
            (to_mma ? mma1_final_ : vec_final_).push_back(it);
            continue;
          }
        }
        (to_mma ? mma_items_[(rows + 15) / 16 - 1] : vec_items_).push_back(it);
      }
    }
  }
  auto cost = [](const WorkItem& w) {
    return w.tok_end < 0 ? -w.tok_end - 1 : w.tok_end - w.tok_begin;
  };
  auto by_cost = [&](const WorkItem& a, const WorkItem& b) { return cost(a) > cost(b); };
  std::stable_sort(vec_items_.begin(), vec_items_.end(), by_cost);
  std::stable_sort(vec_final_.begin(), vec_final_.end(), by_cost);
  std::stable_sort(mma1_final_.begin(), mma1_final_.end(), by_cost);
  out->n_vec_final = (int32_t)vec_final_.size();
  out->n_mma1_final = (int32_t)mma1_final_.size();
  out->n_vec = (int32_t)(vec_items_.size() + vec_final_.size());
  out->n_mma = 0;
  out->items.clear();
  out->items.insert(out->items.end(), vec_items_.begin(), vec_items_.end());
  out->items.insert(out->items.end(), vec_final_.begin(), vec_final_.end());
  for (int k = 3; k >= 0; --k) {          // widest items first
    std::stable_sort(mma_items_[k].begin(), mma_items_[k].end(), by_cost);
    out->n_mma_tiles[k] = (int32_t)mma_items_[k].size() + (k == 0 ? out->n_mma1_final : 0);
    out->n_mma += out->n_mma_tiles[k];
    out->items.insert(out->items.end(), mma_items_[k].begin(), mma_items_[k].end());
  }
  out->items.insert(out->items.end(), mma1_final_.begin(), mma1_final_.end());
  out->total_slots = total_slots;
  out->unique_tokens = unique;
  out->attended_tokens = attended;
  out->chunk_tokens = (int32_t)std::min<int64_t>(chunk, INT32_MAX);
  return true;
}

}  // namespace apar

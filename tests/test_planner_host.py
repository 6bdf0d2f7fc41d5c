"""Host logic without a GPU: the library's planner, called through its host-only entry point,
on block tables produced by the independent pool model.  The plan must read every token a
query attends exactly once for that query, every physical block at most once in all, and its
partial-result bookkeeping (slots, finishing items, merges) must be consistent."""
import random

import numpy as np
import pytest

from oracle import BlockModel
from paper_2401_06761_b200 import binding as B

BS = 16


def random_forest(seed, n_roots, steps, num_blocks=4000, max_threads=400, max_blocks=120):
    rnd = random.Random(seed)
    m = BlockModel(num_blocks, BS, max_threads, max_blocks)
    live = m.new_threads(n_roots)
    m.append(live, [rnd.randrange(1, 400) for _ in live])
    for _ in range(steps):
        op = rnd.random()
        if op < 0.35:
            parents = [rnd.choice(live) for _ in range(rnd.randrange(1, 6))]
            kids, _ = m.fork(parents)
            live += kids
        elif op < 0.9:
            sub = rnd.sample(live, rnd.randrange(1, len(live) + 1))
            m.append(sub, [rnd.randrange(0, 70) for _ in sub])
        elif len(live) > 2:
            t = rnd.choice(live)
            m.release([t])
            live.remove(t)
    live = [t for t in live if m.lens[t] > 0]
    return m, live


def tables_of(m, threads):
    mb = max(len(m.tables[t]) for t in threads)
    tab = np.zeros((len(threads), mb), dtype=np.int32)
    for i, t in enumerate(threads):
        tab[i, :len(m.tables[t])] = m.tables[t]
    return tab, np.array([m.lens[t] for t in threads], dtype=np.int32)


def check_plan(m, threads, hq, hkv, mma_min_rows, fuse_final):
    tab, lens = tables_of(m, threads)
    items, users, merges, c = B.apar_debug_plan(m.num_blocks, hq, hkv, tab, lens, mma_min_rows,
                                                fuse_final)
    n = len(threads)
    assert c["attended_tokens"] == int(lens.sum()) == m.attended_tokens(threads)
    assert c["unique_tokens"] == m.unique_tokens(threads)
    per_query = [[] for _ in range(n)]          # (tok_begin, tok_end, partial row or -1, item)
    tokens = 0
    for k, (row, t0, t1, ub, nu, slot_add, fin_n, fin_begin) in enumerate(items.tolist()):
        assert 0 <= row < n and t0 % BS == 0 and 0 <= t0 < t1 <= lens[row] and nu >= 1
        assert nu * (hq // hkv) <= 64
        tokens += t1 - t0
        blocks = tab[row, t0 // BS:(t1 + BS - 1) // BS].tolist()
        for q, slot in users[ub:ub + nu].tolist():
            assert 0 <= q < n
            assert tab[q, t0 // BS:(t1 + BS - 1) // BS].tolist() == blocks      # same physical run
            assert t1 <= lens[q] and (t1 == lens[q] or t1 % BS == 0)
            if t1 % BS:                       # a ragged end is read by its own thread only
                assert nu == 1
            per_query[q].append((t0, t1, slot + slot_add if slot >= 0 else -1, k))
        if fin_n:
            assert nu == 1 and fuse_final
    # unique reads: a block is read by one item, or (sibling sets of more than 64 rows are cut
    # into groups of users) by the groups of one wide run
    readers = {}
    for k, (row, t0, t1, ub, nu, *_rest) in enumerate(items.tolist()):
        for j, b in enumerate(tab[row, t0 // BS:(t1 + BS - 1) // BS].tolist()):
            readers.setdefault(b, []).append((nu, k))
    group = hq // hkv
    max_users = max(1, 64 // group)
    extra = 0
    for b, rs in readers.items():
        if len(rs) > 1:                       # only when more than 64 rows share the block
            assert sum(nu for nu, _ in rs) > max_users
            assert all(nu == max_users for nu, _ in sorted(rs, reverse=True)[:-1])
            extra += len(rs) - 1
    if extra == 0:
        assert tokens == c["unique_tokens"]
    merged = {q: (s, k) for q, s, k in merges.tolist()}
    assert len(merged) == len(merges)
    rows_used = set()
    for q in range(n):
        parts = sorted(per_query[q])
        assert parts[0][0] == 0 and parts[-1][1] == lens[q]
        for (a0, a1, _, _), (b0, b1, _, _) in zip(parts, parts[1:]):
            assert a1 == b0                                   # contiguous, no overlap
        if len(parts) == 1:
            assert parts[0][2] == -1 and q not in merged
            continue
        slots = [p[2] for p in parts]
        assert slots == list(range(slots[0], slots[0] + len(parts)))   # chain order
        assert not (set(slots) & rows_used)
        rows_used |= set(slots)
        last = items[parts[-1][3]]
        if last[6]:                           # the chain's last item finishes the query
            assert last[6] & 0xff == len(parts) - 1 and last[7] == slots[0] and q not in merged
            # bits 8..: the folded parts that come from single-tile items (2..16 rows), which
            # may share a kernel launch with the finishing item
            g = hq // hkv
            want = sum(1 << j for j, p in enumerate(parts[:-1])
                       if mma_min_rows <= items[p[3]][4] * g <= 16)
            assert last[6] >> 8 == want
        else:
            assert merged[q] == (slots[0], len(parts))
        for p in parts[:-1]:
            assert items[p[3]][6] == 0
    assert not rows_used or max(rows_used) < c["partial_slots"]
    return c


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4), (64, 8), (32, 8)])
@pytest.mark.parametrize("mma_min_rows,fuse_final", [(2, True), (2, False), (1 << 30, False)])
def test_random_forests(hq, hkv, mma_min_rows, fuse_final):
    for seed in range(6):
        m, live = random_forest(100 * hq + seed, n_roots=1 + seed % 3, steps=60)
        check_plan(m, live, hq, hkv, mma_min_rows, fuse_final)
        # a subset of the threads, in another order
        sub = live[::2][::-1]
        check_plan(m, sub, hq, hkv, mma_min_rows, fuse_final)


def test_hand_worked_three_children():
    # prompt 64 -> 4 shared blocks; children of 32, 17, 40 tokens (config 1 of the benchmark)
    m = BlockModel(32, BS, 8, 16)
    (p,) = m.new_threads(1)
    m.append([p], [64])
    kids, _ = m.fork([p, p, p])
    m.append(kids, [32, 17, 40])
    tab, lens = tables_of(m, kids)
    items, users, merges, c = B.apar_debug_plan(32, 8, 2, tab, lens)
    assert c["unique_tokens"] == 153 and c["attended_tokens"] == 281
    shared = [it for it in items.tolist() if it[4] == 3]
    assert len(shared) == 1 and shared[0][1:3] == [0, 64]
    tails = sorted((it[1], it[2]) for it in items.tolist() if it[4] == 1)
    assert tails == [(64, 81), (64, 96), (64, 104)]
    assert len(merges) == 0                      # every chain ends in a private tail
    check_plan(m, kids, 8, 2, 2, True)


def test_wide_fork_is_cut_into_row_groups():
    m = BlockModel(400, BS, 200, 40)
    (p,) = m.new_threads(1)
    m.append([p], [100])
    kids, _ = m.fork([p] * 150)
    m.append(kids, [3] * 150)
    c = check_plan(m, kids, 4, 4, 2, True)       # 150 rows on the shared run: 64 + 64 + 22
    assert c["unique_tokens"] == 96 + 150 * (4 + 3)


def test_rejects_bad_input():
    tab = np.zeros((1, 4), dtype=np.int32)
    with pytest.raises(B.AparError):
        B.apar_debug_plan(8, 4, 4, tab, [0])
    with pytest.raises(B.AparError):
        B.apar_debug_plan(8, 4, 4, tab, [65])
    tab[0, 1] = 9
    with pytest.raises(B.AparError):
        B.apar_debug_plan(8, 4, 4, tab, [20])
    with pytest.raises(B.AparError):
        B.apar_debug_plan(8, 6, 4, tab[:, :1], [5])


def test_few_long_threads_are_spread_over_the_machine():
    m = BlockModel(9000, BS, 8, 8300)
    (p,) = m.new_threads(1)
    m.append([p], [131072 + 5])
    # one thread, 8 kv heads, 8 query rows per kv head: the ring-fed kernels get about one
    # (item, head) pair per CTA slot of the machine
    c = check_plan(m, [p], 64, 8, 2, True)
    assert 140 <= c["items"] <= 160 and c["merges"] == 1        # too many pieces to fold in one CTA
    # single-row items (32 kv heads, no sharing): cut finer, several CTAs per SM
    c1 = check_plan(m, [p], 32, 32, 2, True)
    assert c1["items"] >= 2 * 37
    # many threads: no cut at all
    m2, live = random_forest(5, n_roots=3, steps=40)
    c2 = check_plan(m2, live, 32, 32, 2, True)
    assert c2["items"] <= 2 * c2["users"]


@pytest.mark.parametrize("hq,hkv", [(65, 1), (71, 1), (128, 1), (256, 2)])
def test_more_than_64_query_heads_per_kv_head_are_refused(hq, hkv):
    """A work item carries every query head of a kv head for at least one thread, at most 64
    rows: wider groups have no kernel and must be turned down before any planning."""
    m = BlockModel(64, BS, 4, 16)
    (t,) = m.new_threads(1)
    m.append([t], [40])
    tab, lens = tables_of(m, [t])
    with pytest.raises(B.AparError) as e:
        B.apar_debug_plan(m.num_blocks, hq, hkv, tab, lens, 2, True)
    assert e.value.code == "UNSUPPORTED"
    assert B.apar_workspace_bytes(B.make_config(64, hq, hkv, 4, 16)) == 0
    B.apar_debug_plan(m.num_blocks, 64, 1, tab, lens, 2, True)        # the widest group allowed

"""The library's bookkeeping without a GPU (host-only context) against the independent pool
model: block tables, reference counts, free list and the max-cached counter bit for bit after
every call, the library's own invariant check (which also covers its per-thread group runs),
and the planner walking groups of blocks against the planner walking block ids."""
import random

import numpy as np
import pytest

from oracle import BlockModel
from oracle.bookkeeping import BookkeepingError as ModelError
from paper_2401_06761_b200 import binding as B
from paper_2401_06761_b200 import synth

BS = 16


class HostLibrary:
    """new_threads / fork / append / release through the C ABI of a host-only context."""

    def __init__(self, hq, hkv, num_blocks, max_threads, max_blocks):
        self.cfg = B.make_config(num_blocks, hq, hkv, max_threads, max_blocks)
        self.ctx = B.apar_create_host_only(self.cfg)
        self.num_blocks = num_blocks

    def new_threads(self, n):
        return B.apar_new_threads(self.ctx, n)

    def fork(self, parents):
        return B.apar_fork(self.ctx, parents, 0)

    def append(self, tids, counts, k=None, v=None):
        B.apar_append_kv(self.ctx, tids, counts, 0, 0, 0)

    def release(self, tids):
        B.apar_release(self.ctx, tids)

    def accept(self, tids, n_cand, keep):
        B.apar_accept_candidates(self.ctx, tids, n_cand, keep, 0)

    def close(self):
        B.apar_destroy(self.ctx)


def same_state(lib, m):
    B.apar_check_invariants(lib.ctx)
    for t in m.tables:
        assert B.apar_get_thread(lib.ctx, t) == (m.lens[t], m.tables[t]), f"thread {t}"
    assert B.apar_get_refcounts(lib.ctx, m.num_blocks) == m.refcount
    assert B.apar_get_free_list(lib.ctx, m.num_blocks) == m.free_list()
    st = B.apar_get_stats(lib.ctx)
    assert st["peak_used_blocks"] == m.peak_used and st["used_blocks"] == m.used_blocks()
    assert st["live_threads"] == len(m.tables)


def same_plans(lib, m, threads, hq, hkv):
    """group-walking planner == block-walking planner == planner on the model's tables"""
    for min_rows, fuse in ((2, True), (1, True), (10 ** 9, False)):
        a = B.apar_debug_plan_threads(lib.ctx, threads, True, min_rows, fuse)
        b = B.apar_debug_plan_threads(lib.ctx, threads, False, min_rows, fuse)
        for x, y in zip(a[:3], b[:3]):
            assert np.array_equal(x, y)
        assert a[3] == b[3]
        assert a[3]["unique_tokens"] == m.unique_tokens(threads)
        assert a[3]["attended_tokens"] == m.attended_tokens(threads)


@pytest.mark.parametrize("seed", range(6))
def test_random_replay_matches_the_pool_model(seed):
    rnd = random.Random(seed)
    hq, hkv = rnd.choice([(8, 2), (4, 4), (32, 8), (16, 1)])
    nb, nt, mb = 1500, 120, 40
    lib, m = HostLibrary(hq, hkv, nb, nt, mb), BlockModel(nb, BS, nt, mb)
    live = lib.new_threads(3)
    assert m.new_threads(3) == live
    first = [rnd.randrange(1, 200) for _ in live]
    lib.append(live, first)
    m.append(live, first)
    for step in range(300):
        op = rnd.random()
        try:
            if op < 0.3:
                parents = [rnd.choice(live) for _ in range(rnd.randrange(1, 5))]
                kids, _ = m.fork(parents)
                assert lib.fork(parents) == kids
                live += kids
            elif op < 0.7:
                sub = rnd.sample(live, rnd.randrange(1, len(live) + 1))
                cnt = [rnd.choice([0, 1, 1, 1, 2, 15, 16, 17, 40]) for _ in sub]
                m.append(sub, cnt)
                lib.append(sub, None if all(c == 1 for c in cnt) else cnt)
            elif op < 0.85:
                # predict-verify: speculated rows at the end of some threads, part of them kept
                sub = rnd.sample(live, rnd.randrange(1, min(4, len(live)) + 1))
                cnt = [rnd.randrange(1, 40) for _ in sub]
                m.append(sub, cnt)
                lib.append(sub, cnt)
                same_state(lib, m)
                keep = [sorted(rnd.sample(range(k), rnd.randrange(0, k + 1))) for k in cnt]
                m.accept(sub, cnt, [len(k) for k in keep])
                lib.accept(sub, cnt, keep)
            elif len(live) > 2:
                gone = rnd.sample(live, rnd.randrange(1, 3))
                m.release(gone)
                lib.release(gone)
                live = [t for t in live if t not in gone]
        except ModelError as e:                   # the library refuses the same call, same code
            with pytest.raises(B.AparError) as le:
                if op < 0.3:
                    lib.fork(parents)
                elif op < 0.85:
                    lib.append(sub, cnt)      # (an accept only ever follows its own append)
                else:
                    lib.release(gone)
            assert le.value.code == e.code
        same_state(lib, m)
        if step % 25 == 0:
            q = [t for t in live if m.lens[t] > 0]
            same_plans(lib, m, rnd.sample(q, rnd.randrange(1, len(q) + 1)), hq, hkv)
    lib.release(live)
    m.release(live)
    same_state(lib, m)
    assert B.apar_get_stats(lib.ctx)["free_blocks"] == nb
    lib.close()


@pytest.mark.parametrize("config,nreq", [(1, 1), (2, 3), (3, 12), (4, 3), (5, 40)])
def test_benchmark_forests_on_the_host(config, nreq, monkeypatch):
    """The five workload shapes built through the library's bookkeeping alone."""
    import torch
    spec = synth.forest_spec(config, n_requests=nreq)
    # no values are needed here: the rows themselves never reach a host-only context
    monkeypatch.setattr(synth, "node_kv", lambda s, n, device="cpu": (
        torch.empty((n.n_tok, 0)), torch.empty((n.n_tok, 0))))
    monkeypatch.setattr(synth, "queries", lambda *a, **k: None)
    from paper_2401_06761_b200.session import pool_requirements
    nb, nt, mb = pool_requirements(spec)
    s = spec.shape
    lib, m = HostLibrary(s.num_q_heads, s.num_kv_heads, nb, nt, mb), BlockModel(nb, BS, nt, mb)

    class Both:
        @staticmethod
        def new_threads(n):
            ids = lib.new_threads(n)
            assert m.new_threads(n) == ids
            return ids

        @staticmethod
        def fork(parents):
            ids = lib.fork(parents)
            assert m.fork(parents)[0] == ids
            return ids

        @staticmethod
        def append(tids, counts, k, v):
            counts = [1] * len(tids) if counts is None else list(counts)
            lib.append(tids, counts)
            m.append(tids, counts)

    step = synth.build_forest(spec, Both, device="cpu")
    synth.run_step_forks(step, Both)
    Both.append(step.live_handles, None, None, None)
    same_state(lib, m)
    same_plans(lib, m, step.live_handles, s.num_q_heads, s.num_kv_heads)
    # the hand-worked counts of config 1: 11 blocks in use, attended 96 / 81 / 104
    if config == 1:
        assert B.apar_get_stats(lib.ctx)["used_blocks"] == 11
        assert [B.apar_get_thread(lib.ctx, t)[0] for t in step.live_handles] == [96, 81, 104]
    with pytest.raises(B.AparError) as e:
        B.apar_decode_step(lib.ctx, step.live_handles, 0, 0, 0, 0, 1.0, 0)
    assert e.value.code in ("UNSUPPORTED", "INVALID_ARG")
    lib.close()


def test_accept_events_of_the_golden_file_through_the_library():
    """The hand-worked predict-verify events (tests/golden/accept_candidates.txt), library side."""
    from test_oracle_bookkeeping import accept_events, load_golden
    g = load_golden("accept_candidates.txt")
    lib = HostLibrary(8, 2, g["num_blocks"], 8, 16)
    in_use, peak = [], []
    for ev in accept_events():
        if ev[0] == "new+append":
            (t,) = lib.new_threads(1)
            lib.append([t], [ev[1]])
        elif ev[0] == "append":
            lib.append([ev[1]], [ev[2]])
        elif ev[0] == "fork":
            lib.fork([ev[1]])
        elif ev[0] == "accept":
            lib.accept([ev[1]], [ev[2]], [list(range(ev[3]))])
        else:
            with pytest.raises(B.AparError) as e:
                lib.accept([ev[1]], [ev[2]], [list(range(ev[3]))])
            assert e.value.code == "INVALID_ARG"
        B.apar_check_invariants(lib.ctx)
        st = B.apar_get_stats(lib.ctx)
        in_use.append(st["used_blocks"])
        peak.append(st["peak_used_blocks"])
    assert in_use == g["in_use_after_event"] and peak == g["peak_after_event"]
    for t, table in g["table"].items():
        assert B.apar_get_thread(lib.ctx, t) == (g["len"][t], table)
    assert B.apar_get_refcounts(lib.ctx, g["num_blocks"]) == g["refcount"]
    assert B.apar_get_free_list(lib.ctx, g["num_blocks"]) == g["free_list"]
    lib.close()

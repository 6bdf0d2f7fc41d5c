"""Parity of the CUDA library (through the C ABI) with the CPU checker, element by element:
bookkeeping bit-exact, pool bytes bit-exact, attention within max 2e-2 / mean 1e-3."""
import random

import numpy as np
import pytest
import torch

from helpers import OracleBackend, assert_close, assert_same_bookkeeping
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


def _session(*a, **k):
    from paper_2401_06761_b200.session import PagedSession
    return PagedSession(*a, **k)


class Both:
    """Drives the library and the checker with the same events and checks they agree on ids."""

    def __init__(self, sess, orc):
        self.sess, self.orc = sess, orc

    def new_threads(self, n):
        a, b = self.sess.new_threads(n), self.orc.new_threads(n)
        assert a == b
        return a

    def fork(self, parents):
        a, b = self.sess.fork(parents), self.orc.fork(parents)
        assert a == b
        # copy-on-fork: the r valid rows of the source block, bit for bit
        for src, dst, rows in self.orc.copies:
            for pool in (self.sess.k_pool, self.sess.v_pool):
                assert torch.equal(pool[dst, :, :rows].view(torch.int16),
                                   pool[src, :, :rows].view(torch.int16))
        return a

    def append(self, tids, counts, k, v):
        self.sess.append(tids, counts, k, v)
        self.orc.append(tids, counts, k, v)

    def release(self, tids):
        self.sess.release(tids)
        self.orc.release(tids)


def _bf16_floor(ref):
    """Mean error that rounding the checker's fp64 result to bf16 (nearest even) makes by itself:
    no bf16 output can be closer to it on average."""
    r = torch.from_numpy(np.ascontiguousarray(ref))
    return (r.to(torch.bfloat16).to(torch.float64) - r).abs().mean().item()


def _pool_rows(sess, tid):
    """K and V rows of a thread as the pool holds them, gathered through its block table."""
    ln, blocks = sess.thread(tid)
    idx = torch.tensor(blocks, device=sess.k_pool.device, dtype=torch.long)
    k = sess.k_pool[idx].permute(0, 2, 1, 3).reshape(-1, *sess.k_pool.shape[1:2], 128)[:ln]
    v = sess.v_pool[idx].permute(0, 2, 1, 3).reshape(-1, *sess.v_pool.shape[1:2], 128)[:ln]
    return k.cpu().to(torch.float64).numpy(), v.cpu().to(torch.float64).numpy()


def _make(spec, path, monkeypatch, extra_blocks=0):
    from paper_2401_06761_b200.session import PagedSession, pool_requirements
    monkeypatch.setenv("APAR_ATTN_PATH", path)
    sess = PagedSession.for_spec(spec, poison=True, extra_blocks=extra_blocks)
    _, nt, mb = pool_requirements(spec)
    orc = OracleBackend(spec.shape, sess.num_blocks, nt, mb)
    return sess, orc, Both(sess, orc)


@pytest.mark.parametrize("path", ["vec", "umma", "ws", "auto"])
@pytest.mark.parametrize("config,nreq", [(1, 1), (2, 3), (3, 6), (4, 2), (5, 24)])
def test_config_step_parity(config, nreq, path, monkeypatch):
    spec = synth.forest_spec(config, n_requests=nreq)
    sess, orc, both = _make(spec, path, monkeypatch)
    step = synth.build_forest(spec, both, device="cuda")
    synth.run_step_forks(step, both)                       # the step's own fork (config 3)
    live = step.live_handles
    both.append(live, None, step.k_new, step.v_new)        # the step's KV append
    assert_same_bookkeeping(sess, orc.model, list(orc.model.tables))
    for t in live[:: max(1, len(live) // 16)]:             # pool bytes through the tables
        k, v = _pool_rows(sess, t)
        ck, cv = orc.forest.chain(orc.node_of[t])
        assert np.array_equal(k, ck) and np.array_equal(v, cv)
    out = sess.attention(live, step.q)
    ref = orc.attention(live, step.q, sess.sm_scale)
    assert_close(out, ref, f"config {config} path {path}")
    st = sess.stats()
    assert st["attn_threads"] == len(live)
    assert st["attn_attended_tokens"] == orc.model.attended_tokens(live) == spec.unshared_tokens()
    assert st["attn_unique_tokens"] == orc.model.unique_tokens(live)
    assert st["cow_blocks"] == orc.model.cow_blocks and st["cow_rows"] == orc.model.cow_rows
    if config == 1:
        assert [sess.thread(t)[0] for t in live] == [96, 81, 104]
        assert st["attn_unique_tokens"] == 153 and st["attn_attended_tokens"] == 281
    sess.close()


@pytest.mark.parametrize("path", ["vec", "umma", "ws", "auto"])
def test_random_event_replay_with_plan_reuse(path, monkeypatch):
    shape = synth.LayerShape(8, 2)
    monkeypatch.setenv("APAR_ATTN_PATH", path)
    sess = _session(shape, 600, 48, 40, poison=True)
    orc = OracleBackend(shape, 600, 48, 40)
    both = Both(sess, orc)
    rnd = random.Random(5)
    g = torch.Generator(device="cuda").manual_seed(17)

    def rows(n):
        return torch.randn((n, 2, 128), generator=g, device="cuda").to(torch.bfloat16)

    live = both.new_threads(2)
    cnt = [rnd.randrange(1, 80) for _ in live]
    both.append(live, cnt, rows(sum(cnt)), rows(sum(cnt)))
    reused = 0
    for it in range(60):
        op = rnd.random()
        if op < 0.2 and len(live) < 40:
            parents = [rnd.choice(live) for _ in range(rnd.randrange(1, 4))]
            live += both.fork(parents)                      # parents stay live and keep growing
        elif op < 0.3 and len(live) > 3:
            gone = rnd.sample(live, 1)
            both.release(gone)
            live = [t for t in live if t not in gone]
        elif op < 0.4:
            sub = rnd.sample(live, rnd.randrange(1, len(live) + 1))
            cnt = [rnd.randrange(0, 40) for _ in sub]
            both.append(sub, cnt, rows(sum(cnt)), rows(sum(cnt)))
        # a decode step: one token for everybody, then attention
        both.append(live, None, rows(len(live)), rows(len(live)))
        assert_same_bookkeeping(sess, orc.model, live)
        tids = live if it % 7 else live + live[:2]          # sometimes list a thread twice
        q = torch.randn((len(tids), 8, 128), generator=g, device="cuda").to(torch.bfloat16)
        out = sess.attention(tids, q)
        assert_close(out, orc.attention(tids, q, sess.sm_scale), f"iteration {it}")
        reused += sess.stats()["attn_plan_reused"]
        if it % 7:
            assert sess.stats()["attn_unique_tokens"] == orc.model.unique_tokens(live)
    assert reused > 10          # consecutive steps over the same threads reuse the plan
    both.release(live)
    assert sess.stats()["free_blocks"] == 600
    sess.close()


@pytest.mark.parametrize("path", ["vec", "umma", "ws", "auto"])
@pytest.mark.parametrize("hq,hkv,n_children,prompt", [(4, 4, 40, 100), (16, 2, 12, 333),
                                                      (8, 8, 2, 1), (8, 1, 70, 48)])
def test_wide_forks(hq, hkv, n_children, prompt, path, monkeypatch):
    """More query rows on one shared run than a work item carries; ragged fork point."""
    shape = synth.LayerShape(hq, hkv)
    monkeypatch.setenv("APAR_ATTN_PATH", path)
    sess = _session(shape, 400, n_children + 4, 40, poison=True)
    orc = OracleBackend(shape, 400, n_children + 4, 40)
    both = Both(sess, orc)
    g = torch.Generator(device="cuda").manual_seed(3)

    def rows(n):
        return torch.randn((n, hkv, 128), generator=g, device="cuda").to(torch.bfloat16)

    (p,) = both.new_threads(1)
    both.append([p], [prompt], rows(prompt), rows(prompt))
    kids = both.fork([p] * n_children)
    cnt = [1 + (7 * i) % 23 for i in range(n_children)]
    both.append(kids, cnt, rows(sum(cnt)), rows(sum(cnt)))
    tids = kids + [p]
    q = torch.randn((len(tids), hq, 128), generator=g, device="cuda").to(torch.bfloat16)
    assert_close(sess.attention(tids, q), orc.attention(tids, q, sess.sm_scale))
    assert_same_bookkeeping(sess, orc.model, tids)
    sess.close()


@pytest.mark.parametrize("path", ["vec", "umma", "ws", "auto"])
def test_long_thread_is_split_and_merged(path, monkeypatch):
    shape = synth.LayerShape(8, 2)
    monkeypatch.setenv("APAR_ATTN_PATH", path)
    n = 20011
    sess = _session(shape, 1300, 4, 1300, poison=True)
    orc = OracleBackend(shape, 1300, 4, 1300)
    both = Both(sess, orc)
    g = torch.Generator(device="cuda").manual_seed(9)
    k = torch.randn((n, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn((n, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    (t,) = both.new_threads(1)
    both.append([t], [n], k, v)
    q = torch.randn((1, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.attention([t], q)
    assert_close(out, orc.attention([t], q, sess.sm_scale))
    st = sess.stats()
    assert st["attn_work_items"] > 8 and st["attn_partials"] == st["attn_work_items"] * 8
    sess.close()


def test_single_token_and_scale_argument(monkeypatch):
    shape = synth.LayerShape(8, 2)
    sess = _session(shape, 8, 4, 4, poison=True)
    g = torch.Generator(device="cuda").manual_seed(1)
    k = torch.randn((1, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn((1, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    (t,) = sess.new_threads(1)
    sess.append([t], None, k, v)
    q = torch.randn((1, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.attention([t], q)                 # one token: out = its V row, exactly
    assert torch.equal(out[0], v[0].repeat_interleave(4, 0))
    # scale matters: with two tokens and scale 0 the output is the plain mean of V
    k2 = torch.randn((1, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    v2 = torch.randn((1, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    sess.append([t], None, k2, v2)
    out0 = sess.attention([t], q, sm_scale=0.0)
    mean = ((v.double() + v2.double()) / 2)[0].repeat_interleave(4, 0)
    assert (out0.double() - mean).abs().max() < 1e-2
    sess.close()


def test_tables_entry_point_and_block_placement(monkeypatch):
    """The table-driven call gives the same answer, and physically moving blocks (a shuffled
    placement with the same logical forest) changes nothing beyond rounding."""
    from paper_2401_06761_b200 import binding as B
    spec = synth.forest_spec(3, n_requests=4)
    sess, orc, both = _make(spec, "auto", monkeypatch)
    step = synth.build_forest(spec, both, device="cuda")
    synth.run_step_forks(step, both)
    live = step.live_handles
    both.append(live, None, step.k_new, step.v_new)
    ref = orc.attention(live, step.q, sess.sm_scale)
    out_ctx = sess.attention(live, step.q)
    mb = sess.cfg.max_blocks_per_thread
    lens, tables = zip(*(sess.thread(t) for t in live))
    out_tab = torch.empty_like(step.q)
    B.apar_tree_decode_attention_tables(sess.cfg, [t + [0] * (mb - len(t)) for t in tables], lens,
                                        step.q.data_ptr(), out_tab.data_ptr(), sess.sm_scale,
                                        torch.cuda.current_stream().cuda_stream)
    assert_close(out_tab, ref, "tables entry point")
    assert (out_tab.double() - out_ctx.double()).abs().max() <= 2e-2
    # shuffled placement: new[perm[b]] = old[b]
    perm = torch.randperm(sess.num_blocks, generator=torch.Generator().manual_seed(4))
    k2, v2 = torch.empty_like(sess.k_pool), torch.empty_like(sess.v_pool)
    k2[perm.cuda()] = sess.k_pool
    v2[perm.cuda()] = sess.v_pool
    cfg2 = B.make_config(sess.num_blocks, spec.shape.num_q_heads, spec.shape.num_kv_heads,
                         sess.cfg.max_threads, mb, k2.data_ptr(), v2.data_ptr(),
                         sess.cfg.workspace, sess.cfg.workspace_bytes)
    tables2 = [[int(perm[b]) for b in t] + [0] * (mb - len(t)) for t in tables]
    out_perm = torch.empty_like(step.q)
    B.apar_tree_decode_attention_tables(cfg2, tables2, lens, step.q.data_ptr(),
                                        out_perm.data_ptr(), sess.sm_scale,
                                        torch.cuda.current_stream().cuda_stream)
    assert_close(out_perm, ref, "shuffled placement")
    sess.close()


def test_error_codes_match_the_model_and_change_nothing():
    from paper_2401_06761_b200 import binding as B
    from oracle import BookkeepingError
    shape = synth.LayerShape(8, 2)
    sess = _session(shape, 6, 4, 4)
    orc = OracleBackend(shape, 6, 4, 4)
    both = Both(sess, orc)
    z = torch.zeros((120, 2, 128), dtype=torch.bfloat16, device="cuda")
    a, b = both.new_threads(2)
    both.append([a, b], [20, 17], z[:37], z[:37])
    cases = [
        (lambda s: s.fork([a, b, a]), "NO_THREADS"),
        (lambda s: s.append([a, b], [30, 30], z[:60], z[:60]), "NO_BLOCKS"),
        (lambda s: s.append([a], [60], z[:60], z[:60]), "TABLE_FULL"),
        (lambda s: s.append([a, a], None, z[:2], z[:2]), "INVALID_ARG"),
        (lambda s: s.append([a, 99], None, z[:2], z[:2]), "BAD_THREAD"),
        (lambda s: s.release([a, a]), "BAD_THREAD"),
        (lambda s: s.fork([7]), "BAD_THREAD"),
    ]
    for call, code in cases:
        with pytest.raises(B.AparError) as e:
            call(sess)
        assert e.value.code == code
        with pytest.raises(BookkeepingError) as e2:
            call(orc)
        assert e2.value.code == code
        assert_same_bookkeeping(sess, orc.model, [a, b])
    (c,) = both.new_threads(1)
    q = torch.zeros((1, 8, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.AparError) as e:
        sess.attention([c], q)
    assert e.value.code == "EMPTY_CONTEXT"
    with pytest.raises(B.AparError) as e:
        sess.attention([55], q)
    assert e.value.code == "BAD_THREAD"
    assert sess.attention([], q[:0]).shape[0] == 0
    bad = B.make_config(6, 8, 3, 4, 4)
    assert B.apar_workspace_bytes(bad) == 0
    sess.close()


@pytest.mark.parametrize("path", ["vec", "umma", "ws", "auto"])
@pytest.mark.parametrize("hq,hkv,kids", [(4, 4, 5), (16, 2, 6), (8, 8, 1)])
def test_scores_that_keep_growing_move_the_softmax_reference(hq, hkv, kids, path, monkeypatch):
    """Every later token scores far higher than all earlier ones, so the running maximum rises by
    many powers of two from tile to tile (and the early tokens end up with negligible weight)."""
    shape = synth.LayerShape(hq, hkv)
    monkeypatch.setenv("APAR_ATTN_PATH", path)
    sess = _session(shape, 200, kids + 3, 40, poison=True)
    orc = OracleBackend(shape, 200, kids + 3, 40)
    both = Both(sess, orc)
    g = torch.Generator(device="cuda").manual_seed(21)
    u = torch.randn((128,), generator=g, device="cuda")
    u = u / u.norm()
    n_prompt, n_tail = 330, 45

    def rows(n, start):
        ramp = (torch.arange(start, start + n, device="cuda", dtype=torch.float32) * 0.35)
        k = ramp[:, None, None] * u[None, None, :] + 0.05 * torch.randn((n, hkv, 128), generator=g,
                                                                        device="cuda")
        v = torch.randn((n, hkv, 128), generator=g, device="cuda")
        return k.to(torch.bfloat16), v.to(torch.bfloat16)

    (p,) = both.new_threads(1)
    both.append([p], [n_prompt], *rows(n_prompt, 0))
    tids = both.fork([p] * kids) if kids > 1 else [p]
    for i, t in enumerate(tids):
        both.append([t], [n_tail + i], *rows(n_tail + i, n_prompt))
    q = (8.0 * u[None, None, :] + 0.1 * torch.randn((len(tids), hq, 128), generator=g,
                                                    device="cuda")).to(torch.bfloat16)
    out = sess.attention(tids, q, sm_scale=1.0)
    ref = orc.attention(tids, q, 1.0)
    # The softmax is nearly one-hot here, so outputs are single V rows of magnitude ~1 and the
    # rounding of the exact result to bf16 alone is of the order of the usual mean tolerance.
    # That floor is measured on the checker's own result and added to the bound.
    err = np.abs(out.cpu().to(torch.float64).numpy() - ref)
    assert np.isfinite(err).all() and err.max() <= 2e-2, (path, err.max())
    assert err.mean() <= 1e-3 + _bf16_floor(ref), (path, err.mean())
    sess.close()


@pytest.mark.parametrize("heads", ["1", "2", "4", "8"])
def test_tcgen05_kernel_with_several_kv_heads_per_cta(heads, monkeypatch):
    """The tensor-core kernel lets a CTA walk several kv heads of its item, the barrier phases
    running on from head to head; forced here to every group size, on items with one ragged
    tile, with many tiles, and with scores that make the softmax reference move in each head."""
    monkeypatch.setenv("APAR_UMMA_HEADS", heads)
    for config, nreq in [(4, 2), (5, 24)]:
        spec = synth.forest_spec(config, n_requests=nreq)
        sess, orc, both = _make(spec, "umma", monkeypatch)
        step = synth.build_forest(spec, both, device="cuda")
        live = step.live_handles
        both.append(live, None, step.k_new, step.v_new)
        out = sess.attention(live, step.q)
        assert_close(out, orc.attention(live, step.q, sess.sm_scale), f"cfg{config} heads {heads}")
        assert sess.stats()["device_wait_timeouts"] == 0
        sess.close()
    # wide fork over 8 kv heads, prompt of 37 tokens (a single ragged tile) and of 700
    shape = synth.LayerShape(16, 8)
    for prompt in (37, 700):
        sess = _session(shape, 400, 16, 64, poison=True)
        orc = OracleBackend(shape, 400, 16, 64)
        both = Both(sess, orc)
        g = torch.Generator(device="cuda").manual_seed(prompt)
        (p,) = both.new_threads(1)
        ramp = torch.arange(prompt, device="cuda", dtype=torch.float32)[:, None, None] * 0.3
        k = (ramp * torch.ones((1, 8, 128), device="cuda") / 11.3 +
             torch.randn((prompt, 8, 128), generator=g, device="cuda")).to(torch.bfloat16)
        v = torch.randn((prompt, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
        both.append([p], [prompt], k, v)
        kids = both.fork([p] * 12)
        both.append(kids, None,
                    torch.randn((12, 8, 128), generator=g, device="cuda").to(torch.bfloat16),
                    torch.randn((12, 8, 128), generator=g, device="cuda").to(torch.bfloat16))
        q = (torch.ones((12, 16, 128), device="cuda") +
             0.3 * torch.randn((12, 16, 128), generator=g, device="cuda")).to(torch.bfloat16)
        out = sess.attention(kids, q, sm_scale=1.0)
        ref = orc.attention(kids, q, 1.0)
        err = np.abs(out.cpu().to(torch.float64).numpy() - ref)
        assert np.isfinite(err).all() and err.max() <= 2e-2, (heads, prompt, err.max())
        assert err.mean() <= 1e-3 + _bf16_floor(ref), (heads, prompt, err.mean())
        assert sess.stats()["device_wait_timeouts"] == 0
        sess.close()


@pytest.mark.parametrize("kids", [1, 3, 6])
def test_long_context_shared_by_forks(kids, monkeypatch):
    """A 131 077-token prompt (8193 blocks, ragged end) read by 1, 3 or 6 forked threads: the run
    is cut into chunks over all SMs, shared chunks go to the warp-stream kernel (12 rows) or the
    tensor-core kernel (24 rows), and every query merges dozens of partial results."""
    shape = synth.LayerShape(8, 2)
    monkeypatch.setenv("APAR_ATTN_PATH", "auto")
    n = 131072 + 5
    nb = 8193 + 8 * 3 + 4
    sess = _session(shape, nb, 8, 8200, poison=True)
    orc = OracleBackend(shape, nb, 8, 8200)
    both = Both(sess, orc)
    g = torch.Generator(device="cuda").manual_seed(77)
    k = torch.randn((n, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn((n, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
    (p,) = both.new_threads(1)
    both.append([p], [n], k, v)
    tids = both.fork([p] * kids) if kids > 1 else [p]
    if kids > 1:
        cnt = [3 + 7 * i for i in range(kids)]
        both.append(tids, cnt,
                    torch.randn((sum(cnt), 2, 128), generator=g, device="cuda").to(torch.bfloat16),
                    torch.randn((sum(cnt), 2, 128), generator=g, device="cuda").to(torch.bfloat16))
    assert_same_bookkeeping(sess, orc.model, list(orc.model.tables))
    q = torch.randn((len(tids), 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.attention(tids, q)
    assert_close(out, orc.attention(tids, q, sess.sm_scale), f"128k context, {kids} threads")
    st = sess.stats()
    assert st["device_wait_timeouts"] == 0
    assert st["attn_unique_tokens"] == orc.model.unique_tokens(tids)
    assert st["attn_work_items"] >= 100          # the prompt is spread over the machine
    sess.close()

"""The single-call decode step (append one row per thread + attention) against the pool model
and the fp64 checker: same block ids as the two-call sequence, step after step, across block
boundaries, list changes, forks and releases; and a whole multi-layer step replayed from a CUDA
graph for several consecutive steps."""
import numpy as np
import pytest
import torch

from helpers import OracleBackend, assert_close, assert_same_bookkeeping
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


def _rand(shape, g):
    return torch.randn(shape, generator=g, device="cuda").to(torch.bfloat16)


@pytest.mark.parametrize("config,nreq", [(2, 2), (3, 4), (4, 2), (5, 12)])
def test_steps_match_the_pool_model_and_the_checker(config, nreq):
    from paper_2401_06761_b200.session import PagedSession, pool_requirements
    spec = synth.forest_spec(config, n_requests=nreq)
    shape = spec.shape
    nb, nt, mb = pool_requirements(spec)
    nb, nt, mb = nb + 40 * len(spec.nodes), nt + 8, mb + 6
    sess = PagedSession(shape, nb, nt, mb, poison=True)
    orc = OracleBackend(shape, nb, nt, mb)

    class Both:
        @staticmethod
        def new_threads(n):
            ids = sess.new_threads(n)
            assert orc.new_threads(n) == ids
            return ids

        @staticmethod
        def fork(parents):
            ids = sess.fork(parents)
            assert orc.fork(parents) == ids
            return ids

        @staticmethod
        def append(tids, counts, k, v):
            sess.append(tids, counts, k, v)
            orc.append(tids, counts, k, v)

    step = synth.build_forest(spec, Both, device="cuda")
    synth.run_step_forks(step, Both)
    live = list(step.live_handles)
    g = torch.Generator(device="cuda").manual_seed(config)
    reused = 0
    for i in range(40):
        if i == 13:                    # a listed thread grows outside the step call
            k1, v1 = _rand((1, shape.num_kv_heads, 128), g), _rand((1, shape.num_kv_heads, 128), g)
            Both.append([live[0]], None, k1, v1)
        if i == 21:                    # the list changes: a fork joins, a thread finishes
            (kid,) = Both.fork([live[1]])
            gone = live.pop(2)
            sess.release([gone])
            orc.release([gone])
            live.append(kid)
        n = len(live)
        k = _rand((n, shape.num_kv_heads, 128), g)
        v = _rand((n, shape.num_kv_heads, 128), g)
        q = _rand((n, shape.num_q_heads, 128), g)
        out = sess.decode_step(live, k, v, q)
        orc.append(live, None, k, v)
        reused += sess.stats()["attn_plan_reused"]
        assert_same_bookkeeping(sess, orc.model, list(orc.model.tables))
        if i % 5 == 0 or i in (13, 14, 21, 22, 39):
            assert_close(out, orc.attention(live, q, sess.sm_scale), f"step {i}")
    assert reused >= 20                 # steady steps keep the device-resident plan
    st = sess.stats()
    assert st["attn_attended_tokens"] == sum(orc.model.lens[t] for t in live)
    assert st["device_wait_timeouts"] == 0
    sess.close()


def test_step_errors_change_nothing():
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession
    shape = synth.LayerShape(8, 2)
    sess = PagedSession(shape, 6, 8, 3, poison=True)
    orc = OracleBackend(shape, 6, 8, 3)
    g = torch.Generator(device="cuda").manual_seed(1)
    a, b = sess.new_threads(2)
    assert orc.new_threads(2) == [a, b]
    k, v = _rand((30, 2, 128), g), _rand((30, 2, 128), g)
    for be in (sess, orc):
        be.append([a, b], [16, 14], k, v)
    k2, v2, q2 = _rand((2, 2, 128), g), _rand((2, 2, 128), g), _rand((2, 8, 128), g)

    def refused(tids, code):
        with pytest.raises(B.AparError) as e:
            sess.decode_step(tids, k2[:len(tids)], v2[:len(tids)], q2[:len(tids)].contiguous())
        assert e.value.code == code
        assert_same_bookkeeping(sess, orc.model, [a, b])

    refused([a, a], "INVALID_ARG")
    refused([a, 77], "BAD_THREAD")
    with pytest.raises(B.AparError):
        B.apar_steps_before_new_block(sess.ctx)            # no step list yet
    # two steps fill a's second block position 17.. and b's first block; then pool runs dry
    for _ in range(2):
        out = sess.decode_step([a, b], k2, v2, q2)
        orc.append([a, b], None, k2, v2)
        assert_close(out, orc.attention([a, b], q2, sess.sm_scale))
    assert_same_bookkeeping(sess, orc.model, [a, b])
    assert B.apar_steps_before_new_block(sess.ctx) == 0     # b holds 16 rows: its next row needs a block
    others = sess.new_threads(1)
    assert orc.new_threads(1) == others
    for be in (sess, orc):
        be.append(others, [48], _rand((48, 2, 128), g), _rand((48, 2, 128), g))   # 3 blocks: pool empty
    refused([a, b], "NO_BLOCKS")
    sess.release(others)
    orc.release(others)
    for _ in range(15):                                     # a reaches 33 rows -> needs a 4th block of 3
        sess.decode_step([a], k2[:1], v2[:1], q2[:1].contiguous())
        orc.append([a], None, k2[:1], v2[:1])
    for _ in range(15):
        sess.decode_step([a], k2[:1], v2[:1], q2[:1].contiguous())
        orc.append([a], None, k2[:1], v2[:1])
    assert sess.thread(a)[0] == 48
    refused([a], "TABLE_FULL")
    sess.close()


def _aligned_spec(hq, hkv, n_req):
    """Requests whose live threads all sit two rows into a block after the build, so that the
    next thirteen steps start no block."""
    nodes = []
    for r in range(n_req):
        p = synth.Node(len(nodes), -1, r, 0, 70 + 16 * r, False)
        nodes.append(p)
        for n_tok in (13, 29, 45):                        # (70 + n_tok - 1) % 16 == 2
            c = synth.Node(len(nodes), p.index, r, 1, n_tok, True)
            nodes.append(c)
            p.children.append(c.index)
    return synth.ForestSpec(0, 4242, synth.LayerShape(hq, hkv), nodes)


def _layer_rows(k, v, layer):
    sign = -1.0 if layer % 2 else 1.0
    return ((sign * torch.roll(k, layer * 7, dims=-1)).contiguous(),
            (sign * torch.roll(v, layer * 3, dims=-1)).contiguous())


@pytest.mark.parametrize("hq,hkv", [(64, 8), (8, 8)])
def test_whole_step_of_all_layers_replayed_from_a_cuda_graph(hq, hkv):
    """append + attention of layers 0..L-1 of one decode step, captured once and replayed for
    four consecutive steps with new inputs; every layer against its own checker."""
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession, pool_requirements
    LAYERS = 3
    spec = _aligned_spec(hq, hkv, 3)
    shape = spec.shape
    nb, nt, mb = pool_requirements(spec)
    sess = PagedSession(shape, nb + 32, nt, mb + 2, poison=True, num_layers=LAYERS)
    oracles = [OracleBackend(shape, nb + 32, nt, mb + 2) for _ in range(LAYERS)]

    class Layered:
        @staticmethod
        def new_threads(n):
            ids = sess.new_threads(n)
            assert all(o.new_threads(n) == ids for o in oracles)
            return ids

        @staticmethod
        def fork(parents):
            ids = sess.fork(parents)
            assert all(o.fork(parents) == ids for o in oracles)
            return ids

        @staticmethod
        def append(tids, counts, k, v):
            sess.append(tids, counts, k, v)
            oracles[0].append(tids, counts, k, v)
            for l in range(1, LAYERS):
                kl, vl = _layer_rows(k, v, l)
                sess.append_layer(l, kl, vl)
                oracles[l].append(tids, counts, kl, vl)

    step = synth.build_forest(spec, Layered, device="cuda")
    live = step.live_handles
    n = len(live)
    g = torch.Generator(device="cuda").manual_seed(9)
    kbuf = [torch.empty((n, hkv, 128), dtype=torch.bfloat16, device="cuda") for _ in range(LAYERS)]
    vbuf = [torch.empty_like(kbuf[0]) for _ in range(LAYERS)]
    qbuf = [torch.empty((n, hq, 128), dtype=torch.bfloat16, device="cuda") for _ in range(LAYERS)]
    obuf = [torch.empty_like(qbuf[0]) for _ in range(LAYERS)]

    def new_inputs():
        k, v = _rand((n, hkv, 128), g), _rand((n, hkv, 128), g)
        for l in range(LAYERS):
            kl, vl = _layer_rows(k, v, l)
            kbuf[l].copy_(kl)
            vbuf[l].copy_(vl)
            qbuf[l].copy_(_rand((n, hq, 128), g))
            oracles[l].append(live, None, kl, vl)

    def whole_step():
        sess.decode_step(live, kbuf[0], vbuf[0], qbuf[0], out=obuf[0])
        for l in range(1, LAYERS):
            sess.append_layer(l, kbuf[l], vbuf[l])
            sess.attention_layer(l, qbuf[l], out=obuf[l])

    def check(what):
        torch.cuda.synchronize()
        for l in range(LAYERS):
            assert_close(obuf[l], oracles[l].attention(live, qbuf[l], sess.sm_scale),
                         f"{what}, layer {l}")
        assert_same_bookkeeping(sess, oracles[0].model, list(oracles[0].model.tables))

    # two eager steps: the first brings the list to the device and plans, the second is steady
    for i in range(2):
        new_inputs()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            whole_step()
        torch.cuda.current_stream().wait_stream(side)
        check(f"eager step {i}")
    assert sess.stats()["attn_plan_reused"] == 1
    assert B.apar_steps_before_new_block(sess.ctx) >= 6

    new_inputs()                       # the captured call does the bookkeeping of replay 1
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        whole_step()
    for o in obuf:
        o.zero_()
    graph.replay()
    check("replay 1")
    for r in range(2, 5):
        new_inputs()
        B.apar_note_step_replay(sess.ctx)
        for o in obuf:
            o.zero_()
        graph.replay()
        check(f"replay {r}")
    # an ordinary step afterwards carries on from the same state
    new_inputs()
    whole_step()
    check("eager step after the replays")
    # a bookkeeping call invalidates the replay protocol
    extra = sess.new_threads(1)
    for o in oracles:
        o.new_threads(1)
    sess.release(extra)
    for o in oracles:
        o.release(extra)
    with pytest.raises(B.AparError):
        B.apar_note_step_replay(sess.ctx)
    assert sess.stats()["device_wait_timeouts"] == 0
    sess.close()

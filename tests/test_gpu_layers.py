"""Several attention layers over one set of block tables: the bookkeeping and the plan are made
once per step, the other layers replay the scatter and the attention launches on their own
slab of the pools.  Every layer holds different data and is checked against its own checker."""
import pytest
import torch

from helpers import OracleBackend, assert_close, assert_same_bookkeeping
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu
LAYERS = 3


def _layer_rows(k, v, layer):
    """Rows of another layer derived from layer 0's: rolled along the feature axis and signed."""
    sign = -1.0 if layer % 2 else 1.0
    return ((sign * torch.roll(k, layer * 7, dims=-1)).contiguous(),
            (sign * torch.roll(v, layer * 3, dims=-1)).contiguous())


@pytest.mark.parametrize("config,nreq", [(3, 5), (4, 2), (5, 16)])
def test_layers_share_tables_and_plan(config, nreq):
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession, pool_requirements
    spec = synth.forest_spec(config, n_requests=nreq)
    nb, nt, mb = pool_requirements(spec)
    sess = PagedSession(spec.shape, nb, nt, mb, poison=True, num_layers=LAYERS)
    oracles = [OracleBackend(spec.shape, nb, nt, mb) for _ in range(LAYERS)]

    class Layered:
        def new_threads(self, n):
            ids = sess.new_threads(n)
            assert all(o.new_threads(n) == ids for o in oracles)
            return ids

        def fork(self, parents):
            ids = sess.fork(parents)                       # copies the partial block in every layer
            assert all(o.fork(parents) == ids for o in oracles)
            return ids

        def append(self, tids, counts, k, v):
            sess.append(tids, counts, k, v)                # bookkeeping + layer 0
            oracles[0].append(tids, counts, k, v)
            for l in range(1, LAYERS):
                kl, vl = _layer_rows(k, v, l)
                sess.append_layer(l, kl, vl)               # same slots, no bookkeeping
                oracles[l].append(tids, counts, kl, vl)

    both = Layered()
    step = synth.build_forest(spec, both, device="cuda")
    synth.run_step_forks(step, both)
    live = step.live_handles
    both.append(live, None, step.k_new, step.v_new)
    assert_same_bookkeeping(sess, oracles[0].model, list(oracles[0].model.tables))
    kernels0 = sess.stats()["kernels_total"]
    out0 = sess.attention(live, step.q)                    # plans; runs layer 0
    per_layer = sess.stats()["kernels_total"] - kernels0
    assert_close(out0, oracles[0].attention(live, step.q, sess.sm_scale), "layer 0")
    for l in range(1, LAYERS):
        ql = torch.roll(step.q, l, dims=-1).contiguous()
        before = sess.stats()["kernels_total"]
        outl = sess.attention_layer(l, ql)
        assert sess.stats()["kernels_total"] - before <= per_layer   # launches only, no sync kernel
        assert_close(outl, oracles[l].attention(live, ql, sess.sm_scale), f"layer {l}")
    # layer 0 again through the layer call gives the same bits as the planning call
    assert torch.equal(sess.attention_layer(0, step.q), out0)
    # a bookkeeping call invalidates the replay until the next planning call
    extra = sess.new_threads(1)
    with pytest.raises(B.AparError) as e:
        sess.attention_layer(1, step.q)
    assert e.value.code == "INVALID_ARG"
    sess.release(extra)
    assert sess.stats()["device_wait_timeouts"] == 0
    sess.close()


def test_layer_loop_replayed_from_a_cuda_graph():
    """The per-layer calls only launch kernels, with sizes fixed by the cached plan: the loop over
    layers 1.. of a step is captured once in a CUDA graph and replayed, for this step and - the
    plan being reused while threads only grow - for the next one."""
    from paper_2401_06761_b200.session import PagedSession, pool_requirements
    spec = synth.forest_spec(4, n_requests=3)
    nb, nt, mb = pool_requirements(spec)
    sess = PagedSession(spec.shape, nb + 64, nt, mb + 2, poison=True, num_layers=LAYERS)

    class Layered:
        new_threads, fork = sess.new_threads, sess.fork

        @staticmethod
        def append(tids, counts, k, v):
            sess.append(tids, counts, k, v)
            for l in range(1, LAYERS):
                sess.append_layer(l, *_layer_rows(k, v, l))

    step = synth.build_forest(spec, Layered, device="cuda")
    live = step.live_handles
    Layered.append(live, None, step.k_new, step.v_new)
    sess.attention(live, step.q)                                   # plans; layer 0
    q = [torch.roll(step.q, l, dims=-1).contiguous() for l in range(LAYERS)]
    kv = [list(_layer_rows(step.k_new, step.v_new, l)) for l in range(LAYERS)]
    eager = {l: sess.attention_layer(l, q[l]) for l in range(1, LAYERS)}
    out_g = {l: torch.zeros_like(step.q) for l in range(1, LAYERS)}

    def layer_loop():
        for l in range(1, LAYERS):
            sess.append_layer(l, kv[l][0], kv[l][1])
            sess.attention_layer(l, q[l], out=out_g[l])

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        layer_loop()                                               # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        layer_loop()
    for o in out_g.values():
        o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for l in range(1, LAYERS):
        assert torch.equal(out_g[l], eager[l]), l
    # next decode step: bookkeeping and layer 0 as usual, the other layers from the same graph
    g = torch.Generator(device="cuda").manual_seed(5)
    k2 = torch.randn(step.k_new.shape, generator=g, device="cuda").to(torch.bfloat16)
    v2 = torch.randn(step.v_new.shape, generator=g, device="cuda").to(torch.bfloat16)
    sess.append(live, None, k2, v2)
    sess.attention(live, step.q)
    assert sess.stats()["attn_plan_reused"] == 1
    for l in range(1, LAYERS):
        kl, vl = _layer_rows(k2, v2, l)
        kv[l][0].copy_(kl)
        kv[l][1].copy_(vl)
        out_g[l].zero_()
    graph.replay()
    torch.cuda.synchronize()
    for l in range(1, LAYERS):
        assert torch.equal(out_g[l], sess.attention_layer(l, q[l])), l   # eager, same pools
    assert sess.stats()["device_wait_timeouts"] == 0
    sess.close()

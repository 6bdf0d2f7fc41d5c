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

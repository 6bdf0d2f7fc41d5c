"""Full-size workloads, in the launch configuration the benchmark times: the library builds
the whole forest, runs the decode step, and a seeded sample of threads (every region of the
request range represented) is checked against the CPU checker one thread at a time.  The
checker's inputs are regenerated from the seeds, never read back from the pool."""
import numpy as np
import pytest
import torch

from helpers import MAX_ABS, MEAN_ABS, assert_same_bookkeeping
from oracle import BlockModel, Forest, tree_decode_attention
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


class WithModel:
    """Replays every bookkeeping event on the integer pool model as well (ids must agree); the
    rows themselves only go to the library - the attention checker regenerates them from seeds."""

    def __init__(self, sess, model):
        self.sess, self.model = sess, model

    def new_threads(self, n):
        a, b = self.sess.new_threads(n), self.model.new_threads(n)
        assert a == b
        return a

    def fork(self, parents):
        a, (b, _) = self.sess.fork(parents), self.model.fork(parents)
        assert a == b
        return a

    def append(self, tids, counts, k, v):
        self.sess.append(tids, counts, k, v)
        self.model.append(tids, counts)


# every thread of configs 1-3 (config 1 is covered in test_gpu_parity), a tenth of configs 4
# and 5 (the checker does 50-400 threads per second)
@pytest.mark.parametrize("config,samples", [(2, None), (3, None), (4, 410), (5, 704)])
def test_full_size_step(config, samples):
    from paper_2401_06761_b200.session import PagedSession, pool_requirements
    spec = synth.forest_spec(config)
    sess = PagedSession.for_spec(spec, extra_blocks=len(spec.nodes) + 64)
    _, nt, mb = pool_requirements(spec)
    model = BlockModel(sess.num_blocks, 16, nt, mb)
    both = WithModel(sess, model)
    step = synth.build_forest(spec, both, device="cuda")
    synth.run_step_forks(step, both)
    live = step.live_handles
    both.append(live, None, step.k_new, step.v_new)
    # tables, reference counts and free list of the whole pool, entry by entry
    assert_same_bookkeeping(sess, model, list(model.tables))
    assert sess.stats()["cow_blocks"] == model.cow_blocks
    assert sess.stats()["peak_used_blocks"] == model.peak_used
    out = sess.attention(live, step.q)
    out2 = sess.attention(live, step.q)          # the cached plan gives the same answer
    torch.cuda.synchronize()
    st = sess.stats()
    assert st["device_wait_timeouts"] == 0
    assert st["attn_plan_reused"] == 1 and torch.equal(out, out2)
    assert st["attn_attended_tokens"] == spec.unshared_tokens()
    # every logical token once, plus the (at most 15) rows each fork copied for its child
    assert spec.unique_tokens() <= st["attn_unique_tokens"] <= spec.unique_tokens() + 15 * st["forks"]
    assert torch.isfinite(out.float()).all()
    assert st["attn_unique_tokens"] == model.unique_tokens(live)
    nodes = step.live_nodes
    rng = np.random.default_rng(config)
    if samples is None:
        idx = list(range(len(nodes)))
    else:
        idx = sorted(set(np.linspace(0, len(nodes) - 1, samples // 2).astype(int).tolist()) |
                     set(rng.integers(0, len(nodes), samples // 2).tolist()))
    errs = []
    for i in idx:
        k, v = synth.chain_kv(spec, nodes[i], "cuda")
        assert sess.thread(live[i])[0] == k.shape[0]
        f = Forest(spec.shape.num_kv_heads, spec.shape.head_dim)
        t = f.new_thread()
        f.append(t, k.cpu().to(torch.float64).numpy(), v.cpu().to(torch.float64).numpy())
        ref = tree_decode_attention(f, [t], step.q[i:i + 1].cpu().to(torch.float64).numpy(),
                                    sess.sm_scale)
        errs.append(np.abs(out[i:i + 1].cpu().to(torch.float64).numpy() - ref))
    err = np.concatenate(errs)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())
    sess.close()

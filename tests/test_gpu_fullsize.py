"""Full-size workloads, in the launch configuration the benchmark times: the library builds
the whole forest, runs the decode step, and a seeded sample of threads (every region of the
request range represented) is checked against the CPU checker one thread at a time.  The
checker's inputs are regenerated from the seeds, never read back from the pool."""
import numpy as np
import pytest
import torch

from helpers import MAX_ABS, MEAN_ABS
from oracle import Forest, tree_decode_attention
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


# all threads of config 2, a fifth of config 3, a tenth of configs 4 and 5 (the checker does
# 50-400 threads per second)
@pytest.mark.parametrize("config,samples", [(2, 128), (3, 800), (4, 410), (5, 704)])
def test_full_size_step_sampled(config, samples):
    from paper_2401_06761_b200.session import PagedSession
    spec = synth.forest_spec(config)
    sess = PagedSession.for_spec(spec, extra_blocks=len(spec.nodes) + 64)
    step = synth.build_forest(spec, sess, device="cuda")
    synth.run_step_forks(step, sess)
    live = step.live_handles
    sess.append(live, None, step.k_new, step.v_new)
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
    nodes = step.live_nodes
    rng = np.random.default_rng(config)
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

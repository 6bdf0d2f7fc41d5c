"""Queries at arbitrary chain positions: the tree mask of training / prefill (Section 2.2), where
every token of every paragraph node attends its ancestors' tokens and, causally, its own."""
import numpy as np
import pytest
import torch

from helpers import OracleBackend, assert_close
from oracle import dense_attention
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4)])
def test_every_token_of_a_paragraph_tree(hq, hkv):
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession
    shape = synth.LayerShape(hq, hkv)
    sess = PagedSession(shape, 200, 700, 40, poison=True)
    orc = OracleBackend(shape, 200, 700, 40)
    g = torch.Generator(device="cuda").manual_seed(31)

    def rows(n):
        kv = torch.randn((2, n, hkv, 128), generator=g, device="cuda").to(torch.bfloat16)
        return kv[0].contiguous(), kv[1].contiguous()

    def both(fn, *a):
        x, y = getattr(sess, fn)(*a), getattr(orc, fn)(*a)
        return x

    # a paragraph tree: root 70 tokens, three children forked at its end (one of them again)
    (root,) = both("new_threads", 1)
    both("append", [root], [70], *rows(70))
    kids = both("fork", [root] * 3)
    for t, n in zip(kids, (33, 5, 48)):
        both("append", [t], [n], *rows(n))
    (grand,) = both("fork", [kids[2]])
    both("append", [grand], [21], *rows(21))
    both("append", [root], [9], *rows(9))          # the root goes on after the forks

    # one query per token of every node: (thread, position + 1); own tokens start at `first`
    tids, lens = [], []
    for t, first in ((root, 0), (kids[0], 70), (kids[1], 70), (kids[2], 70), (grand, 70 + 48)):
        total = sess.thread(t)[0]
        tids += [t] * (total - first)
        lens += list(range(first + 1, total + 1))
    q = torch.randn((len(tids), hq, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.prefix_attention(tids, lens, q)
    qq = q.cpu().to(torch.float64).numpy()
    ref = np.empty_like(qq)
    chains = {t: orc.forest.chain(orc.node_of[t]) for t in set(tids)}
    for i, (t, L) in enumerate(zip(tids, lens)):
        K, V = chains[t]
        ref[i] = dense_attention(qq[i], K[:L], V[:L], sess.sm_scale)
    assert_close(out, ref, "tree-masked attention at every position")
    st = sess.stats()
    assert st["attn_attended_tokens"] == sum(lens) and st["device_wait_timeouts"] == 0
    # decode attention is the special case attend_len = len
    live = [root] + kids + [grand]
    full = [sess.thread(t)[0] for t in live]
    qd = q[: len(live)].contiguous()
    assert torch.equal(sess.prefix_attention(live, full, qd), sess.attention(live, qd))
    for bad in ([0], [10 ** 6]):
        with pytest.raises(B.AparError):
            sess.prefix_attention([root], bad, qd[:1].contiguous())
    sess.close()

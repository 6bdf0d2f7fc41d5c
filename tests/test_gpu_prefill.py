"""Tree-masked attention over whole runs of tokens (prompt prefill and the training mask of
Section 2.2): every token of every node of a paragraph tree attends its ancestors' tokens and,
causally, its own node's.  Checked position by position against plain dense attention over
the first p + 1 rows of the thread's chain."""
import numpy as np
import pytest
import torch

from helpers import OracleBackend, assert_close
from oracle import dense_attention
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


def _tree(sess, orc, hkv, g, sizes):
    """root -> three children (the third one forks a grandchild); the root goes on afterwards.
    Returns [(thread, first own position)] in creation order."""
    def rows(n):
        kv = torch.randn((2, n, hkv, 128), generator=g, device="cuda").to(torch.bfloat16)
        return kv[0].contiguous(), kv[1].contiguous()

    def both(fn, *a):
        x = getattr(sess, fn)(*a)
        getattr(orc, fn)(*a)
        return x

    n_root, n_kids, n_grand, n_more = sizes
    (root,) = both("new_threads", 1)
    both("append", [root], [n_root], *rows(n_root))
    kids = both("fork", [root] * 3)
    for t, n in zip(kids, n_kids):
        both("append", [t], [n], *rows(n))
    (grand,) = both("fork", [kids[2]])
    both("append", [grand], [n_grand], *rows(n_grand))
    both("append", [root], [n_more], *rows(n_more))
    return [(root, 0), (kids[0], n_root), (kids[1], n_root), (kids[2], n_root),
            (grand, n_root + n_kids[2])]


def _check_all_positions(sess, orc, nodes, q, out):
    qq = q.cpu().to(torch.float64).numpy()
    ref = np.empty_like(qq)
    i = 0
    for t, first in nodes:
        K, V = orc.forest.chain(orc.node_of[t])
        for p in range(first, sess.thread(t)[0]):
            ref[i] = dense_attention(qq[i], K[:p + 1], V[:p + 1], sess.sm_scale)
            i += 1
    assert i == len(qq)
    return assert_close(out, ref, "tree-masked attention at every position")


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4), (64, 8), (6, 1), (2, 2)])
def test_every_token_of_a_paragraph_tree(hq, hkv):
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession
    shape = synth.LayerShape(hq, hkv)
    sess = PagedSession(shape, 200, 16, 40, poison=True)
    orc = OracleBackend(shape, 200, 16, 40)
    g = torch.Generator(device="cuda").manual_seed(31)
    nodes = _tree(sess, orc, hkv, g, (70, (33, 5, 48), 21, 9))
    tids = [t for t, _ in nodes]
    begins = [first for _, first in nodes]
    counts = [sess.thread(t)[0] - first for t, first in nodes]
    q = torch.randn((sum(counts), hq, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.prefill_attention(tids, begins, counts, q)
    _check_all_positions(sess, orc, nodes, q, out)
    st = sess.stats()
    assert st["attn_threads"] == sum(counts) and st["device_wait_timeouts"] == 0
    assert st["attn_attended_tokens"] == sum(b * c + c * (c + 1) // 2 for b, c in zip(begins, counts))
    # decode attention is the special case of one query at the last position
    live = tids
    qd = q[: len(live)].contiguous()
    last = [sess.thread(t)[0] - 1 for t in live]
    got = sess.prefill_attention(live, last, [1] * len(live), qd)
    ref = orc.attention(live, qd, sess.sm_scale)
    assert_close(got, ref, "last position = decode attention")
    for bad in (([tids[0]], [0], [10 ** 6]), ([tids[0]], [-1], [2]), ([tids[0]], [3], [0])):
        with pytest.raises(B.AparError) as e:
            sess.prefill_attention(*bad, qd[:1].contiguous())
        assert e.value.code == "INVALID_ARG"
    # the queries are read by TMA: an array that does not start on a 16-byte boundary is refused
    flat = torch.zeros(hq * 128 + 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.AparError) as e:
        sess.prefill_attention([tids[0]], [0], [1], flat[1:1 + hq * 128].view(1, hq, 128))
    assert e.value.code == "INVALID_ARG"
    sess.close()


def test_long_tree_in_batches_and_second_layer():
    """More than two thousand tokens in nodes of many tiles, and the same mask on a second pool
    layer."""
    from paper_2401_06761_b200.session import PagedSession
    hq, hkv = 8, 2
    shape = synth.LayerShape(hq, hkv)
    sess = PagedSession(shape, 400, 40, 160, poison=True, num_layers=2)
    orc = OracleBackend(shape, 400, 40, 160)
    g = torch.Generator(device="cuda").manual_seed(5)
    nodes = _tree(sess, orc, hkv, g, (1500, (210, 330, 170), 260, 40))
    tids = [t for t, _ in nodes]
    begins = [first for _, first in nodes]
    counts = [sess.thread(t)[0] - first for t, first in nodes]
    assert sum(counts) > 2400
    q = torch.randn((sum(counts), hq, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.prefill_attention(tids, begins, counts, q)
    _check_all_positions(sess, orc, nodes, q, out)
    # layer 1 holds other rows (layer 0's, negated): same mask, other result
    sess.k_pool[400:].copy_(-sess.k_pool[:400])
    sess.v_pool[400:].copy_(-sess.v_pool[:400])
    out1 = sess.prefill_attention(tids, begins, counts, q, layer=1)
    torch.cuda.synchronize()
    # softmax(-s) over -V: checked through the checker on negated rows for one node
    t, first = nodes[4]
    K, V = orc.forest.chain(orc.node_of[t])
    qq = q.cpu().to(torch.float64).numpy()
    base = sum(counts[:4])
    ref = np.stack([dense_attention(qq[base + j], -K[:first + j + 1], -V[:first + j + 1],
                                    sess.sm_scale) for j in range(counts[4])])
    assert_close(out1[base:base + counts[4]], ref, "layer 1")
    assert sess.stats()["device_wait_timeouts"] == 0
    sess.close()


def test_batches_when_the_work_list_is_split(monkeypatch):
    """A 10 000-token prompt with one query head: 40 work items of 256 tokens, here limited to
    16 per launch (the limit that applies otherwise, the size of the work-list area, is out of
    reach of a test)."""
    from paper_2401_06761_b200.session import PagedSession
    monkeypatch.setenv("APAR_PREFILL_BATCH", "16")
    shape = synth.LayerShape(1, 1)
    sess = PagedSession(shape, 700, 4, 640, poison=True)
    orc = OracleBackend(shape, 700, 4, 640)
    g = torch.Generator(device="cuda").manual_seed(17)
    n = 10000
    kv = torch.randn((2, n, 1, 128), generator=g, device="cuda").to(torch.bfloat16)
    (t,) = sess.new_threads(1)
    orc.new_threads(1)
    sess.append([t], [n], kv[0].contiguous(), kv[1].contiguous())
    orc.append([t], [n], kv[0], kv[1])
    q = torch.randn((n, 1, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.prefill_attention([t], [0], [n], q)
    assert sess.stats()["attn_kernels"] == 3
    K, V = orc.forest.chain(orc.node_of[t])
    qq = q.cpu().to(torch.float64).numpy()
    pick = list(range(0, n, 37)) + [n - 1, 9471, 9472, 9473, 4095, 4096, 127, 128, 255, 256]
    ref = np.stack([dense_attention(qq[p], K[:p + 1], V[:p + 1], sess.sm_scale) for p in pick])
    assert_close(out[pick], ref, "sampled positions of a 10 000-token prompt")
    assert sess.stats()["device_wait_timeouts"] == 0
    sess.close()

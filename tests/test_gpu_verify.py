"""Predict-verify with tree attention among speculated tokens (the paper's Medusa setting):
the candidates of a thread are appended once to its own tail, each candidate is a query with a
mask over the candidates, and accepted candidates are moved up behind the committed rows.

The checker has no such operation and needs none: a candidate that sees its ancestors among the
candidates is a thread forked from its parent candidate (oracle.Forest), and an arbitrary mask
is dense attention over the gathered rows."""
import numpy as np
import pytest
import torch

from helpers import OracleBackend, assert_close, assert_same_bookkeeping
from oracle import dense_attention, tree_decode_attention
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


def medusa_tree(top_k):
    """Parents of a candidate tree: the model's own next token, then the top-k guesses of each
    extra head below every node of the level before.  top_k = (3, 2) -> 1 + 3 + 6 nodes."""
    parents, level = [-1], [0]
    for k in top_k:
        nxt = []
        for p in level:
            for _ in range(k):
                parents.append(p)
                nxt.append(len(parents) - 1)
        level = nxt
    return parents


def masks_of(parents):
    masks = []
    for j, p in enumerate(parents):
        masks.append((1 << j) | (masks[p] if p >= 0 else 0))
    return masks


def _rand(shape, g):
    return torch.randn(shape, generator=g, device="cuda").to(torch.bfloat16)


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4), (64, 8)])
def test_candidate_trees_accept_and_next_step(hq, hkv):
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession
    shape = synth.LayerShape(hq, hkv)
    sess = PagedSession(shape, 400, 300, 40, poison=True)
    orc = OracleBackend(shape, 400, 300, 40)
    g = torch.Generator(device="cuda").manual_seed(hq)

    def rows(n):
        return _rand((n, hkv, 128), g), _rand((n, hkv, 128), g)

    def both(fn, *a):
        x, y = getattr(sess, fn)(*a), getattr(orc, fn)(*a)
        if fn in ("new_threads", "fork"):
            assert x == y
        return x

    # a request of 150 prompt tokens forked into three threads, and an unforked thread
    root, solo = both("new_threads", 2)
    both("append", [root, solo], [150, 43], *rows(193))
    kids = both("fork", [root] * 3)
    both("append", kids, [9, 30, 18], *rows(57))
    threads = kids + [solo]
    trees = [medusa_tree((3, 2)), medusa_tree((2, 2)), medusa_tree((4,)), medusa_tree((2, 3))]
    n_cand = [len(t) for t in trees]
    base = [sess.thread(t)[0] for t in threads]

    # expected: every candidate as a thread forked from its parent candidate, in the checker only
    cand_rows = [rows(k) for k in n_cand]
    cand_node = []
    for t, parents, (ck, cv) in zip(threads, trees, cand_rows):
        nodes = []
        for j, p in enumerate(parents):
            node = orc.forest.fork(nodes[p] if p >= 0 else orc.node_of[t])
            orc.forest.append(node, ck[j:j + 1].cpu().to(torch.float64).numpy(),
                              cv[j:j + 1].cpu().to(torch.float64).numpy())
            nodes.append(node)
        cand_node += nodes
    q = _rand((sum(n_cand), hq, 128), g)
    ref = tree_decode_attention(orc.forest, cand_node, q.cpu().to(torch.float64).numpy(),
                                sess.sm_scale)

    # the library: candidates appended once to each thread's own tail (pool model follows)
    sess.append(threads, n_cand, torch.cat([r[0] for r in cand_rows]),
                torch.cat([r[1] for r in cand_rows]))
    orc.model.append(threads, n_cand)
    masks = [m for t in trees for m in masks_of(t)]
    out = sess.verify_attention(threads, n_cand, masks, q)
    assert_close(out, ref, "candidate trees")
    st = sess.stats()
    assert st["attn_attended_tokens"] == sum(
        b * k for b, k in zip(base, n_cand)) + sum(bin(m).count("1") for m in masks)
    assert_same_bookkeeping(sess, orc.model, list(orc.model.tables))

    # bad masks are refused
    for bad in ([masks[0] & ~1] + masks[1:], [masks[0] | (1 << 40)] + masks[1:]):
        with pytest.raises(B.AparError) as e:
            sess.verify_attention(threads, n_cand, bad, q)
        assert e.value.code == "INVALID_ARG"

    # accept one root-to-leaf path per thread (the last thread keeps nothing but the first token)
    keep = [[0, 2, 6], [0, 1, 4], [0, 3], [0]]
    sess.accept(threads, n_cand, keep)
    orc.model.accept(threads, n_cand, [len(k) for k in keep])
    for t, (ck, cv), idx in zip(threads, cand_rows, keep):
        orc.forest.append(orc.node_of[t], ck[idx].cpu().to(torch.float64).numpy(),
                          cv[idx].cpu().to(torch.float64).numpy())
    assert_same_bookkeeping(sess, orc.model, list(orc.model.tables))
    assert [sess.thread(t)[0] for t in threads] == [b + len(k) for b, k in zip(base, keep)]
    # the next decode step sees the accepted rows in place and nothing of the rejected ones
    k1, v1 = rows(len(threads))
    q1 = _rand((len(threads), hq, 128), g)
    out1 = sess.decode_step(threads, k1, v1, q1)
    orc.append(threads, None, k1, v1)
    assert_close(out1, orc.attention(threads, q1, sess.sm_scale), "step after accept")
    assert_same_bookkeeping(sess, orc.model, list(orc.model.tables))
    assert sess.stats()["device_wait_timeouts"] == 0
    sess.close()


def test_arbitrary_masks_no_prefix_and_other_layers():
    """Masks that are not trees, a thread whose every row is a candidate, 64 candidates, and the
    same verification replayed on a second layer."""
    from paper_2401_06761_b200.session import PagedSession
    hq, hkv = 8, 2
    shape = synth.LayerShape(hq, hkv)
    sess = PagedSession(shape, 64, 80, 12, poison=True, num_layers=2)
    g = torch.Generator(device="cuda").manual_seed(3)
    rng = np.random.default_rng(3)
    a, b = sess.new_threads(2)
    ctx_a = 21
    n_cand = [64, 7]
    rows = [[_rand((n, hkv, 128), g) for n in (ctx_a + 64, 7)] for _ in range(4)]   # k0 v0 k1 v1
    for layer in range(2):
        k, v = torch.cat(rows[2 * layer]), torch.cat(rows[2 * layer + 1])
        if layer == 0:
            sess.append([a, b], [ctx_a + 64, 7], k, v)
        else:
            sess.append_layer(1, k, v)
    masks = []
    for k in n_cand:
        for j in range(k):
            m = int(rng.integers(0, 2 ** 63)) & ((1 << k) - 1) | (1 << j)
            masks.append(m)
    q = [_rand((sum(n_cand), hq, 128), g) for _ in range(2)]
    out = [sess.verify_attention([a, b], n_cand, masks, q[0]), None]
    out[1] = sess.attention_layer(1, q[1])
    for layer in range(2):
        K = [t.cpu().to(torch.float64).numpy() for t in rows[2 * layer]]
        V = [t.cpu().to(torch.float64).numpy() for t in rows[2 * layer + 1]]
        qq = q[layer].cpu().to(torch.float64).numpy()
        ref = np.empty_like(qq)
        i = 0
        for th, (k, base) in enumerate(zip(n_cand, (ctx_a, 0))):
            for j in range(k):
                sel = list(range(base)) + [base + x for x in range(k) if (masks[i] >> x) & 1]
                ref[i] = dense_attention(qq[i], K[th][sel], V[th][sel], sess.sm_scale)
                i += 1
        assert_close(out[layer], ref, f"layer {layer}")
    assert sess.stats()["device_wait_timeouts"] == 0
    sess.close()

"""Pins for the fp64 attention checker: each test reaches the expected value by a route
that does not pass through the checker's own code."""
import math

import numpy as np
import pytest
import torch

from oracle import Forest, dense_attention, softmax_weights, tree_decode_attention

D = 128


def _rand(rng, *shape):
    return rng.standard_normal(shape)


def test_hand_computed_two_keys():
    # s = scale * q.k = [ln 2, 0]  ->  p = [2/3, 1/3]; worked by hand.
    scale = 0.5
    q = np.array([[1.0, 0.0]])
    K = np.array([[[2 * math.log(2.0), 5.0]], [[0.0, -3.0]]])      # [L=2][Hkv=1][D=2]
    V = np.array([[[3.0, -6.0]], [[9.0, 12.0]]])
    o = dense_attention(q, K, V, scale)
    np.testing.assert_allclose(o, [[2 / 3 * 3 + 1 / 3 * 9, 2 / 3 * -6 + 1 / 3 * 12]],
                               rtol=0, atol=1e-14)
    np.testing.assert_allclose(softmax_weights(q[0], K[:, 0], scale), [2 / 3, 1 / 3],
                               atol=1e-15)


def test_single_thread_equals_causal_decode_library_routine():
    # A tree with one thread is ordinary causal decoding: the new token is the last row of
    # causal attention over the sequence.  The library routine decides here.
    rng = np.random.default_rng(1)
    L, Hq, Hkv = 37, 4, 4
    k, v = _rand(rng, L, Hkv, D), _rand(rng, L, Hkv, D)
    qs = _rand(rng, L, Hq, D)          # a query per position; only the last one is decoded
    scale = 1 / math.sqrt(D)
    f = Forest(Hkv, D)
    t = f.new_thread()
    f.append(t, k[:20], v[:20])
    f.append(t, k[20:], v[20:])
    got = tree_decode_attention(f, [t], qs[-1:], scale)[0]
    tq = torch.from_numpy(qs).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True,
                                                           scale=scale)
    np.testing.assert_allclose(got, ref[0, :, -1, :].numpy(), rtol=0, atol=1e-12)


def test_gqa_head_mapping_via_library_routine():
    rng = np.random.default_rng(2)
    L, Hq, Hkv = 19, 8, 2
    k, v, q = _rand(rng, L, Hkv, D), _rand(rng, L, Hkv, D), _rand(rng, Hq, D)
    got = dense_attention(q, k, v, 0.11)
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)[None]
    tq = torch.from_numpy(q)[None, :, None, :]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.11)
    np.testing.assert_allclose(got, ref[0, :, 0].numpy(), rtol=0, atol=1e-12)
    # and directly: V of kv head g constant g  ->  o[h] = h // group
    vc = np.broadcast_to(np.arange(Hkv, dtype=float)[None, :, None], v.shape)
    o = dense_attention(q, k, vc, 0.11)
    np.testing.assert_allclose(o, np.repeat([0.0, 1.0], 4)[:, None] * np.ones((1, D)),
                               atol=1e-13)


def _build_random_tree(rng, Hkv, events):
    """Replays (op, arg) events on a Forest and, independently, on a flat token log:
    every token records (owner thread, K row, V row); visibility is rebuilt from
    per-token parent links, not from the Forest."""
    f = Forest(Hkv, D)
    tok_k, tok_v, tok_prev = [], [], []     # flat log; tok_prev = previous token on path
    last_tok = {}                           # thread -> its newest token (or inherited one)
    for op, arg in events:
        if op == "new":
            t = f.new_thread()
            last_tok[t] = -1
        elif op == "fork":
            t = f.fork(arg)
            last_tok[t] = last_tok[arg]
        else:
            t, n = arg
            k, v = _rand(rng, n, Hkv, D), _rand(rng, n, Hkv, D)
            f.append(t, k, v)
            for i in range(n):
                tok_k.append(k[i]); tok_v.append(v[i]); tok_prev.append(last_tok[t])
                last_tok[t] = len(tok_k) - 1
    return f, np.array(tok_k), np.array(tok_v), tok_prev, last_tok


def _brute_force(tok_k, tok_v, tok_prev, last, q, scale, group):
    """Dense masked softmax over *all* tokens of the forest with a boolean ancestor mask."""
    n = len(tok_prev)
    mask = np.zeros(n, dtype=bool)
    j = last
    while j >= 0:
        mask[j] = True
        j = tok_prev[j]
    out = np.zeros_like(q)
    for h in range(q.shape[0]):
        s = scale * np.einsum("jd,d->j", tok_k[:, h // group], q[h])
        s = np.where(mask, s, -np.inf)
        e = np.exp(s - s[mask].max())
        out[h] = (e / e.sum()) @ tok_v[:, h // group]
    return out


def test_tree_equals_bruteforce_over_masked_global_tokens():
    rng = np.random.default_rng(3)
    Hq, Hkv = 4, 2
    events = [("new", None), ("app", (0, 21)), ("fork", 0), ("fork", 0), ("app", (1, 5)),
              ("app", (0, 9)),            # the parent goes on after forking
              ("app", (2, 18)), ("fork", 2), ("app", (3, 1)), ("app", (2, 2)),
              ("new", None), ("app", (4, 3)), ("fork", 4), ("app", (5, 7)), ("fork", 1),
              ("app", (6, 4))]
    f, tk, tv, prev, last = _build_random_tree(rng, Hkv, events)
    threads = [0, 1, 2, 3, 4, 5, 6]
    q = _rand(rng, len(threads), Hq, D)
    scale = 1 / math.sqrt(D)
    got = tree_decode_attention(f, threads, q, scale)
    for i, t in enumerate(threads):
        ref = _brute_force(tk, tv, prev, last[t], q[i], scale, Hq // Hkv)
        np.testing.assert_allclose(got[i], ref, rtol=0, atol=1e-12)
    # attended tokens = length of the path to the root (Section 3.4 definition)
    assert [f.length(t) for t in threads] == [30, 26, 41, 40, 3, 10, 30]


def test_weights_sum_to_one_and_output_in_value_range():
    rng = np.random.default_rng(4)
    k, v, q = _rand(rng, 300, 1, D) * 3, _rand(rng, 300, 1, D), _rand(rng, 1, D) * 3
    p = softmax_weights(q[0], k[:, 0], 0.7)
    assert abs(p.sum() - 1) < 1e-12 and (p >= 0).all()
    o = dense_attention(q, k, v, 0.7)[0]
    assert (o <= v[:, 0].max(0) + 1e-12).all() and (o >= v[:, 0].min(0) - 1e-12).all()


def test_closed_forms():
    rng = np.random.default_rng(5)
    L, Hq, Hkv = 50, 2, 1
    k, v, q = _rand(rng, L, Hkv, D), _rand(rng, L, Hkv, D), _rand(rng, Hq, D)
    # zero query -> uniform weights -> mean of V
    np.testing.assert_allclose(dense_attention(np.zeros((Hq, D)), k, v, 1.0),
                               np.broadcast_to(v[:, 0].mean(0), (Hq, D)), atol=1e-13)
    # all keys equal -> mean of V
    ke = np.broadcast_to(k[:1], k.shape)
    np.testing.assert_allclose(dense_attention(q, ke, v, 1.0),
                               np.broadcast_to(v[:, 0].mean(0), (Hq, D)), atol=1e-12)
    # constant V -> that constant
    vc = np.full_like(v, 2.5)
    np.testing.assert_allclose(dense_attention(q, k, vc, 1.0), 2.5, atol=1e-13)
    # one dominating key -> its V row
    kd = k.copy(); kd[17, 0] = 100 * q[0]
    np.testing.assert_allclose(dense_attention(q[:1], kd, v, 1.0)[0], v[17, 0], atol=1e-9)
    # a single token -> its V row, whatever the query
    np.testing.assert_allclose(dense_attention(q, k[:1], v[:1], 1.0),
                               np.broadcast_to(v[0, 0], (Hq, D)), atol=0)
    with pytest.raises(ValueError):
        dense_attention(q, k[:0], v[:0], 1.0)


def test_sibling_isolation_and_shared_ancestor():
    rng = np.random.default_rng(6)
    Hq = Hkv = 2

    def build(sib_rows, root_rows):
        f = Forest(Hkv, D)
        r = f.new_thread(); f.append(r, *root_rows)
        a = f.fork(r); b = f.fork(r)
        f.append(a, *a_rows); f.append(b, *sib_rows)
        return f, a, b

    root_rows = (_rand(rng, 10, Hkv, D), _rand(rng, 10, Hkv, D))
    a_rows = (_rand(rng, 4, Hkv, D), _rand(rng, 4, Hkv, D))
    b1 = (_rand(rng, 6, Hkv, D), _rand(rng, 6, Hkv, D))
    b2 = (_rand(rng, 6, Hkv, D), _rand(rng, 6, Hkv, D))
    q = _rand(rng, 2, Hq, D)
    f1, a, b = build(b1, root_rows)
    f2, _, _ = build(b2, root_rows)
    o1 = tree_decode_attention(f1, [a, b], q, 0.1)
    o2 = tree_decode_attention(f2, [a, b], q, 0.1)
    assert np.array_equal(o1[0], o2[0])          # a never sees its sibling's tokens
    assert not np.allclose(o1[1], o2[1])
    root2 = (root_rows[0].copy(), root_rows[1].copy()); root2[1][3] += 1.0
    f3, _, _ = build(b1, root2)
    o3 = tree_decode_attention(f3, [a, b], q, 0.1)
    assert not np.allclose(o1[0], o3[0]) and not np.allclose(o1[1], o3[1])


def test_child_does_not_see_parent_tokens_appended_after_the_fork():
    rng = np.random.default_rng(7)
    Hq = Hkv = 1
    f = Forest(Hkv, D)
    p = f.new_thread(); f.append(p, _rand(rng, 5, 1, D), _rand(rng, 5, 1, D))
    c = f.fork(p)
    f.append(p, _rand(rng, 3, 1, D), _rand(rng, 3, 1, D))
    f.append(c, _rand(rng, 2, 1, D), _rand(rng, 2, 1, D))
    assert f.length(c) == 7 and f.length(p) == 8
    Kc, _ = f.chain(c); Kp, _ = f.chain(p)
    assert np.array_equal(Kc[:5], Kp[:5]) and not np.array_equal(Kc[5], Kp[5])

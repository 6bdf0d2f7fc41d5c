"""fp64 dense softmax attention over a thread's path to the root.

Test infrastructure only (see oracle/__init__).  The method computes, exactly up to
rounding, ordinary softmax attention over a restricted key set: a new token attends only
to the tokens on its path to the root of the paragraph tree, itself included (Section 2.2
"Training attention"; Section 2.4 feature 3).  So this file is that definition written
out, with no blocking, no online softmax and no sharing between threads.
"""
from __future__ import annotations

import numpy as np


def softmax_weights(q_h, K_g, sm_scale):
    """p_j = exp(s_j - max s) / sum, s_j = sm_scale * <q_h, K_g[j]>.  q_h [D], K_g [L][D]."""
    s = sm_scale * (K_g @ q_h)
    e = np.exp(s - s.max())
    return e / e.sum()


def dense_attention(q, K, V, sm_scale):
    """q [H_q][D]; K, V [L][H_kv][D] (fp64).  Query head h reads KV head h // (H_q/H_kv).
    Returns o [H_q][D] with o[h] = sum_j p_j V[j][g]."""
    q = np.asarray(q, dtype=np.float64)
    num_q_heads, _ = q.shape
    length, num_kv_heads, _ = K.shape
    if length == 0:
        raise ValueError("attention over an empty context is undefined")
    group = num_q_heads // num_kv_heads
    o = np.empty_like(q)
    for h in range(num_q_heads):
        g = h // group
        p = softmax_weights(q[h], K[:, g, :], sm_scale)
        o[h] = p @ V[:, g, :]
    return o


def tree_decode_attention(forest, threads, q, sm_scale):
    """One decode step: query i belongs to threads[i] and sees exactly that thread's chain.
    q [n][H_q][D] -> out [n][H_q][D] fp64."""
    q = np.asarray(q, dtype=np.float64)
    out = np.empty_like(q)
    for i, t in enumerate(threads):
        K, V = forest.chain(t)
        out[i] = dense_attention(q[i], K, V, sm_scale)
    return out

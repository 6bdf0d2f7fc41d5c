"""Logical store of generation threads.  Test infrastructure only (see oracle/__init__).

A thread is a sequence of Algorithm 1.  It knows its parent, how many of the parent's
tokens it inherited when it was forked, and the (k, v) rows appended to it since.  There
are no blocks here: the visible tokens of a thread are *defined* as its path to the root
(Section 2.2 "Training attention"; Section 2.4 feature 3; Fig. 2 caption).
"""
from __future__ import annotations

import numpy as np


class Forest:
    def __init__(self, num_kv_heads: int, head_dim: int):
        self.num_kv_heads = num_kv_heads
        self.head_dim = head_dim
        self.parent = []          # thread -> parent thread or -1
        self.inherited = []       # thread -> tokens of the parent's chain it shares
        self.k_rows = []          # thread -> list of fp64 arrays [n][H_kv][D]
        self.v_rows = []

    def new_thread(self) -> int:
        """A prompt sequence: no parent (the initial member of Algorithm 1's sequence group)."""
        self.parent.append(-1)
        self.inherited.append(0)
        self.k_rows.append([])
        self.v_rows.append([])
        return len(self.parent) - 1

    def length(self, t: int) -> int:
        """Attended tokens of thread t = tokens on its path to the root (Section 3.4)."""
        return self.inherited[t] + sum(a.shape[0] for a in self.k_rows[t])

    def fork(self, p: int) -> int:
        """The sequence duplication of Algorithm 1: the child shares every token the parent has now."""
        t = self.new_thread()
        self.parent[t] = p
        self.inherited[t] = self.length(p)
        return t

    def append(self, t: int, k, v) -> None:
        """Token append of Algorithm 1: rows [n][H_kv][D] produced for thread t's new tokens."""
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        assert k.shape == v.shape and k.shape[1:] == (self.num_kv_heads, self.head_dim)
        self.k_rows[t].append(k)
        self.v_rows[t].append(v)

    def chain(self, t: int):
        """K, V of every token thread t may attend to, root first: [L][H_kv][D] fp64."""
        shape = (0, self.num_kv_heads, self.head_dim)
        if self.parent[t] >= 0:
            pk, pv = self.chain(self.parent[t])
            ks, vs = [pk[: self.inherited[t]]], [pv[: self.inherited[t]]]
        else:
            ks, vs = [np.zeros(shape)], [np.zeros(shape)]
        ks += self.k_rows[t]
        vs += self.v_rows[t]
        return np.concatenate(ks, 0), np.concatenate(vs, 0)

"""Seeded synthetic workloads: paragraph-tree shapes and Q/K/V values.

This module only *describes inputs*: which generation threads exist, who forked from whom
and how many tokens each one holds, plus the random bf16 rows that stand for the
(already rotated) keys, values and queries a model would have produced.  It contains none
of the method's arithmetic (no attention, no block bookkeeping), so the CUDA path and the
CPU checker can both be fed from it without sharing any of their own code.

The five tree shapes stand in for the paper's serving workloads (Vicuna Bench, MT Bench
and the ShareGPT-derived APAR test set, Section 3.2 "Evaluation datasets"), which need the
fine-tuned models to turn prompts into paragraph trees.  A tree here is what Algorithm 1
would have produced up to one decode step: a prompt sequence, the threads forked from it
(Section 2.3 "Decoding"), optionally threads forked from those.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

BLOCK_SIZE = 16
HEAD_DIM = 128


@dataclass(frozen=True)
class LayerShape:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int = HEAD_DIM
    block_size: int = BLOCK_SIZE

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def bytes_per_token(self) -> int:
        # one token's K row and V row over all KV heads, bf16
        return 2 * self.num_kv_heads * self.head_dim * 2


LAYER_SHAPES = {
    1: LayerShape(8, 2),     # single request, GQA 8/2
    2: LayerShape(32, 32),   # 7B-like MHA
    3: LayerShape(40, 40),   # 13B-like MHA
    4: LayerShape(64, 8),    # 70B-like GQA
    5: LayerShape(32, 8),    # high-throughput mix, GQA 32/8
}

DEFAULT_REQUESTS = {1: 1, 2: 32, 3: 256, 4: 512, 5: 2048}


@dataclass
class Node:
    """One generation thread (a sequence of Algorithm 1) of the synthetic forest.

    n_tok counts the KV rows the thread itself owns when the measured decode step attends:
    for a live leaf that includes the token appended in that step.
    """
    index: int
    parent: int            # -1 for a prompt sequence
    request: int
    depth: int
    n_tok: int
    live: bool             # takes part in the measured decode step (a leaf)
    step_fork: bool = False  # created by the fork that belongs to the measured step
    children: List[int] = field(default_factory=list)


@dataclass
class ForestSpec:
    config: int
    seed: int
    shape: LayerShape
    nodes: List[Node]

    # ---- derived counts (pure tree arithmetic on the spec, used for sizing only) ----
    def live_nodes(self) -> List[Node]:
        return [n for n in self.nodes if n.live]

    def chain(self, node: Node) -> List[Node]:
        out = []
        cur: Optional[Node] = node
        while cur is not None:
            out.append(cur)
            cur = self.nodes[cur.parent] if cur.parent >= 0 else None
        return out[::-1]

    def attended_tokens(self, node: Node) -> int:
        return sum(n.n_tok for n in self.chain(node))

    def unique_tokens(self) -> int:
        return sum(n.n_tok for n in self.nodes)

    def unshared_tokens(self) -> int:
        return sum(self.attended_tokens(n) for n in self.live_nodes())


def default_seed(config: int, k: int = 0) -> int:
    return 1000 * config + k


def _lognormal_int(rng, median, sigma, lo, hi, size=None):
    x = rng.lognormal(mean=math.log(median), sigma=sigma, size=size)
    return np.clip(np.rint(x), lo, hi).astype(np.int64)


def forest_spec(config: int, seed: Optional[int] = None,
                n_requests: Optional[int] = None) -> ForestSpec:
    """Tree shapes of workload `config` (1..5); `n_requests` shrinks it for tests."""
    if config not in LAYER_SHAPES:
        raise ValueError(f"unknown config {config}")
    seed = default_seed(config) if seed is None else seed
    nreq = DEFAULT_REQUESTS[config] if n_requests is None else n_requests
    rng = np.random.default_rng(seed)
    nodes: List[Node] = []

    def add(parent, request, depth, n_tok, live, step_fork=False):
        n = Node(len(nodes), parent, request, depth, int(n_tok), live, step_fork)
        nodes.append(n)
        if parent >= 0:
            nodes[parent].children.append(n.index)
        return n.index

    for r in range(nreq):
        if config == 1:
            p = add(-1, r, 0, 64, False)
            for n_tok in (32, 17, 40):
                add(p, r, 1, n_tok, True)
        elif config == 2:
            p = add(-1, r, 0, 512, False)
            for n_tok in rng.integers(128, 257, size=4):
                add(p, r, 1, n_tok, True)
        elif config == 3:
            p = add(-1, r, 0, rng.integers(128, 1025), False)
            b1 = int(rng.integers(2, 9))
            for _ in range(b1):
                n_tok = rng.integers(32, 257)
                if rng.random() < 0.5:
                    c = add(p, r, 1, n_tok, False)
                    b2 = int(rng.integers(2, 9))
                    lens = rng.integers(32, 257, size=b2)
                    for j in range(b2):
                        last = j == b2 - 1
                        # the last grandchild is forked inside the measured step and
                        # therefore attends with a branch of exactly one token
                        add(c, r, 2, 1 if last else lens[j], True, step_fork=last)
                else:
                    add(p, r, 1, n_tok, True)
        elif config == 4:
            p = add(-1, r, 0, 2048, False)
            for n_tok in rng.integers(128, 513, size=8):
                add(p, r, 1, n_tok, True)
        elif config == 5:
            plen = int(_lognormal_int(rng, 256, 0.8, 1, 4096))
            if rng.random() < 0.6:
                p = add(-1, r, 0, plen, False)
                k = int(rng.integers(2, 9))
                for n_tok in _lognormal_int(rng, 96, 0.8, 1, 4096, size=k):
                    add(p, r, 1, n_tok, True)
            else:
                blen = int(_lognormal_int(rng, 384, 0.8, 1, 4096))
                add(-1, r, 0, plen + blen, True)
    return ForestSpec(config, seed, LAYER_SHAPES[config], nodes)


def unshared_spec(spec: ForestSpec) -> ForestSpec:
    """Same live threads, but each one owns a private copy of its whole ancestor chain
    (the copy-the-prefix-on-fork policy of the paper's Appendix C.1)."""
    nodes = []
    for n in spec.live_nodes():
        nodes.append(Node(len(nodes), -1, n.request, 0, spec.attended_tokens(n), True))
    return ForestSpec(spec.config, spec.seed, spec.shape, nodes)


# ------------------------------------------------------------------ values

def _gen(seed: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1_000_003 + stream * 7919 + 12345) % (2 ** 63 - 1))
    return g


def node_kv(spec: ForestSpec, node: Node, device="cpu"):
    """K and V rows owned by `node`: two bf16 tensors [n_tok][H_kv][D], N(0,1)."""
    s = spec.shape
    g = _gen(spec.seed, 2 * node.index + 1, device)
    kv = torch.randn((2, node.n_tok, s.num_kv_heads, s.head_dim), generator=g,
                     device=device, dtype=torch.float32).to(torch.bfloat16)
    return kv[0], kv[1]


def chain_kv(spec: ForestSpec, node: Node, device="cpu"):
    """K and V rows of the whole root-to-node chain, concatenated in chain order."""
    ks, vs = zip(*(node_kv(spec, n, device) for n in spec.chain(node)))
    return torch.cat(ks, 0), torch.cat(vs, 0)


def queries(spec: ForestSpec, n: int, device="cpu") -> torch.Tensor:
    """One query row per live thread: bf16 [n][H_q][D], N(0,1)."""
    s = spec.shape
    g = _gen(spec.seed, 0, device)
    return torch.randn((n, s.num_q_heads, s.head_dim), generator=g, device=device,
                       dtype=torch.float32).to(torch.bfloat16)


# ------------------------------------------------------------------ replay

@dataclass
class StepInputs:
    """What one measured decode step consumes, in call order."""
    fork_parents: list          # handles of the threads forked inside the step
    fork_nodes: List[Node]
    live_nodes: List[Node]      # one query each, in this order
    live_handles: list
    k_new: torch.Tensor         # [T][H_kv][D] rows appended in the step
    v_new: torch.Tensor
    q: torch.Tensor             # [T][H_q][D]
    handles: dict               # node index -> backend handle


def build_forest(spec: ForestSpec, backend, device="cpu",
                 batch_bytes: int = 256 << 20) -> StepInputs:
    """Replay the setup of `spec` on `backend` (anything with new_threads / fork / append)
    and return the inputs of the measured step.

    Setup order: all prompt sequences, then level by level: fork the children, append
    their tokens.  Live leaves receive all but their last token; the step appends it.
    Nodes flagged step_fork are not created here: the step forks them.
    """
    s = spec.shape
    handles: dict = {}
    row_bytes = s.num_kv_heads * s.head_dim * 2

    def append_nodes(group: Sequence[Node]):
        batch, counts, ks, vs, size = [], [], [], [], 0

        def flush():
            nonlocal batch, counts, ks, vs, size
            if batch:
                backend.append([handles[n.index] for n in batch], counts,
                               torch.cat(ks, 0), torch.cat(vs, 0))
            batch, counts, ks, vs, size = [], [], [], [], 0

        for n in group:
            cnt = n.n_tok - 1 if n.live else n.n_tok
            if cnt <= 0:
                continue
            k, v = node_kv(spec, n, device)
            batch.append(n); counts.append(cnt); ks.append(k[:cnt]); vs.append(v[:cnt])
            size += cnt * row_bytes
            if size >= batch_bytes:
                flush()
        flush()

    roots = [n for n in spec.nodes if n.parent < 0]
    for n, h in zip(roots, backend.new_threads(len(roots))):
        handles[n.index] = h
    append_nodes(roots)
    level = roots
    while level:
        kids = [spec.nodes[c] for n in level for c in n.children
                if not spec.nodes[c].step_fork]
        if kids:
            for n, h in zip(kids, backend.fork([handles[n.parent] for n in kids])):
                handles[n.index] = h
            append_nodes(kids)
        level = kids

    fork_nodes = [n for n in spec.nodes if n.step_fork]
    live = spec.live_nodes()
    k_rows, v_rows = [], []
    for n in live:
        k, v = node_kv(spec, n, device)
        k_rows.append(k[n.n_tok - 1:]); v_rows.append(v[n.n_tok - 1:])
    return StepInputs(
        fork_parents=[handles[n.parent] for n in fork_nodes],
        fork_nodes=fork_nodes,
        live_nodes=live,
        live_handles=[handles.get(n.index) for n in live],
        k_new=torch.cat(k_rows, 0).contiguous(),
        v_new=torch.cat(v_rows, 0).contiguous(),
        q=queries(spec, len(live), device),
        handles=handles,
    )


def run_step_forks(step: StepInputs, backend) -> None:
    """Perform the fork that belongs to the measured step and fill in the new handles."""
    if step.fork_nodes:
        for n, h in zip(step.fork_nodes, backend.fork(step.fork_parents)):
            step.handles[n.index] = h
        step.live_handles = [step.handles[n.index] for n in step.live_nodes]


# ------------------------------------------------------------------ request lifecycle replay

@dataclass
class LifecycleStep:
    """Events of one decode step, in the order of Algorithm 1: new requests are admitted, threads
    whose last token was the fork token are duplicated, every live thread appends one token (and
    attends), threads that produced the end token finish."""
    arrive: List[tuple] = field(default_factory=list)   # (thread key, request, prompt length)
    fork: List[tuple] = field(default_factory=list)     # (parent key, child key)
    finish: List[int] = field(default_factory=list)     # thread keys


def lifecycle_schedule(seed: int, n_requests: int, n_steps: int, max_live: int = 48):
    """A token-free replay of Algorithm 1 for a stream of requests: which thread forks and which
    one finishes at which step.  Thread keys are small integers private to the schedule.
    Returns (steps, request_of_thread)."""
    rng = np.random.default_rng(seed)
    steps: List[LifecycleStep] = []
    remaining = {}            # live thread key -> tokens still to generate
    request_of = {}
    next_key, admitted = 0, 0
    for _ in range(n_steps):
        st = LifecycleStep()
        while admitted < n_requests and len(remaining) < max_live // 2 and rng.random() < 0.5:
            st.arrive.append((next_key, admitted, int(rng.integers(5, 90))))
            remaining[next_key] = int(rng.integers(20, 120))
            request_of[next_key] = admitted
            next_key += 1
            admitted += 1
        for key in list(remaining):
            if len(remaining) < max_live and remaining[key] > 8 and rng.random() < 0.06:
                st.fork.append((key, next_key))            # the child writes the detail paragraph
                remaining[next_key] = int(rng.integers(4, 60))
                request_of[next_key] = request_of[key]
                next_key += 1
        for key in list(remaining):
            remaining[key] -= 1
            if remaining[key] <= 0:
                st.finish.append(key)
                del remaining[key]
        steps.append(st)
    return steps, request_of


def lifecycle_longest_thread(steps) -> int:
    """Most tokens any thread of the schedule ever holds (its whole chain), for sizing block
    tables: a thread starts with its prompt or its parent's length and gains a token per step."""
    length, live, longest = {}, [], 0
    for st in steps:
        for key, _, prompt in st.arrive:
            length[key] = prompt
            live.append(key)
        for parent, child in st.fork:
            length[child] = length[parent]
            live.append(child)
        for key in live:
            length[key] += 1
            longest = max(longest, length[key])
        for key in st.finish:
            live.remove(key)
    return longest


def run_lifecycle(steps, request_of, backend, rows, early_release: bool = True, on_step=None):
    """Drive `backend` through the schedule.  `rows(n)` supplies (k, v) for n new token rows.
    With early_release a thread's cache is released the moment it finishes (Section 2.3);
    otherwise only when its whole request has finished.  on_step(step_index, live_handles) runs
    after the step's appends."""
    handle, live, finished_of_request, alive_of_request = {}, [], {}, {}
    for i, st in enumerate(steps):
        if st.arrive:
            hs = backend.new_threads(len(st.arrive))
            counts = [p for _, _, p in st.arrive]
            backend.append(hs, counts, *rows(sum(counts)))
            for (key, req, _), h in zip(st.arrive, hs):
                handle[key] = h
                live.append(key)
                alive_of_request[req] = alive_of_request.get(req, 0) + 1
        if st.fork:
            hs = backend.fork([handle[p] for p, _ in st.fork])
            for (_, child), h in zip(st.fork, hs):
                handle[child] = h
                live.append(child)
                alive_of_request[request_of[child]] += 1
        if live:
            backend.append([handle[k] for k in live], None, *rows(len(live)))
            if on_step is not None:
                on_step(i, [handle[k] for k in live])
        for key in st.finish:
            live.remove(key)
            req = request_of[key]
            alive_of_request[req] -= 1
            if early_release:
                backend.release([handle[key]])
            else:
                finished_of_request.setdefault(req, []).append(handle[key])
                if alive_of_request[req] == 0:
                    backend.release(finished_of_request.pop(req))
    leftovers = [handle[k] for k in live] + [h for hs in finished_of_request.values() for h in hs]
    if leftovers:
        backend.release(leftovers)

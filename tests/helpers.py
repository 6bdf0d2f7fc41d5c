"""Shared test plumbing: the CPU checker as a replay backend and comparison helpers."""
import numpy as np
import torch

from oracle import BlockModel, Forest, tree_decode_attention

MAX_ABS, MEAN_ABS = 2e-2, 1e-3     # bf16 in/out against the fp64 checker


class OracleBackend:
    """Logical forest plus the integer pool model, driven by the same events as the library."""

    def __init__(self, shape, num_blocks, max_threads, max_blocks_per_thread):
        self.shape = shape
        self.forest = Forest(shape.num_kv_heads, shape.head_dim)
        self.model = BlockModel(num_blocks, shape.block_size, max_threads, max_blocks_per_thread)
        self.node_of = {}          # thread id -> forest node
        self.copies = []

    def new_threads(self, n):
        tids = self.model.new_threads(n)
        for t in tids:
            self.node_of[t] = self.forest.new_thread()
        return tids

    def fork(self, parents):
        kids, copies = self.model.fork(parents)
        self.copies = copies
        for p, c in zip(parents, kids):
            self.node_of[c] = self.forest.fork(self.node_of[p])
        return kids

    def append(self, tids, counts, k_rows, v_rows):
        counts = [1] * len(tids) if counts is None else list(counts)
        self.model.append(tids, counts)
        k = k_rows.detach().cpu().to(torch.float64).numpy()
        v = v_rows.detach().cpu().to(torch.float64).numpy()
        off = 0
        for t, n in zip(tids, counts):
            if n:
                self.forest.append(self.node_of[t], k[off:off + n], v[off:off + n])
            off += n

    def release(self, tids):
        self.model.release(tids)

    def attention(self, tids, q, sm_scale):
        qq = q.detach().cpu().to(torch.float64).numpy()
        return tree_decode_attention(self.forest, [self.node_of[t] for t in tids], qq, sm_scale)


def assert_close(got_bf16: torch.Tensor, ref: np.ndarray, what=""):
    got = got_bf16.detach().cpu().to(torch.float64).numpy()
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    assert err.max() <= MAX_ABS, f"{what}: max abs err {err.max():.3e}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean abs err {err.mean():.3e}"
    return err.max(), err.mean()


def assert_same_bookkeeping(sess, model, tids):
    from paper_2401_06761_b200 import binding as B
    code = B.apar_get_stats(sess.ctx)["device_wait_timeouts"]
    assert code == 0, f"a kernel gave up a bounded wait (code {code})"
    B.apar_check_invariants(sess.ctx)
    for t in tids:
        ln, blocks = B.apar_get_thread(sess.ctx, t)
        assert ln == model.lens[t] and blocks == model.tables[t], f"thread {t}"
    assert B.apar_get_refcounts(sess.ctx, model.num_blocks) == model.refcount
    assert B.apar_get_free_list(sess.ctx, model.num_blocks) == model.free_list()

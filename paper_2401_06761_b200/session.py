"""A pool plus a library context: device memory from PyTorch, every operation through the
C-ABI binding.  Used by the tests, the benchmark and the smoke entry."""
from __future__ import annotations

import math

import torch

from . import binding as B
from .synth import ForestSpec, LayerShape


def pool_requirements(spec: ForestSpec, slack: float = 0.05):
    """(num_blocks, max_threads, max_blocks_per_thread) that hold `spec`."""
    bs = spec.shape.block_size
    blocks = sum(-(-n.n_tok // bs) + 1 for n in spec.nodes)
    longest = max(spec.attended_tokens(n) for n in spec.nodes)
    depth = max(n.depth for n in spec.nodes) + 1
    return (int(blocks * (1 + slack)) + 16, len(spec.nodes) + 8, -(-longest // bs) + depth + 1)


class PagedSession:
    def __init__(self, shape: LayerShape, num_blocks: int, max_threads: int,
                 max_blocks_per_thread: int, device="cuda", poison: bool = False,
                 num_layers: int = 1):
        if not torch.cuda.is_available():
            raise RuntimeError("the APAR library needs a CUDA device; there is no CPU path")
        self.shape, self.device = shape, torch.device(device)
        self.num_blocks = num_blocks
        self.num_layers = num_layers
        pool_shape = (num_layers * num_blocks, shape.num_kv_heads, shape.block_size,
                      shape.head_dim)
        if poison:   # NaN bit patterns everywhere: any read of an unwritten row shows up
            self.k_pool = torch.full(pool_shape, float("nan"), dtype=torch.bfloat16, device=device)
            self.v_pool = torch.full(pool_shape, float("nan"), dtype=torch.bfloat16, device=device)
        else:
            self.k_pool = torch.zeros(pool_shape, dtype=torch.bfloat16, device=device)
            self.v_pool = torch.zeros(pool_shape, dtype=torch.bfloat16, device=device)
        cfg = B.make_config(num_blocks, shape.num_q_heads, shape.num_kv_heads, max_threads,
                            max_blocks_per_thread, num_layers=num_layers)
        ws_bytes = B.apar_workspace_bytes(cfg)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
        cfg.k_pool, cfg.v_pool = self.k_pool.data_ptr(), self.v_pool.data_ptr()
        cfg.workspace, cfg.workspace_bytes = self.workspace.data_ptr(), ws_bytes
        self.cfg = cfg
        self.ctx = B.apar_create(cfg)
        self.sm_scale = 1.0 / math.sqrt(shape.head_dim)

    @classmethod
    def for_spec(cls, spec: ForestSpec, device="cuda", poison=False, extra_blocks=0):
        nb, nt, mb = pool_requirements(spec)
        return cls(spec.shape, nb + extra_blocks, nt, mb, device, poison)

    def close(self):
        if self.ctx is not None:
            torch.cuda.synchronize()
            B.apar_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _stream() -> int:
        return torch.cuda.current_stream().cuda_stream

    # the replay protocol of synth.build_forest
    def new_threads(self, n):
        return B.apar_new_threads(self.ctx, n)

    def fork(self, parents):
        return B.apar_fork(self.ctx, parents, self._stream())

    def append(self, tids, counts, k_rows: torch.Tensor, v_rows: torch.Tensor):
        assert k_rows.is_cuda and k_rows.is_contiguous() and v_rows.is_contiguous()
        assert k_rows.dtype == torch.bfloat16 and k_rows.shape == v_rows.shape
        assert k_rows.shape[0] == (sum(counts) if counts is not None else len(tids))
        B.apar_append_kv(self.ctx, tids, counts, k_rows.data_ptr(), v_rows.data_ptr(),
                         self._stream())

    def attention(self, tids, q: torch.Tensor, out: torch.Tensor = None, sm_scale=None):
        assert q.is_cuda and q.is_contiguous() and q.dtype == torch.bfloat16
        if out is None:
            out = torch.empty_like(q)
        B.apar_tree_decode_attention(self.ctx, tids, q.data_ptr(), out.data_ptr(),
                                     self.sm_scale if sm_scale is None else sm_scale,
                                     self._stream())
        return out

    def decode_step(self, tids, k_rows: torch.Tensor, v_rows: torch.Tensor, q: torch.Tensor,
                    out: torch.Tensor = None, sm_scale=None):
        assert k_rows.is_cuda and k_rows.is_contiguous() and v_rows.is_contiguous()
        assert q.is_cuda and q.is_contiguous() and q.dtype == torch.bfloat16
        if out is None:
            out = torch.empty_like(q)
        B.apar_decode_step(self.ctx, tids, k_rows.data_ptr(), v_rows.data_ptr(), q.data_ptr(),
                           out.data_ptr(), self.sm_scale if sm_scale is None else sm_scale,
                           self._stream())
        return out

    def prefix_attention(self, tids, attend_len, q: torch.Tensor, sm_scale=None):
        assert q.is_cuda and q.is_contiguous() and q.dtype == torch.bfloat16
        out = torch.empty_like(q)
        B.apar_tree_prefix_attention(self.ctx, tids, attend_len, q.data_ptr(), out.data_ptr(),
                                     self.sm_scale if sm_scale is None else sm_scale,
                                     self._stream())
        return out

    def verify_attention(self, tids, n_cand, anc_mask, q: torch.Tensor, sm_scale=None):
        assert q.is_cuda and q.is_contiguous() and q.dtype == torch.bfloat16
        out = torch.empty_like(q)
        B.apar_tree_verify_attention(self.ctx, tids, n_cand, anc_mask, q.data_ptr(),
                                     out.data_ptr(),
                                     self.sm_scale if sm_scale is None else sm_scale,
                                     self._stream())
        return out

    def accept(self, tids, n_cand, keep):
        B.apar_accept_candidates(self.ctx, tids, n_cand, keep, self._stream())

    def prefill_attention(self, tids, q_begin, q_count, q: torch.Tensor, out: torch.Tensor = None,
                          layer: int = 0, sm_scale=None):
        assert q.is_cuda and q.is_contiguous() and q.dtype == torch.bfloat16
        if out is None:
            out = torch.empty_like(q)
        B.apar_tree_prefill_attention(self.ctx, layer, tids, q_begin, q_count, q.data_ptr(),
                                      out.data_ptr(),
                                      self.sm_scale if sm_scale is None else sm_scale,
                                      self._stream())
        return out

    def append_layer(self, layer: int, k_rows: torch.Tensor, v_rows: torch.Tensor):
        assert k_rows.is_cuda and k_rows.is_contiguous() and v_rows.is_contiguous()
        B.apar_append_kv_layer(self.ctx, layer, k_rows.data_ptr(), v_rows.data_ptr(),
                               self._stream())

    def attention_layer(self, layer: int, q: torch.Tensor, out: torch.Tensor = None,
                        sm_scale=None):
        assert q.is_cuda and q.is_contiguous() and q.dtype == torch.bfloat16
        if out is None:
            out = torch.empty_like(q)
        B.apar_tree_decode_attention_layer(self.ctx, layer, q.data_ptr(), out.data_ptr(),
                                           self.sm_scale if sm_scale is None else sm_scale,
                                           self._stream())
        return out

    def release(self, tids):
        B.apar_release(self.ctx, tids)

    def stats(self):
        return B.apar_get_stats(self.ctx)

    def thread(self, tid):
        return B.apar_get_thread(self.ctx, tid)

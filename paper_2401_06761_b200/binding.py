"""ctypes binding of libapar.so: the same names and arguments as include/apar.h.

Argument marshalling only.  Device buffers are passed as integer addresses (for example
`tensor.data_ptr()`), host arrays as sequences of ints.  There is no fallback: if the
library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libapar.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2401_06761_b200.build`")
lib = C.CDLL(_LIB_PATH)

APAR_OK = 0
STATUS = {0: "OK", -1: "INVALID_ARG", -2: "BAD_THREAD", -3: "NO_BLOCKS", -4: "NO_THREADS",
          -5: "TABLE_FULL", -6: "EMPTY_CONTEXT", -7: "WORKSPACE_TOO_SMALL", -8: "CUDA",
          -9: "UNSUPPORTED"}


class AparError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        self.code = STATUS.get(status, "UNKNOWN")
        super().__init__(lib.apar_status_string(status).decode())


class apar_config(C.Structure):
    _fields_ = [("num_blocks", C.c_int32), ("block_size", C.c_int32),
                ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("max_threads", C.c_int32),
                ("max_blocks_per_thread", C.c_int32), ("num_layers", C.c_int32),
                ("k_pool", C.c_void_p), ("v_pool", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class apar_stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "live_threads", "free_blocks", "used_blocks", "forks", "cow_blocks", "cow_rows",
        "attn_threads", "attn_attended_tokens", "attn_unique_tokens", "attn_work_items",
        "attn_partials", "attn_kernels", "attn_plan_reused", "attn_vec_items",
        "attn_mma_items", "kernels_total", "peak_used_blocks", "device_wait_timeouts",
        "attn_plan_host_us", "attn_upload_bytes")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


_i32p = C.POINTER(C.c_int32)
_ctx = C.c_void_p
_cfgp = C.POINTER(apar_config)

_SIGS = {
    "apar_workspace_bytes": (C.c_size_t, [_cfgp]),
    "apar_create": (C.c_int32, [_cfgp, C.POINTER(_ctx)]),
    "apar_create_host_only": (C.c_int32, [_cfgp, C.POINTER(_ctx)]),
    "apar_destroy": (C.c_int32, [_ctx]),
    "apar_new_threads": (C.c_int32, [_ctx, C.c_int32, _i32p]),
    "apar_fork": (C.c_int32, [_ctx, C.c_int32, _i32p, _i32p, C.c_void_p]),
    "apar_append_kv": (C.c_int32, [_ctx, C.c_int32, _i32p, _i32p, C.c_void_p, C.c_void_p,
                                   C.c_void_p]),
    "apar_tree_decode_attention": (C.c_int32, [_ctx, C.c_int32, _i32p, C.c_void_p, C.c_void_p,
                                               C.c_float, C.c_void_p]),
    "apar_tree_prefix_attention": (C.c_int32, [_ctx, C.c_int32, _i32p, _i32p, C.c_void_p,
                                               C.c_void_p, C.c_float, C.c_void_p]),
    "apar_tree_verify_attention": (C.c_int32, [_ctx, C.c_int32, _i32p, _i32p,
                                               C.POINTER(C.c_uint64), C.c_void_p, C.c_void_p,
                                               C.c_float, C.c_void_p]),
    "apar_accept_candidates": (C.c_int32, [_ctx, C.c_int32, _i32p, _i32p, _i32p, _i32p,
                                           C.c_void_p]),
    "apar_tree_prefill_attention": (C.c_int32, [_ctx, C.c_int32, C.c_int32, _i32p, _i32p, _i32p,
                                                C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "apar_append_kv_layer": (C.c_int32, [_ctx, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "apar_tree_decode_attention_layer": (C.c_int32, [_ctx, C.c_int32, C.c_void_p, C.c_void_p,
                                                     C.c_float, C.c_void_p]),
    "apar_decode_step": (C.c_int32, [_ctx, C.c_int32, _i32p, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_float, C.c_void_p]),
    "apar_steps_before_new_block": (C.c_int32, [_ctx, _i32p]),
    "apar_note_step_replay": (C.c_int32, [_ctx]),
    "apar_release": (C.c_int32, [_ctx, C.c_int32, _i32p]),
    "apar_tree_decode_attention_tables": (C.c_int32, [_cfgp, C.c_int32, _i32p, _i32p,
                                                      C.c_void_p, C.c_void_p, C.c_float,
                                                      C.c_void_p]),
    "apar_tree_decode_attention_static": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                                      C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                                      C.c_int32, C.c_void_p, C.c_void_p, C.c_float,
                                                      C.c_void_p]),
    "apar_paragraph_root": (C.c_int32, [_ctx, C.c_int32]),
    "apar_restore": (C.c_int32, [_ctx, C.c_int32, _i32p, C.c_int32, _i32p]),
    "apar_get_thread": (C.c_int32, [_ctx, C.c_int32, _i32p, _i32p, _i32p, C.c_int32]),
    "apar_get_refcounts": (C.c_int32, [_ctx, _i32p]),
    "apar_get_free_list": (C.c_int32, [_ctx, _i32p, C.c_int32, _i32p]),
    "apar_get_stats": (C.c_int32, [_ctx, C.POINTER(apar_stats)]),
    "apar_check_invariants": (C.c_int32, [_ctx]),
    "apar_debug_plan": (C.c_int32, [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _i32p,
                                    _i32p, C.c_int32, C.c_int32, _i32p, C.c_int32, _i32p,
                                    C.c_int32, _i32p, C.c_int32, C.POINTER(C.c_int64)]),
    "apar_debug_plan_threads": (C.c_int32, [_ctx, C.c_int32, _i32p, C.c_int32, C.c_int32,
                                            C.c_int32, _i32p, C.c_int32, _i32p, C.c_int32, _i32p,
                                            C.c_int32, C.POINTER(C.c_int64)]),
    "apar_stream_read": (C.c_int32, [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]),
    "apar_set_timing_events": (C.c_int32, [_ctx, C.c_void_p, C.c_void_p]),
    "apar_last_cuda_error": (C.c_int32, [_ctx]),
    "apar_status_string": (C.c_char_p, [C.c_int32]),
}
for _name, (_res, _args) in _SIGS.items():
    _f = getattr(lib, _name)
    _f.restype, _f.argtypes = _res, _args

EXPORTS = tuple(_SIGS)


def _arr(xs):
    if isinstance(xs, tuple) and len(xs) == 2 and isinstance(xs[1], int):
        return xs          # already marshalled by int32_array()
    a = np.ascontiguousarray(np.fromiter(xs, dtype=np.int32) if not isinstance(xs, np.ndarray)
                             else xs.astype(np.int32, copy=False))
    buf = (C.c_int32 * max(a.size, 1)).from_buffer_copy(a.tobytes() if a.size else b"\0" * 4)
    return buf, int(a.size)


def _check(status: int):
    if status != APAR_OK:
        raise AparError(status)


def make_config(num_blocks, num_q_heads, num_kv_heads, max_threads, max_blocks_per_thread,
                k_pool=0, v_pool=0, workspace=0, workspace_bytes=0, block_size=16, head_dim=128,
                num_layers=1):
    return apar_config(num_blocks, block_size, num_q_heads, num_kv_heads, head_dim, max_threads,
                       max_blocks_per_thread, num_layers, k_pool, v_pool, workspace,
                       workspace_bytes)


def apar_workspace_bytes(cfg: apar_config) -> int:
    return lib.apar_workspace_bytes(C.byref(cfg))


def apar_create(cfg: apar_config):
    ctx = _ctx()
    _check(lib.apar_create(C.byref(cfg), C.byref(ctx)))
    return ctx


def apar_create_host_only(cfg: apar_config):
    ctx = _ctx()
    _check(lib.apar_create_host_only(C.byref(cfg), C.byref(ctx)))
    return ctx


def apar_destroy(ctx):
    _check(lib.apar_destroy(ctx))


def apar_new_threads(ctx, n: int):
    out = (C.c_int32 * max(n, 1))()
    _check(lib.apar_new_threads(ctx, n, out))
    return list(out[:n])


def apar_fork(ctx, parent_tid, stream=0):
    parents, n = _arr(parent_tid)
    out = (C.c_int32 * max(n, 1))()
    _check(lib.apar_fork(ctx, n, parents, out, stream))
    return list(out[:n])


def apar_append_kv(ctx, tid, n_tok, k_new: int, v_new: int, stream=0):
    tids, n = _arr(tid)
    counts = _arr(n_tok)[0] if n_tok is not None else None
    _check(lib.apar_append_kv(ctx, n, tids, counts, k_new, v_new, stream))


def apar_tree_decode_attention(ctx, tid, q: int, out: int, sm_scale: float, stream=0):
    tids, n = _arr(tid)
    _check(lib.apar_tree_decode_attention(ctx, n, tids, q, out, sm_scale, stream))


def apar_tree_prefix_attention(ctx, tid, attend_len, q: int, out: int, sm_scale: float, stream=0):
    tids, n = _arr(tid)
    lens, _ = _arr(attend_len)
    _check(lib.apar_tree_prefix_attention(ctx, n, tids, lens, q, out, sm_scale, stream))


def apar_tree_verify_attention(ctx, tid, n_cand, anc_mask, q: int, out: int, sm_scale: float,
                               stream=0):
    """anc_mask: one Python int (uint64 bit mask) per candidate, all threads' candidates in order."""
    tids, n = _arr(tid)
    cands, _ = _arr(n_cand)
    masks = (C.c_uint64 * max(len(anc_mask), 1))(*anc_mask)
    _check(lib.apar_tree_verify_attention(ctx, n, tids, cands, masks, q, out, sm_scale, stream))


def apar_accept_candidates(ctx, tid, n_cand, keep, stream=0):
    """keep: per thread, the list of candidate indices that stay (increasing)."""
    tids, n = _arr(tid)
    cands, _ = _arr(n_cand)
    counts, _ = _arr([len(k) for k in keep])
    flat, _ = _arr([x for k in keep for x in k])
    _check(lib.apar_accept_candidates(ctx, n, tids, cands, counts, flat, stream))


def apar_tree_prefill_attention(ctx, layer: int, tid, q_begin, q_count, q: int, out: int,
                                sm_scale: float, stream=0):
    tids, n = _arr(tid)
    begins, _ = _arr(q_begin)
    counts, _ = _arr(q_count)
    _check(lib.apar_tree_prefill_attention(ctx, layer, n, tids, begins, counts, q, out, sm_scale,
                                           stream))


def apar_append_kv_layer(ctx, layer: int, k_new: int, v_new: int, stream=0):
    _check(lib.apar_append_kv_layer(ctx, layer, k_new, v_new, stream))


def apar_tree_decode_attention_layer(ctx, layer: int, q: int, out: int, sm_scale: float, stream=0):
    _check(lib.apar_tree_decode_attention_layer(ctx, layer, q, out, sm_scale, stream))


def apar_decode_step(ctx, tid, k_new: int, v_new: int, q: int, out: int, sm_scale: float,
                     stream=0):
    tids, n = _arr(tid)
    _check(lib.apar_decode_step(ctx, n, tids, k_new, v_new, q, out, sm_scale, stream))


def apar_steps_before_new_block(ctx) -> int:
    steps = C.c_int32()
    _check(lib.apar_steps_before_new_block(ctx, C.byref(steps)))
    return steps.value


def apar_note_step_replay(ctx):
    _check(lib.apar_note_step_replay(ctx))


def apar_release(ctx, tid):
    tids, n = _arr(tid)
    _check(lib.apar_release(ctx, n, tids))


def apar_tree_decode_attention_tables(cfg, block_tables, ctx_lens, q: int, out: int,
                                      sm_scale: float, stream=0):
    """block_tables: n rows, each padded by the caller to cfg.max_blocks_per_thread ints."""
    lens, n = _arr(ctx_lens)
    flat, _ = _arr(x for row in block_tables for x in row)
    _check(lib.apar_tree_decode_attention_tables(C.byref(cfg), n, flat, lens, q, out,
                                                 sm_scale, stream))


def apar_tree_decode_attention_static(k_pool: int, v_pool: int, num_q_heads: int,
                                      num_kv_heads: int, n_threads: int,
                                      max_blocks_per_thread: int, block_tables: int,
                                      ctx_lens: int, max_ctx_len: int, q: int, out: int,
                                      sm_scale: float, stream=0):
    """Allocation-free variant: block_tables and ctx_lens are DEVICE addresses here."""
    _check(lib.apar_tree_decode_attention_static(k_pool, v_pool, num_q_heads, num_kv_heads,
                                                 n_threads, max_blocks_per_thread, block_tables,
                                                 ctx_lens, max_ctx_len, q, out, sm_scale, stream))


def apar_paragraph_root(ctx, tid: int):
    _check(lib.apar_paragraph_root(ctx, tid))


def apar_restore(ctx, root_tid: int):
    """Slices (tid, start, end) of the response in reading order."""
    n = C.c_int32()
    _check(lib.apar_restore(ctx, root_tid, None, 0, C.byref(n)))
    buf = (C.c_int32 * max(3 * n.value, 1))()
    _check(lib.apar_restore(ctx, root_tid, buf, n.value, C.byref(n)))
    return [tuple(buf[3 * i:3 * i + 3]) for i in range(n.value)]


def apar_get_thread(ctx, tid: int, cap: int = 0):
    """Returns (len, blocks)."""
    ln, nb = C.c_int32(), C.c_int32()
    _check(lib.apar_get_thread(ctx, tid, C.byref(ln), C.byref(nb), None, 0))
    blocks = (C.c_int32 * max(nb.value, 1))()
    _check(lib.apar_get_thread(ctx, tid, None, None, blocks, nb.value))
    return ln.value, list(blocks[:nb.value])


def apar_get_refcounts(ctx, num_blocks: int):
    out = (C.c_int32 * num_blocks)()
    _check(lib.apar_get_refcounts(ctx, out))
    return list(out)


def apar_get_free_list(ctx, num_blocks: int):
    out = (C.c_int32 * max(num_blocks, 1))()
    n = C.c_int32()
    _check(lib.apar_get_free_list(ctx, out, num_blocks, C.byref(n)))
    return list(out[:min(n.value, num_blocks)])


def apar_get_stats(ctx) -> dict:
    s = apar_stats()
    _check(lib.apar_get_stats(ctx, C.byref(s)))
    return s.as_dict()


def apar_check_invariants(ctx):
    _check(lib.apar_check_invariants(ctx))


def apar_debug_plan(num_blocks, num_q_heads, num_kv_heads, tables, lens, mma_min_rows=2,
                    fuse_final=True):
    """Host-only planning of one attention call; `tables` is an [n][max_blocks] int32 array.
    Returns (items [k][8], users [m][2], merges [j][3], counts dict) as numpy arrays."""
    tables = np.ascontiguousarray(tables, dtype=np.int32)
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    n, mb = tables.shape
    cap_users = int(sum((int(l) + 15) // 16 for l in lens)) + 1
    cap_items = 4 * cap_users + 16
    items = np.zeros((cap_items, 8), dtype=np.int32)
    users = np.zeros((cap_users, 2), dtype=np.int32)
    merges = np.zeros((n + 1, 3), dtype=np.int32)
    counts = (C.c_int64 * 6)()
    p = lambda a: a.ctypes.data_as(_i32p)
    _check(lib.apar_debug_plan(num_blocks, num_q_heads, num_kv_heads, n, mb, p(tables), p(lens),
                               mma_min_rows, int(bool(fuse_final)), p(items), cap_items,
                               p(users), cap_users, p(merges), n + 1, counts))
    names = ("items", "users", "merges", "partial_slots", "unique_tokens", "attended_tokens")
    c = dict(zip(names, (int(x) for x in counts)))
    return items[:c["items"]], users[:c["users"]], merges[:c["merges"]], c


def apar_debug_plan_threads(ctx, tid, by_groups: bool, mma_min_rows=2, fuse_final=True):
    """Host-only planning for threads of a context; same return value as apar_debug_plan."""
    tids, n = _arr(tid)
    lens = [apar_get_thread(ctx, t)[0] for t in tid]
    cap_users = int(sum((int(l) + 15) // 16 for l in lens)) + 1
    cap_items = 4 * cap_users + 16
    items = np.zeros((cap_items, 8), dtype=np.int32)
    users = np.zeros((cap_users, 2), dtype=np.int32)
    merges = np.zeros((n + 1, 3), dtype=np.int32)
    counts = (C.c_int64 * 6)()
    p = lambda a: a.ctypes.data_as(_i32p)
    _check(lib.apar_debug_plan_threads(ctx, n, tids, int(bool(by_groups)), mma_min_rows,
                                       int(bool(fuse_final)), p(items), cap_items, p(users),
                                       cap_users, p(merges), n + 1, counts))
    names = ("items", "users", "merges", "partial_slots", "unique_tokens", "attended_tokens")
    c = dict(zip(names, (int(x) for x in counts)))
    return items[:c["items"]], users[:c["users"]], merges[:c["merges"]], c


def apar_stream_read(src: int, nbytes: int, sink: int, stream=0):
    _check(lib.apar_stream_read(src, nbytes, sink, stream))


def apar_set_timing_events(ctx, start: int, stop: int):
    """cudaEvent_t handles (integers), or 0, 0 to turn the recording off."""
    _check(lib.apar_set_timing_events(ctx, start or None, stop or None))


def apar_last_cuda_error(ctx) -> int:
    return lib.apar_last_cuda_error(ctx)


def int32_array(xs):
    """Pre-marshalled id list for repeated calls of apar_tree_decode_attention."""
    return _arr(xs)

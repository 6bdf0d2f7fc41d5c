"""The allocation-free attention entry point against the CPU checker.

apar_tree_decode_attention_static exists for callers that may not allocate GPU or pinned
memory from inside a library call (pre-carved serving processes, plugins without access to
the host's CUDA allocator, threads that must not trigger allocator-induced device syncs).
It keeps its scratch in an array inside the library image, shared by all calls, so every test
calls it twice in a row with different inputs: the second result must not be polluted by
what the first call left behind.  The expected values come from the fp64 checker over rows
gathered from the pools through the test's own tables; the regular table-driven entry point
is compared as well.  This file sorts last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import dense_attention

pytestmark = pytest.mark.gpu

SCALE = 0.088


def _problem(seed, lens, hq, hkv, num_blocks, max_blocks):
    """Random pools and queries; private rows whose blocks are scattered over the pool."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    k = torch.randn((num_blocks, hkv, 16, 128), generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn((num_blocks, hkv, 16, 128), generator=g, device="cuda").to(torch.bfloat16)
    q = torch.randn((len(lens), hq, 128), generator=g, device="cuda").to(torch.bfloat16)
    perm = torch.randperm(num_blocks, generator=torch.Generator().manual_seed(seed)).tolist()
    tables, used = [], 0
    for ln in lens:
        nb = min(max_blocks, -(-max(ln, 0) // 16))
        tables.append(perm[used:used + nb] + [0] * (max_blocks - nb))
        used += nb
    assert used <= num_blocks
    return k, v, q, tables


def _expected(k, v, q, tables, lens):
    """The checker's answer, row by row; a row without tokens is defined as zeros."""
    kc, vc = k.cpu().to(torch.float64).numpy(), v.cpu().to(torch.float64).numpy()
    qc = q.cpu().to(torch.float64).numpy()
    ref = np.zeros(qc.shape)
    for i, ln in enumerate(lens):
        if ln <= 0:
            continue
        ids = tables[i][:-(-ln // 16)]
        K = kc[ids].transpose(0, 2, 1, 3).reshape(-1, kc.shape[1], 128)[:ln]
        V = vc[ids].transpose(0, 2, 1, 3).reshape(-1, vc.shape[1], 128)[:ln]
        ref[i] = dense_attention(qc[i], K, V, SCALE)
    return ref


def _run_static(k, v, q, tables, lens, hq, hkv, max_blocks, max_ctx_len):
    from paper_2401_06761_b200 import binding as B
    d_tables = torch.tensor(tables, dtype=torch.int32, device="cuda")
    d_lens = torch.tensor(lens, dtype=torch.int32, device="cuda")
    got = torch.full_like(q, float("nan"))
    B.apar_tree_decode_attention_static(k.data_ptr(), v.data_ptr(), hq, hkv, len(lens), max_blocks,
                                        d_tables.data_ptr(), d_lens.data_ptr(), max_ctx_len,
                                        q.data_ptr(), got.data_ptr(), SCALE,
                                        torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return got


def _check(got, ref, what):
    g = got.cpu().to(torch.float64).numpy()
    assert np.isfinite(g).all(), what
    err = np.abs(g - ref)
    assert err.max() <= 2e-2 and err.mean() <= 1e-3, (what, err.max(), err.mean())


def _random_lens(seed, n, max_len):
    cpu = torch.Generator().manual_seed(seed)
    lens = torch.randint(1, max_len + 1, (n,), generator=cpu).tolist()
    lens[0], lens[-1] = max_len, 1
    return lens


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4)])
def test_static_entry_point_matches_the_checker_twice(hq, hkv):
    from paper_2401_06761_b200 import binding as B
    n, max_len, max_blocks, num_blocks = 12, 3000, 192, 2400
    cfg = B.make_config(num_blocks, hq, hkv, n, max_blocks)
    ws = torch.empty(B.apar_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for call, seed in enumerate((11, 12)):       # two calls in a row, different data and lengths
        lens = _random_lens(seed, n, max_len - 700 * call)
        k, v, q, tables = _problem(seed, lens, hq, hkv, num_blocks, max_blocks)
        ref = _expected(k, v, q, tables, lens)
        got = _run_static(k, v, q, tables, lens, hq, hkv, max_blocks, max(lens))
        _check(got, ref, f"static call {call}")
        cfg.k_pool, cfg.v_pool = k.data_ptr(), v.data_ptr()
        cfg.workspace, cfg.workspace_bytes = ws.data_ptr(), ws.numel()
        other = torch.empty_like(q)
        B.apar_tree_decode_attention_tables(cfg, tables, lens, q.data_ptr(), other.data_ptr(),
                                            SCALE, stream)
        torch.cuda.synchronize()
        _check(other, ref, f"table-driven call {call}")


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4)])
def test_static_entry_point_with_an_upper_bound_below_the_longest_row(hq, hkv):
    """max_ctx_len is only a hint for how to cut the rows: rows longer than it must still be
    read to their end (the last range takes the excess), here with 2 and with 1 range."""
    n, max_blocks, num_blocks = 10, 192, 1600
    for call, (seed, hint) in enumerate(((21, 1500), (22, 700))):
        lens = _random_lens(seed, n, 2500)
        k, v, q, tables = _problem(seed, lens, hq, hkv, num_blocks, max_blocks)
        got = _run_static(k, v, q, tables, lens, hq, hkv, max_blocks, hint)
        _check(got, _expected(k, v, q, tables, lens), f"hint {hint}, call {call}")


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4)])
def test_static_entry_point_with_eight_ranges_and_short_rows(hq, hkv):
    """Eight ranges of 1024 tokens: rows shorter than one range leave the later ranges empty,
    a row of length 0 receives zeros, and a length beyond what a table row can hold is read as
    the row's capacity (the lengths live on the device, so the host cannot refuse them)."""
    n, max_blocks, num_blocks = 9, 512, 2300
    for call, seed in enumerate((31, 32)):
        lens = [8192, 5, 1023, 1024, 1025, 0, 3000 + 17 * call, 16, 8192 + 400]
        k, v, q, tables = _problem(seed, lens, hq, hkv, num_blocks, max_blocks)
        seen = [min(ln, 16 * max_blocks) for ln in lens]          # what the call must compute
        got = _run_static(k, v, q, tables, lens, hq, hkv, max_blocks, 8192)
        _check(got, _expected(k, v, q, tables, seen), f"eight ranges, call {call}")
        assert not got[5].float().abs().max().item()                # the empty row: exact zeros


def test_static_entry_point_refuses_oversized_requests():
    from paper_2401_06761_b200 import binding as B
    z = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.AparError) as e:        # 512 rows x 64 heads x 8 splits: beyond 16 MiB
        B.apar_tree_decode_attention_static(z.data_ptr(), z.data_ptr(), 64, 8, 512, 512,
                                            z.data_ptr(), z.data_ptr(), 8192, z.data_ptr(),
                                            z.data_ptr(), 0.1, 0)
    assert e.value.code == "WORKSPACE_TOO_SMALL"
    with pytest.raises(B.AparError) as e:
        B.apar_tree_decode_attention_static(z.data_ptr(), z.data_ptr(), 8, 3, 1, 4, z.data_ptr(),
                                            z.data_ptr(), 16, z.data_ptr(), z.data_ptr(), 0.1, 0)
    assert e.value.code == "UNSUPPORTED"

"""The allocation-free attention entry point against the regular table-driven one.

apar_tree_decode_attention_static exists for callers that may not allocate GPU or pinned
memory from inside a library call (pre-carved serving processes, plugins without access to
the host's CUDA allocator, threads that must not trigger allocator-induced device syncs).
It keeps its scratch in an array inside the library image, shared by all calls, so the test
calls it twice in a row with different inputs: the second result must not be polluted by
what the first call left behind.  This file sorts last on purpose.
"""
import pytest
import torch

from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


def _problem(seed, n, hq, hkv, max_len, num_blocks, max_blocks):
    g = torch.Generator(device="cuda").manual_seed(seed)
    k = torch.randn((num_blocks, hkv, 16, 128), generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn((num_blocks, hkv, 16, 128), generator=g, device="cuda").to(torch.bfloat16)
    q = torch.randn((n, hq, 128), generator=g, device="cuda").to(torch.bfloat16)
    cpu = torch.Generator().manual_seed(seed)
    lens = torch.randint(1, max_len + 1, (n,), generator=cpu).tolist()
    lens[0], lens[-1] = max_len, 1
    perm = torch.randperm(num_blocks, generator=cpu).tolist()
    tables, used = [], 0
    for ln in lens:                      # private rows, blocks scattered over the pool
        nb = -(-ln // 16)
        tables.append(perm[used:used + nb] + [0] * (max_blocks - nb))
        used += nb
    assert used <= num_blocks
    return k, v, q, lens, tables


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4)])
def test_static_entry_point_matches_table_entry_point_twice(hq, hkv):
    from paper_2401_06761_b200 import binding as B
    n, max_len, max_blocks, num_blocks = 12, 3000, 192, 2400
    cfg = B.make_config(num_blocks, hq, hkv, n, max_blocks)
    ws = torch.empty(B.apar_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for call, seed in enumerate((11, 12)):       # two calls in a row, different data and lengths
        k, v, q, lens, tables = _problem(seed, n, hq, hkv, max_len - 700 * call, num_blocks,
                                         max_blocks)
        cfg.k_pool, cfg.v_pool = k.data_ptr(), v.data_ptr()
        cfg.workspace, cfg.workspace_bytes = ws.data_ptr(), ws.numel()
        want = torch.empty_like(q)
        B.apar_tree_decode_attention_tables(cfg, tables, lens, q.data_ptr(), want.data_ptr(),
                                            0.088, stream)
        d_tables = torch.tensor(tables, dtype=torch.int32, device="cuda")
        d_lens = torch.tensor(lens, dtype=torch.int32, device="cuda")
        got = torch.full_like(q, float("nan"))
        B.apar_tree_decode_attention_static(k.data_ptr(), v.data_ptr(), hq, hkv, n, max_blocks,
                                            d_tables.data_ptr(), d_lens.data_ptr(), max(lens),
                                            q.data_ptr(), got.data_ptr(), 0.088, stream)
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all()
        err = (got.double() - want.double()).abs()
        assert err.max() <= 2e-2 and err.mean() <= 1e-3, (call, err.max(), err.mean())


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

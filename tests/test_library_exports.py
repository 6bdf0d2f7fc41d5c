"""The C-ABI library loads without a GPU and exports every function the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "apar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(apar_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    from paper_2401_06761_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert "apar_fork" in names and "apar_append_kv" in names
    assert "apar_tree_decode_attention" in names
    for n in names:
        assert hasattr(lib, n), n
    from paper_2401_06761_b200 import binding
    assert sorted(binding.EXPORTS) == names
    for n in names:
        if n not in ("apar_status_string",):
            assert callable(getattr(binding, n)), n


def test_host_only_calls_work_without_a_device():
    from paper_2401_06761_b200 import binding as B
    cfg = B.make_config(1000, 32, 8, 64, 40)
    assert B.apar_workspace_bytes(cfg) > 0
    assert B.apar_workspace_bytes(B.make_config(1000, 32, 8, 64, 40, block_size=32)) == 0
    assert B.apar_workspace_bytes(B.make_config(1000, 32, 8, 64, 40, head_dim=64)) == 0
    assert B.lib.apar_status_string(-3) == b"APAR_ERR_NO_BLOCKS"

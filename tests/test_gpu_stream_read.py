"""The read-only streaming probe must really read every 16-byte unit exactly once: its xor
word is compared with the same fold done by numpy on the host."""
import numpy as np
import pytest
import torch

from paper_2401_06761_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_bytes", [16, 4096 + 32, 148 * 8 * 256 * 16 * 8 + 48, 100_000_007])
def test_xor_of_everything_read_once(n_bytes):
    rng = np.random.default_rng(n_bytes)
    host = rng.integers(0, 2 ** 32, size=(n_bytes + 3) // 4, dtype=np.uint32)
    dev = torch.from_numpy(host.view(np.int32)).cuda()
    start = 0x1234_5678_9ABC_DEF0
    sink = torch.tensor([start], dtype=torch.int64, device="cuda")
    B.apar_stream_read(dev.data_ptr(), n_bytes, sink.data_ptr())
    B.apar_stream_read(dev.data_ptr(), n_bytes, sink.data_ptr())      # xor twice: back to start
    assert int(sink.item()) == start
    B.apar_stream_read(dev.data_ptr(), n_bytes, sink.data_ptr())
    words = host[: (n_bytes // 16) * 4]
    expect = start ^ int(np.bitwise_xor.reduce(words))
    assert int(sink.item()) == expect


def test_rejects_bad_pointers():
    buf = torch.zeros(64, dtype=torch.int32, device="cuda")
    sink = torch.zeros(1, dtype=torch.int64, device="cuda")
    with pytest.raises(B.AparError):
        B.apar_stream_read(0, 64, sink.data_ptr())
    with pytest.raises(B.AparError):
        B.apar_stream_read(buf.data_ptr() + 4, 64, sink.data_ptr())
    with pytest.raises(B.AparError):
        B.apar_stream_read(buf.data_ptr(), 64, 0)

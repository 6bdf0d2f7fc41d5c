"""Early release and block recycling over a stream of requests (Section 2.3 and feature 2 of
Section 2.4: a finished thread gives its own cache back at once, which lowers the peak)."""
import numpy as np
import pytest
import torch

from helpers import OracleBackend, assert_close, assert_same_bookkeeping
from paper_2401_06761_b200 import synth

SHAPE = synth.LayerShape(8, 2)


def _rows_factory(device, seed):
    g = torch.Generator(device=device).manual_seed(seed)

    def rows(n):
        kv = torch.randn((2, n, 2, 128), generator=g, device=device).to(torch.bfloat16)
        return kv[0].contiguous(), kv[1].contiguous()
    return rows


def test_early_release_lowers_the_peak_in_the_pool_model():
    steps, req = synth.lifecycle_schedule(seed=3, n_requests=30, n_steps=400)
    peaks = {}
    for early in (True, False):
        orc = OracleBackend(SHAPE, 4000, 600, 40)
        synth.run_lifecycle(steps, req, orc, _rows_factory("cpu", 1), early_release=early)
        assert len(orc.model.free) == 4000 and not any(orc.model.refcount)
        peaks[early] = orc.model.peak_used
    assert peaks[True] < peaks[False]          # same work, less cache held at the worst moment
    assert sum(len(s.fork) for s in steps) > 20 and sum(len(s.finish) for s in steps) > 30


@pytest.mark.gpu
def test_library_peak_counter_against_the_hand_worked_events():
    """The library's max-cached counter against the values worked out by hand in
    tests/golden/release_refork_peak.txt (not against the pool model)."""
    from test_oracle_bookkeeping import load_golden, release_refork_events
    from paper_2401_06761_b200.session import PagedSession
    g = load_golden("release_refork_peak.txt")
    sess = PagedSession(SHAPE, g["num_blocks"], 8, 16)
    z = torch.zeros((64, 2, 128), dtype=torch.bfloat16, device="cuda")
    in_use, peak = [], []
    for ev in release_refork_events():
        if ev[0] == "new+append":
            (t,) = sess.new_threads(1)
            sess.append([t], [ev[1]], z[:ev[1]], z[:ev[1]])
        elif ev[0] == "fork":
            sess.fork([ev[1]])
        elif ev[0] == "append":
            sess.append([ev[1]], [ev[2]], z[:ev[2]], z[:ev[2]])
        else:
            sess.release([ev[1]])
        st = sess.stats()
        in_use.append(st["used_blocks"])
        peak.append(st["peak_used_blocks"])
    assert in_use == g["in_use_after_event"] and peak == g["peak_after_event"]
    for t, table in g["table"].items():
        assert sess.thread(t) == (g["len"][t], table)
    sess.close()


@pytest.mark.gpu
def test_lifecycle_replay_on_the_library_matches_the_model():
    from paper_2401_06761_b200.session import PagedSession
    steps, req = synth.lifecycle_schedule(seed=5, n_requests=24, n_steps=300)
    sess = PagedSession(SHAPE, 1500, 64, 40, poison=True)
    orc = OracleBackend(SHAPE, 1500, 64, 40)

    class Both:
        def new_threads(self, n):
            a, b = sess.new_threads(n), orc.new_threads(n)
            assert a == b
            return a

        def fork(self, parents):
            a, b = sess.fork(parents), orc.fork(parents)
            assert a == b
            return a

        def append(self, tids, counts, k, v):
            sess.append(tids, counts, k, v)
            orc.append(tids, counts, k, v)

        def release(self, tids):
            sess.release(tids)
            orc.release(tids)

    g = torch.Generator(device="cuda").manual_seed(9)
    checked = []

    def on_step(i, live):
        assert_same_bookkeeping(sess, orc.model, live)
        if i % 6 == 0:
            q = torch.randn((len(live), 8, 128), generator=g, device="cuda").to(torch.bfloat16)
            assert_close(sess.attention(live, q), orc.attention(live, q, sess.sm_scale), f"step {i}")
            checked.append(i)

    synth.run_lifecycle(steps, req, Both(), _rows_factory("cuda", 2), early_release=True,
                        on_step=on_step)
    st = sess.stats()
    assert st["free_blocks"] == 1500 and st["live_threads"] == 0
    assert st["peak_used_blocks"] == orc.model.peak_used < 1500
    assert len(checked) > 30 and st["device_wait_timeouts"] == 0
    sess.close()

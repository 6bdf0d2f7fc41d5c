"""Seeded random forests over many head shapes, every kernel family and every launch switch,
checked against the CPU checker after each round of forks, appends and releases."""
import random

import numpy as np
import pytest
import torch

from helpers import MAX_ABS, MEAN_ABS, OracleBackend
from paper_2401_06761_b200 import synth
from test_gpu_parity import Both, _session

pytestmark = pytest.mark.gpu

SHAPES = [(4, 4), (8, 2), (8, 8), (16, 2), (16, 8), (32, 8), (64, 8), (40, 40), (12, 4), (6, 1)]


@pytest.mark.parametrize("seed", range(6))
def test_random_forest_random_shape(seed, monkeypatch):
    rnd = random.Random(1000 + seed)
    for case in range(5):
        hq, hkv = rnd.choice(SHAPES)
        monkeypatch.setenv("APAR_ATTN_PATH", rnd.choice(["auto", "auto", "umma", "ws", "vec"]))
        monkeypatch.setenv("APAR_PLANNER", rnd.choice(["groups", "groups", "tables"]))
        monkeypatch.setenv("APAR_UMMA_MODE", rnd.choice(["persist", "grid"]))
        monkeypatch.setenv("APAR_WS_MODE", rnd.choice(["persist", "grid"]))
        monkeypatch.setenv("APAR_UMMA_HEADS", rnd.choice(["1", "2", "4", "8"]))
        monkeypatch.setenv("APAR_PDL", rnd.choice(["0", "1"]))
        shape = synth.LayerShape(hq, hkv)
        nb, nt, mb = 6000, 300, 140
        sess = _session(shape, nb, nt, mb, poison=True)
        orc = OracleBackend(shape, nb, nt, mb)
        both = Both(sess, orc)
        g = torch.Generator(device="cuda").manual_seed(seed * 100 + case)

        def rows(n):
            return (torch.randn((n, hkv, 128), generator=g, device="cuda").to(torch.bfloat16),
                    torch.randn((n, hkv, 128), generator=g, device="cuda").to(torch.bfloat16))

        live = both.new_threads(rnd.randrange(1, 4))
        for t in live:
            n = rnd.choice([1, 15, 16, 17, 63, 64, 65, 200, 500, 1100])
            both.append([t], [n], *rows(n))
        for _ in range(rnd.randrange(1, 5)):
            if len(live) < 150:
                parents = [rnd.choice(live) for _ in range(rnd.choice([1, 2, 5, 9, 20, 70]))]
                live += both.fork(parents[:max(1, 200 - len(live))])
            sub = rnd.sample(live, rnd.randrange(1, len(live) + 1))
            cnt = [rnd.choice([0, 1, 1, 3, 16, 40, 130]) for _ in sub]
            if sum(cnt):
                both.append(sub, cnt, *rows(sum(cnt)))
            if rnd.random() < 0.3 and len(live) > 3:
                t = rnd.choice(live)
                both.release([t])
                live.remove(t)
            qs = [t for t in live if sess.thread(t)[0] > 0]
            if not qs:
                continue
            qs = rnd.sample(qs, rnd.randrange(1, len(qs) + 1))
            q = torch.randn((len(qs), hq, 128), generator=g, device="cuda").to(torch.bfloat16)
            out = sess.attention(qs, q)
            ref = orc.attention(qs, q, sess.sm_scale)
            err = np.abs(out.cpu().to(torch.float64).numpy() - ref)
            assert np.isfinite(err).all(), (seed, case, hq, hkv)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (seed, case, hq, hkv, err.max())
        assert sess.stats()["device_wait_timeouts"] == 0
        sess.close()

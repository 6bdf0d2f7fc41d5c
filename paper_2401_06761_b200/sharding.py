"""Multi-GPU sharding of the decode hot path: requests are independent, so every rank owns its
own requests and pool and nothing is exchanged on the data path.  The only cross-rank traffic is
the benchmark's timing reduction (max of the per-rank times, sum of the units processed)."""
from __future__ import annotations

import torch

from . import synth


def shard_spec(config: int, rank: int, n_requests=None) -> synth.ForestSpec:
    """The shard of `config` that `rank` owns: the same workload shape drawn with a
    rank-specific seed (weak scaling: per-GPU work is fixed as ranks are added)."""
    return synth.forest_spec(config, seed=synth.default_seed(config, rank), n_requests=n_requests)


def reduce_timing(local_ms: float, local_units: float, dist=None, device="cpu"):
    """(max over ranks of the elapsed milliseconds, sum over ranks of the units processed)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms), float(local_units)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def whole_job_rate(local_ms: float, local_units_per_step: float, steps: int, dist=None,
                   device="cpu") -> float:
    """Units per second of the whole job: all ranks' units over the slowest rank's time."""
    ms, units = reduce_timing(local_ms, local_units_per_step, dist, device)
    return units * steps / (ms * 1e-3)

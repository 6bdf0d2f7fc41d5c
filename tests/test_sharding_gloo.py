"""The N > 1 path of the benchmark on CPU: two gloo ranks own different shards and reduce
their timings the way bench.py does (max time, summed units).  No data-path collective exists."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2401_06761_b200 import sharding, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = sharding.shard_spec(5, rank, n_requests=40)
    units = len(spec.live_nodes())
    local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    ms, total = sharding.reduce_timing(local_ms, units, dist)
    rate = sharding.whole_job_rate(local_ms, units, 7, dist)
    gathered = [None] * world
    dist.all_gather_object(gathered, (units, spec.seed, spec.unique_tokens()))
    if rank == 0:
        out.put((ms, total, rate, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_without_exchange_and_reduce_timing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, total, rate, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (u0, s0, q0), (u1, s1, q1) = gathered
    assert s0 != s1 and (u0, q0) != (u1, q1)          # different requests on each rank
    assert ms == 15.0 and total == u0 + u1            # slowest rank's time, everybody's units
    assert abs(rate - (u0 + u1) * 7 / 15e-3) < 1e-6
    # shards are reproducible and rank 0's shard is the single-GPU workload
    again = sharding.shard_spec(5, 1, n_requests=40)
    assert len(again.live_nodes()) == u1 and again.unique_tokens() == q1
    assert sharding.shard_spec(5, 0, n_requests=40).seed == synth.default_seed(5)


def test_single_process_reduction_is_identity():
    assert sharding.reduce_timing(3.5, 10) == (3.5, 10.0)
    assert sharding.whole_job_rate(2.0, 100, 4) == 100 * 4 / 2e-3

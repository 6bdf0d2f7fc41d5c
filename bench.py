#!/usr/bin/env python
"""Benchmark of the APAR decode hot path on B200: one step = (the step's fork, if the workload
has one) + KV append of one token per live thread + tree decode attention over all live
threads, for one attention layer.  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

The headline numbers (`value`, `roofline`, `e2e`) belong to `--workload` (default cfg4, the
largest configuration by bytes).  With the default workload on one GPU the same line also
carries, under `sweep`, the device-arm numbers of the other configurations (cfg1, cfg2, cfg3,
cfg5 and cfg5 with every prefix copied instead of shared), the headline workload once more
over a longer run (`sustained`: hundreds of steps, where the power cap sets the clock), and
the early-release replay (`lifecycle`: most cached tokens at once when a finished thread
gives its cache back at once, against at the end of its request).

With N > 1 (under torchrun) every rank runs its own shard of requests (a different seed of the
same workload) on its own GPU; there is no exchange between shards.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2401_06761_b200 import sharding, synth  # noqa: E402

METRIC = "tree decode-attention thread-tokens/s"
UNIT = "thread-tokens/s"
SWEEP = (("cfg1", False), ("cfg2", False), ("cfg3", False), ("cfg5", False), ("cfg5", True))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def read_only_rate(dev, n_bytes=4 << 30, reps=10):
    """GB/s of the library's read-only streaming probe over a buffer far larger than L2."""
    from paper_2401_06761_b200 import binding as B
    buf = torch.empty(n_bytes, dtype=torch.uint8, device=dev)
    sink = torch.zeros(1, dtype=torch.int64, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(3):
        B.apar_stream_read(buf.data_ptr(), n_bytes, sink.data_ptr(), stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        B.apar_stream_read(buf.data_ptr(), n_bytes, sink.data_ptr(), stream)
    e1.record()
    torch.cuda.synchronize()
    del buf
    return n_bytes * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc, self.lines, self.index = None, [], index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
            t0 = time.time()         # the first sample has arrived before the timed region starts
            while not self.lines and time.time() - t0 < 3.0:
                time.sleep(0.01)
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.1)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_mhz_min": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def parse_workload(name: str) -> int:
    if not (name.startswith("cfg") and name[3:].isdigit() and int(name[3:]) in synth.LAYER_SHAPES):
        raise SystemExit(f"unknown workload {name}; use cfg1..cfg5, lifecycle or prefill")
    return int(name[3:])


def workload_config(name, spec, unshared, layers=1, graph=False, world=1):
    """The `config` object of the JSON line; both arms print the same one."""
    shape = spec.shape
    small = spec.unique_tokens() * shape.bytes_per_token < 4 * 126e6
    has_fork = any(n.step_fork for n in spec.nodes)
    return {
        "workload": name + ("-unshared" if unshared else ""),
        "threads_per_gpu": len(spec.live_nodes()),
        "requests": len({n.request for n in spec.nodes}),
        "num_q_heads": shape.num_q_heads, "num_kv_heads": shape.num_kv_heads,
        "head_dim": shape.head_dim, "block_size": shape.block_size,
        "step": ("fork+" if has_fork else "") + "append+attention, " +
                ("one layer" if layers == 1 else f"{layers} layers (value counts thread-tokens "
                                                 f"per layer)") +
                (", layers 1.. replayed from a CUDA graph" if graph else ""),
        "l2": "inputs larger than L2 (unique KV bytes per step >> 126 MB)" if not small else
              "KV fits in L2: 256 MB written between steps, each step timed on its own "
              "(device arm)",
        "parallelism": f"{world} independent shard(s), no collective",
    }


# ------------------------------------------------------------------------------ CPU baseline
def _oracle_worker(job):
    """One host core: times the fp64 checker, as it stands, on live threads of the workload
    until the budget is used.  Runs in a process of its own; one BLAS thread."""
    cfg_id, seed, n_requests, unshared, offset, stride, budget_s = job
    import numpy as np
    try:
        from threadpoolctl import threadpool_limits
        threadpool_limits(1)
    except Exception:
        pass
    torch.set_num_threads(1)
    from oracle import Forest, tree_decode_attention
    spec = synth.forest_spec(cfg_id, seed=seed, n_requests=n_requests)
    if unshared:
        spec = synth.unshared_spec(spec)
    live = spec.live_nodes()
    scale = spec.shape.head_dim ** -0.5
    q_all = synth.queries(spec, len(live), "cpu").to(torch.float64).numpy()
    done, spent = 0, 0.0
    # this worker's share: threads offset, offset + stride, ... of a walk that visits every
    # region of the request range first
    coarse = list(range(0, len(live), max(1, len(live) // 64)))
    first = set(coarse)
    order = coarse + [i for i in range(len(live)) if i not in first]
    for i in order[offset::stride]:
        node = live[i]
        k, v = synth.chain_kv(spec, node, "cpu")          # input generation: not timed
        k, v = k.to(torch.float64).numpy(), v.to(torch.float64).numpy()
        t0 = time.perf_counter()
        f = Forest(spec.shape.num_kv_heads, spec.shape.head_dim)
        t = f.new_thread()
        f.append(t, k, v)
        out = tree_decode_attention(f, [t], q_all[i:i + 1], scale)
        spent += time.perf_counter() - t0
        assert np.isfinite(out).all()
        done += 1
        if spent >= budget_s:
            break
    return done, spent


class OraclePool:
    """The checker on all host cores: one single-threaded process per core, each timing its own
    share of the workload's live threads.  Rate = sum of the per-core rates, every core's rate
    taken while all the others were busy as well."""

    def __init__(self, max_cores=None):
        import multiprocessing as mp
        try:
            avail = len(os.sched_getaffinity(0))
        except AttributeError:
            avail = os.cpu_count() or 1
        self.cores = max(1, min(avail, max_cores or 32))
        os.environ.setdefault("OMP_NUM_THREADS", "1")
        os.environ.setdefault("MKL_NUM_THREADS", "1")
        os.environ.setdefault("OPENBLAS_NUM_THREADS", "1")
        self.pool = mp.get_context("spawn").Pool(self.cores)

    def sample(self, cfg_id, seed, n_requests, unshared, budget_s):
        """(thread-tokens per second over all cores, threads done, cores that did work)."""
        jobs = [(cfg_id, seed, n_requests, unshared, w, self.cores, budget_s)
                for w in range(self.cores)]
        res = [r for r in self.pool.map(_oracle_worker, jobs) if r[0] > 0]
        return sum(d / s for d, s in res), sum(d for d, _ in res), len(res)

    def close(self):
        self.pool.close()
        self.pool.join()


def run_reference(args, cfg_id):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = synth.forest_spec(cfg_id, n_requests=args.requests)
    if args.unshared:
        spec = synth.unshared_spec(spec)
    # about a minute of timed checker work per core over the whole run (input generation,
    # untimed, takes about as long again)
    per_step = max(0.5, min(20.0, 60.0 / max(1, args.steps + args.warmup)))
    pool = OraclePool()
    for _ in range(args.warmup):
        pool.sample(cfg_id, spec.seed, args.requests, args.unshared, per_step / 4)
    rates, threads, cores = [], 0, 0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        r, n, cores = pool.sample(cfg_id, spec.seed, args.requests, args.unshared, per_step)
        rates.append(r); threads += n
    wall = time.perf_counter() - t0
    pool.close()
    value = statistics.mean(rates)
    sample = (f"{threads} live threads of {args.workload} over {args.steps} steps on {cores} host "
              f"cores (one single-threaded process per core), one thread at a time: chain "
              f"materialised in fp64 + dense softmax attention, all {spec.shape.num_q_heads} "
              f"query heads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wall / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": workload_config(args.workload, spec, args.unshared, max(1, args.layers),
                                  args.graph, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------ DRAM traffic
def profiled_traffic(workload_key, requests_run):
    """DRAM bytes (read + write) of the attention kernels of one call, from the ncu captures
    summarised in profiles/dram_traffic.txt: taken on a small case of the same kernels and
    scaled by the requests processed (DRAM traffic is proportional to them).  None when there
    is no capture for the workload, or when a kernel source has changed since its capture
    (the file records a digest of every source file)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None, "no capture"
    total, found = 0.0, False
    for line in open(path):
        f = line.split()
        if len(f) < 7 or f[0].startswith("#") or f[0] != workload_key:
            continue
        _, kernel, source, digest, req, rd_mb, wr_mb = f[:7]
        src = os.path.join(ROOT, "paper_2401_06761_b200", "csrc", source)
        if not os.path.exists(src) or hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] != digest:
            return None, f"{source} changed since the capture"
        total += (float(rd_mb) + float(wr_mb)) * 1e6 * requests_run / float(req)
        found = True
    return (total, "profiles/dram_traffic.txt, scaled by requests") if found else (None, "no capture")


# ------------------------------------------------------------------------------ GPU arm
class DeviceRun:
    """One workload on this rank's GPU: builds the forest through the library, runs steps."""

    def __init__(self, name, cfg_id, unshared, args, dev, rank, steps_total, layers=1):
        from paper_2401_06761_b200 import binding as B
        from paper_2401_06761_b200.session import pool_requirements
        self.B, self.name, self.cfg_id, self.unshared, self.dev = B, name, cfg_id, unshared, dev
        spec = sharding.shard_spec(cfg_id, rank, n_requests=args.requests)
        if unshared:
            spec = synth.unshared_spec(spec)
        self.spec, self.shape, self.L = spec, spec.shape, layers
        nb, nt, mb = pool_requirements(spec)
        self.T = len(spec.live_nodes())
        steps_total += 12          # the host-cost pass after the timed steps
        self.n_step_forks = sum(1 for n in spec.nodes if n.step_fork)
        grow = (self.T + self.n_step_forks) * (2 * steps_total // 16 + 2) + 2 * self.n_step_forks
        self.dims = (nb + grow, nt + self.n_step_forks, mb + 2 * steps_total // 16 + 2)
        self.sess = self.step0 = self.graph = None
        self.setup_s = 0.0
        self.attn_events = []
        g = torch.Generator(device=dev).manual_seed(spec.seed + 99)
        self.row_shape = (self.T, self.shape.num_kv_heads, self.shape.head_dim)
        self.q_shape = (self.T, self.shape.num_q_heads, self.shape.head_dim)
        self.inputs = [tuple(torch.randn(s, generator=g, device=dev).to(torch.bfloat16)
                             for s in (self.q_shape, self.row_shape, self.row_shape))
                       for _ in range(min(4, steps_total))]
        self.out = torch.empty(self.q_shape, dtype=torch.bfloat16, device=dev)
        self.stream = torch.cuda.current_stream().cuda_stream
        self.small = spec.unique_tokens() * self.shape.bytes_per_token < 4 * 126e6

    def make_session(self):
        from paper_2401_06761_b200.session import PagedSession
        self.close()
        t0 = time.perf_counter()
        self.sess = PagedSession(self.shape, *self.dims, device=self.dev, num_layers=self.L)
        self.step0 = synth.build_forest(self.spec, self.sess, device=self.dev)
        if self.L > 1:      # give the other layers the same rows as layer 0 (setup, untimed)
            for pool in (self.sess.k_pool, self.sess.v_pool):
                per = pool.shape[0] // self.L
                for l in range(1, self.L):
                    pool[l * per:(l + 1) * per].copy_(pool[:per])
        torch.cuda.synchronize()
        self.setup_s = time.perf_counter() - t0
        self.base_live = [h for h, n in zip(self.step0.live_handles, self.step0.live_nodes)
                          if not n.step_fork]
        self.base_live_arr = self.B.int32_array(self.base_live)
        self.attn_events = []

    def close(self):
        if self.sess is not None:
            self.sess.close()
            self.sess = self.step0 = self.graph = None
            torch.cuda.empty_cache()

    def one_step(self, q, k_new, v_new, record, stream=None, out=None, host=None):
        """fork (if the workload has one) + one decode step (apar_decode_step: append of one row
        per live thread + attention) [+ release of the step's forks].  record: the library
        records a pair of CUDA events around the attention kernels of the step.  host: a dict
        that receives the wall time of each library call."""
        B, sess, step0 = self.B, self.sess, self.step0
        stream = self.stream if stream is None else stream
        out = self.out if out is None else out
        t0 = time.perf_counter()
        kids = B.apar_fork(sess.ctx, step0.fork_parents, stream) if step0.fork_parents else []
        live = B.int32_array(self.base_live + kids) if kids else self.base_live_arr
        t1 = time.perf_counter()
        if record:
            pair = self.event_pool[len(self.attn_events)]
            B.apar_set_timing_events(sess.ctx, pair[0].cuda_event, pair[1].cuda_event)
            self.attn_events.append(pair)
        B.apar_decode_step(sess.ctx, live, k_new.data_ptr(), v_new.data_ptr(), q.data_ptr(),
                           out.data_ptr(), sess.sm_scale, stream)
        if record:
            B.apar_set_timing_events(sess.ctx, 0, 0)
        t2 = time.perf_counter()
        if self.graph is not None:        # the other layers, replayed from the captured graph
            if (q.data_ptr(), k_new.data_ptr(), out.data_ptr()) != self.graph_ptrs:
                for dst, src in zip(self.graph_in, (q, k_new, v_new)):
                    dst.copy_(src)
            self.graph.replay()
        else:
            for l in range(1, self.L):      # the other layers: scatter + attention launches only
                B.apar_append_kv_layer(sess.ctx, l, k_new.data_ptr(), v_new.data_ptr(), stream)
                B.apar_tree_decode_attention_layer(sess.ctx, l, q.data_ptr(), out.data_ptr(),
                                                   sess.sm_scale, stream)
        t3 = time.perf_counter()
        if kids:
            B.apar_release(sess.ctx, kids)
        if host is not None:
            t4 = time.perf_counter()
            for key, dt in (("fork", t1 - t0), ("decode_step", t2 - t1), ("other_layers", t3 - t2),
                            ("release", t4 - t3), ("total", t4 - t0)):
                host.setdefault(key, []).append(dt)

    def capture_layer_loop(self):
        """Layers 1.. of a step only launch kernels whose sizes the cached plan fixes: capture
        them once; valid while the plan is reused (threads only grow)."""
        B = self.B
        self.graph_in = [torch.empty_like(t) for t in self.inputs[0]]
        for dst, src in zip(self.graph_in, self.inputs[0]):
            dst.copy_(src)
        gq, gk, gv = self.graph_in
        self.graph_ptrs = (gq.data_ptr(), gk.data_ptr(), self.out.data_ptr())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            cs = torch.cuda.current_stream().cuda_stream
            for l in range(1, self.L):
                B.apar_append_kv_layer(self.sess.ctx, l, gk.data_ptr(), gv.data_ptr(), cs)
                B.apar_tree_decode_attention_layer(self.sess.ctx, l, gq.data_ptr(),
                                                   self.out.data_ptr(), self.sess.sm_scale, cs)
        self.graph = graph

    def timed_device_arm(self, steps, warmup, sync, reduce_ms, clock_index=None, graph=False):
        """`warmup` untimed steps, then exactly `steps` timed ones.  Returns a dict of raw
        results of this rank (times already reduced over ranks by `reduce_ms`)."""
        inputs = self.inputs
        for i in range(warmup):
            self.one_step(*inputs[i % len(inputs)], record=False)
        sync()
        if graph:
            self.capture_layer_loop()
            self.one_step(*inputs[0], record=False)
            sync()
        k0 = self.sess.stats()["kernels_total"]
        # events the library records around the attention kernels of every timed step
        self.event_pool = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                           for _ in range(steps)]
        for a, b in self.event_pool:
            a.record(); b.record()            # creates the handles
        sync()
        self.attn_events = []
        sampler = ClockSampler(clock_index).start() if clock_index is not None else None
        host_t0 = time.perf_counter()
        # A workload whose KV fits in the L2 cache would be timed on cache hits: for those,
        # every step is timed on its own and a buffer larger than L2 is written between steps.
        if self.small:
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=self.dev)
            step_events = []
            for i in range(steps):
                flush.fill_(i & 0xff)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                self.one_step(*inputs[i % len(inputs)], record=True)
                b.record()
                step_events.append((a, b))
            host_ms = 1e3 * (time.perf_counter() - host_t0)
            sync()
            total_ms = reduce_ms(sum(a.elapsed_time(b) for a, b in step_events))
            del flush
        else:
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            for i in range(steps):
                self.one_step(*inputs[i % len(inputs)], record=True)
            ev1.record()
            host_ms = 1e3 * (time.perf_counter() - host_t0)
            sync()
            total_ms = reduce_ms(ev0.elapsed_time(ev1))
        clocks = sampler.stop() if sampler is not None else None
        st = self.sess.stats()
        if st["device_wait_timeouts"]:
            raise SystemExit(f"a kernel gave up a bounded wait (code {st['device_wait_timeouts']}): "
                             "the timed results are invalid")
        attn = sorted(a.elapsed_time(b) for a, b in self.attn_events)
        # What the calls of a step cost the host thread: further steps, each started on an idle
        # GPU (so that no call waits for a staging buffer the GPU still holds), calls timed alone.
        host = {}
        plan_us = []
        for i in range(min(steps, 10)):
            sync()
            self.one_step(*inputs[i % len(inputs)], record=False, host=host)
            plan_us.append(self.B.apar_get_stats(self.sess.ctx)["attn_plan_host_us"])
        sync()
        host_calls = {k: 1e3 * statistics.median(v) for k, v in host.items()}
        host_calls["planner"] = 1e-3 * statistics.median(plan_us)
        return {"total_ms": total_ms, "host_issue_ms": host_ms, "clocks": clocks, "stats": st,
                "launches": st["kernels_total"] - k0, "attn_ms": statistics.mean(attn),
                "attn_ms_median": attn[len(attn) // 2], "attn_ms_min": attn[0], "steps": steps,
                "host_calls_ms": host_calls}

    def summary(self, r, peak):
        """Throughput, byte counts and roofline figures of one timed device arm."""
        st, steps, shape = r["stats"], r["steps"], self.shape
        bpt = shape.bytes_per_token
        # every persistent thread grows by one token per step: the counters of the last timed
        # step are brought back to their mean over the timed steps
        grow = len(self.base_live) * (steps - 1) / 2.0
        unique_tokens = st["attn_unique_tokens"] - grow
        attended_tokens = st["attn_attended_tokens"] - grow
        unique_bytes, unshared_bytes = unique_tokens * bpt, attended_tokens * bpt
        qo_bytes = 2 * self.T * shape.num_q_heads * shape.head_dim * 2
        algo_bytes = unique_bytes + qo_bytes
        achieved = algo_bytes / (r["attn_ms"] * 1e-3) / 1e9
        return {
            "threads": self.T, "steps": steps, "ms_per_step": r["total_ms"] / steps,
            "thread_tokens_per_s": self.T * self.L * steps / (r["total_ms"] * 1e-3),
            "attention_ms": r["attn_ms"], "attention_ms_median": r["attn_ms_median"],
            "attention_ms_min": r["attn_ms_min"],
            "unique_kv_bytes_per_step": unique_bytes, "unshared_kv_bytes_per_step": unshared_bytes,
            "sharing_ratio": unshared_bytes / max(1.0, unique_bytes),
            "unique_tokens": unique_tokens, "attended_tokens": attended_tokens,
            "algorithmic_bytes": algo_bytes, "achieved_gbs": achieved,
            "frac_of_measured_peak": achieved / peak,
            "unique_kv_frac_of_nominal": unique_bytes / (r["attn_ms"] * 1e-3) / 1e9 / 8000.0,
            # wall time of the issuing loop per step (the host runs ahead of the GPU until the
            # staging ring is full, then at the GPU's pace) and the calls' own cost on an idle GPU
            "host_issue_ms_per_step": r["host_issue_ms"] / steps,
            "host_calls_ms_per_step": r["host_calls_ms"]["total"],
            "host_calls_ms": r["host_calls_ms"],
            "gpu_launches": r["launches"], "clocks": r["clocks"],
            "l2": "flushed between steps" if self.small else "inputs larger than L2",
        }


def lifecycle_report(dev, n_requests=96, n_steps=1500, max_live=96):
    """Early release as a measurement (Section 2.4 feature 2; "max cached tokens", Section 3.4):
    a seeded stream of requests whose threads fork and finish at different steps is replayed
    through the library twice, once giving a finished thread's cache back at once and once only
    when its whole request has finished.  Both peaks are the library's own counter."""
    from paper_2401_06761_b200.session import PagedSession
    shape = synth.LAYER_SHAPES[1]
    steps, req = synth.lifecycle_schedule(seed=7, n_requests=n_requests, n_steps=n_steps,
                                          max_live=max_live)
    z = torch.zeros((4096, shape.num_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=dev)
    q = torch.zeros((max_live + 8, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16,
                    device=dev)
    rep = {"requests": n_requests, "steps": n_steps, "max_live_threads": max_live,
           "threads": len(req), "forks": sum(len(s.fork) for s in steps)}
    table_blocks = synth.lifecycle_longest_thread(steps) // shape.block_size + 2
    for early in (True, False):
        sess = PagedSession(shape, 16384, len(req) + 8, table_blocks, device=dev)
        tokens = [0]

        def rows(n):
            return z[:n], z[:n]

        def on_step(i, live):
            tokens[0] += len(live)
            sess.attention(live, q[:len(live)])

        t0 = time.perf_counter()
        synth.run_lifecycle(steps, req, sess, rows, early_release=early, on_step=on_step)
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
        st = sess.stats()
        assert st["free_blocks"] == 16384 and st["device_wait_timeouts"] == 0
        key = "early_release" if early else "release_at_request_end"
        rep[key] = {"peak_cached_tokens": 16 * st["peak_used_blocks"],
                    "peak_used_blocks": st["peak_used_blocks"],
                    "thread_tokens": tokens[0], "wall_s": wall}
        sess.close()
    rep["peak_saving"] = 1.0 - (rep["early_release"]["peak_cached_tokens"] /
                                rep["release_at_request_end"]["peak_cached_tokens"])
    return rep


def run_prefill(args):
    """--workload prefill: the tensor-core side of the path.  A step = 64 new prompts of 2048
    tokens (7B-like MHA layer: 32 heads) appended into the paged pool + tree-masked attention
    over all of their tokens (every token attends the tokens before it) + release.  A second
    arm applies the paragraph-tree mask of Section 2.2 to every token of a config-3-shaped
    forest (each node a segment that attends its ancestors and, causally, itself)."""
    from paper_2401_06761_b200 import build
    build.build()
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession, pool_requirements
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("--workload prefill runs on one GPU")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) \
        if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    peak_tf = float(peaks.get("bf16_tflops_sustained", 1400.0))
    peak_kind = "measured, sustained" if peaks else "fallback"
    n_prompts, plen = args.requests or 64, 2048
    shape = synth.LAYER_SHAPES[2]
    sess = PagedSession(shape, n_prompts * plen // 16 + 64, n_prompts + 8, plen // 16 + 1,
                        device=dev)
    g = torch.Generator(device=dev).manual_seed(2024)
    rows = n_prompts * plen
    k = torch.randn((rows, shape.num_kv_heads, 128), generator=g, device=dev).to(torch.bfloat16)
    v = torch.randn((rows, shape.num_kv_heads, 128), generator=g, device=dev).to(torch.bfloat16)
    q = torch.randn((rows, shape.num_q_heads, 128), generator=g, device=dev).to(torch.bfloat16)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream().cuda_stream
    flops = 4.0 * 128 * shape.num_q_heads * n_prompts * (plen * (plen + 1) / 2)

    def step(events=None):
        tids = B.apar_new_threads(sess.ctx, n_prompts)
        B.apar_append_kv(sess.ctx, tids, [plen] * n_prompts, k.data_ptr(), v.data_ptr(), stream)
        if events:
            B.apar_set_timing_events(sess.ctx, events[0].cuda_event, events[1].cuda_event)
        B.apar_tree_prefill_attention(sess.ctx, 0, tids, [0] * n_prompts, [plen] * n_prompts,
                                      q.data_ptr(), out.data_ptr(), sess.sm_scale, stream)
        if events:
            B.apar_set_timing_events(sess.ctx, 0, 0)
        B.apar_release(sess.ctx, tids)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    pool = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            for _ in range(args.steps)]
    for a, b in pool:
        a.record(); b.record()
    torch.cuda.synchronize()
    sampler = ClockSampler(0).start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k0 = sess.stats()["kernels_total"]
    ev0.record()
    for i in range(args.steps):
        step(pool[i])
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = ev0.elapsed_time(ev1)
    attn_ms = statistics.mean(a.elapsed_time(b) for a, b in pool)
    st = sess.stats()
    if st["device_wait_timeouts"]:
        raise SystemExit("a kernel gave up a bounded wait: the timed results are invalid")
    launches = st["kernels_total"] - k0
    sess.close()
    del k, v, q, out
    torch.cuda.empty_cache()

    # ---- the paragraph-tree mask on a config-3-shaped forest: every token of every node
    spec = synth.forest_spec(3, n_requests=64)
    nb, nt, mb = pool_requirements(spec)
    tsess = PagedSession(spec.shape, nb, nt, mb, device=dev)
    tstep = synth.build_forest(spec, tsess, device=dev)
    synth.run_step_forks(tstep, tsess)
    tsess.append(tstep.live_handles, None, tstep.k_new, tstep.v_new)
    segs = []
    for node in spec.nodes:
        h = tstep.handles[node.index]
        total = tsess.thread(h)[0]
        own = node.n_tok
        segs.append((h, spec.attended_tokens(node) - own, own))
    # (a node that was forked from keeps only its own tokens: children hold theirs)
    t_tids = [s[0] for s in segs]
    t_begin = [s[1] for s in segs]
    t_count = [s[2] for s in segs]
    nq = sum(t_count)
    tq = torch.randn((nq, spec.shape.num_q_heads, 128), generator=torch.Generator(device=dev)
                     .manual_seed(7), device=dev).to(torch.bfloat16)
    tout = torch.empty_like(tq)
    t_flops = 4.0 * 128 * spec.shape.num_q_heads * sum(b * c + c * (c + 1) / 2
                                                     for b, c in zip(t_begin, t_count))
    for _ in range(3):
        tsess.prefill_attention(t_tids, t_begin, t_count, tq, out=tout)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 10
    e0.record()
    for _ in range(reps):
        tsess.prefill_attention(t_tids, t_begin, t_count, tq, out=tout)
    e1.record()
    torch.cuda.synchronize()
    tree_ms = e0.elapsed_time(e1) / reps
    assert tsess.stats()["device_wait_timeouts"] == 0
    tsess.close()

    achieved = flops / (attn_ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": METRIC, "value": rows * args.steps / (total_ms * 1e-3), "unit": UNIT,
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "prefill", "prompts": n_prompts, "prompt_tokens": plen,
                   "num_q_heads": shape.num_q_heads, "num_kv_heads": shape.num_kv_heads,
                   "head_dim": 128, "block_size": 16,
                   "step": "new threads + append of all prompt rows + tree-masked attention "
                           "over every token + release",
                   "l2": "K, V, Q and out of a step are 2.1 GB, larger than L2",
                   "note": "value counts query tokens (one per prompt position) per second"},
        "clocks": clocks, "gpu_launches": launches,
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
                     "frac": achieved / peak_tf, "traffic": None,
                     "peak_kind": f"cuBLAS bf16 GEMM, {peak_kind}",
                     "flops_per_step": flops, "attention_ms": attn_ms,
                     "kernel": "attn_prefill_kernel: tcgen05, 2 x 128 query rows per CTA share the K/V tiles"},
        "tree_mask": {"workload": "every token of a config-3-shaped forest of 64 requests",
                      "queries": nq, "segments": len(segs), "ms": tree_ms,
                      "tflops": t_flops / (tree_ms * 1e-3) / 1e12,
                      "frac_of_peak": t_flops / (tree_ms * 1e-3) / 1e12 / peak_tf,
                      "note": "host planning and uploads of the call included"},
    }))


def run_ours(args):
    from paper_2401_06761_b200 import build
    build.build()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def sync():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_ms(ms):
        return sharding.reduce_timing(ms, 0.0, dist, dev)[0]

    peak, peak_kind = measured_peaks()
    if args.workload == "lifecycle":
        if rank == 0:
            rep = lifecycle_report(dev)
            e = rep["early_release"]
            print(json.dumps({
                "metric": METRIC, "value": e["thread_tokens"] / e["wall_s"], "unit": UNIT,
                "n_gpus": 1, "steps": rep["steps"], "warmup": 0,
                "ms_per_step": 1e3 * e["wall_s"] / rep["steps"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "lifecycle"}, "lifecycle": rep}))
        return
    cfg_id = parse_workload(args.workload)
    L = max(1, args.layers)
    steps_total = args.warmup + args.steps
    run = DeviceRun(args.workload, cfg_id, args.unshared, args, dev, rank, steps_total, L)
    if args.graph and (L < 2 or any(n.step_fork for n in run.spec.nodes)):
        raise SystemExit("--graph needs --layers >= 2 and a workload without forks in the step")

    # ---------------- device-resident arm
    run.make_session()
    t_setup = run.setup_s
    r = run.timed_device_arm(args.steps, args.warmup, sync, reduce_ms,
                             clock_index=local if rank == 0 else None, graph=args.graph)
    head = run.summary(r, peak)
    T, shape = run.T, run.shape
    q_shape, row_shape = run.q_shape, run.row_shape
    out, inputs = run.out, run.inputs

    # ---------------- end-to-end arm: host buffers in, host buffer out, copies inside the timing
    hq = [torch.empty(q_shape, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    hk = [torch.empty(row_shape, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    hv = [torch.empty(row_shape, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    hout = torch.empty(q_shape, dtype=torch.bfloat16).pin_memory()
    for i in range(2):
        hq[i].copy_(inputs[i % len(inputs)][0]); hk[i].copy_(inputs[i % len(inputs)][1])
        hv[i].copy_(inputs[i % len(inputs)][2])
    # A serving loop would overlap the copies of neighbouring steps with compute, so the end-to-
    # end arm does: inputs of step i+1 go up (copy stream) and the result of step i-1 comes
    # down (second copy stream) while step i computes, with two device buffers of each kind.
    # Every step's own copies are inside the timed region.
    dq = [torch.empty(q_shape, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    dk = [torch.empty(row_shape, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    dv = [torch.empty(row_shape, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    dout = [torch.empty(q_shape, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    s_cmp = torch.cuda.current_stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_cmp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        b = i % 2
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(ev_cmp[b])          # step i-2 has consumed these input buffers
            dq[b].copy_(hq[b], non_blocking=True)
            dk[b].copy_(hk[b], non_blocking=True)
            dv[b].copy_(hv[b], non_blocking=True)
            ev_in[b].record(s_in)
        s_cmp.wait_event(ev_in[b])
        if i >= 2:
            s_cmp.wait_event(ev_out[b])             # the result of step i-2 has left dout[b]
        run.one_step(dq[b], dk[b], dv[b], record=False, out=dout[b])
        ev_cmp[b].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[b])
            hout.copy_(dout[b], non_blocking=True)
            ev_out[b].record(s_out)

    # The end-to-end arm starts from the same forest as the device arm did (every step makes
    # each thread one token longer, so carrying on would time a larger problem): rebuild it,
    # then the same number of warm-up steps, untimed.
    run.make_session()
    e2e_steps = args.steps
    for i in range(args.warmup):
        e2e_step(i)
    sync()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    s_cmp.wait_event(ev_out[(e2e_steps - 1) % 2])
    if e2e_steps >= 2:
        s_cmp.wait_event(ev_out[e2e_steps % 2])
    ev1.record()
    sync()
    e2e_ms = reduce_ms(ev0.elapsed_time(ev1))
    h2d = sum(t[0].numel() * 2 for t in (dq, dk, dv))
    d2h = out.numel() * 2

    # the same copies alone, both directions at once: the PCIe time a step cannot go below
    def copies_only():
        with torch.cuda.stream(s_in):
            dq[0].copy_(hq[0], non_blocking=True)
            dk[0].copy_(hk[0], non_blocking=True)
            dv[0].copy_(hv[0], non_blocking=True)
        with torch.cuda.stream(s_out):
            hout.copy_(dout[0], non_blocking=True)
    copies_only()
    torch.cuda.synchronize()
    reps = 10
    t_c = time.perf_counter()
    for _ in range(reps):
        copies_only()
    torch.cuda.synchronize()
    copy_ms = 1e3 * (time.perf_counter() - t_c) / reps
    run.close()
    del hq, hk, hv, hout, dq, dk, dv, dout

    # ---------------- the rest of the contract: longer run, other workloads, early release
    extras = {}
    default_line = (world == 1 and not args.no_sweep and args.workload == "cfg4" and
                    not args.unshared and args.requests is None and L == 1)
    if default_line:
        n_sus = args.sustained_steps
        sus = DeviceRun(args.workload, cfg_id, False, args, dev, rank, n_sus + args.warmup, 1)
        sus.make_session()
        extras["sustained"] = sus.summary(
            sus.timed_device_arm(n_sus, args.warmup, sync, reduce_ms, clock_index=local), peak)
        sus.close()
        del sus
        sweep = {}
        for name, unshared in SWEEP:
            n_sw = max(30, args.sweep_steps)
            w = DeviceRun(name, parse_workload(name), unshared, args, dev, rank,
                          n_sw + args.warmup, 1)
            w.make_session()
            sweep[name + ("-unshared" if unshared else "")] = w.summary(
                w.timed_device_arm(n_sw, args.warmup, sync, reduce_ms, clock_index=local), peak)
            w.close()
            del w
        extras["sweep"] = sweep
        extras["lifecycle"] = lifecycle_report(dev)

    # ---------------- numbers
    total_T = sharding.reduce_timing(0.0, float(T), dist, dev)[1]
    value = total_T * L * args.steps / (r["total_ms"] * 1e-3)
    e2e_value = total_T * L * e2e_steps / (e2e_ms * 1e-3)
    read_peak = read_only_rate(dev) if rank == 0 else None
    traffic, traffic_src = (None, "not the profiled workload")
    if L == 1 and world == 1:
        traffic, traffic_src = profiled_traffic(
            args.workload + ("-unshared" if args.unshared else ""),
            len({n.request for n in run.spec.nodes}))

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": r["total_ms"] / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": workload_config(args.workload, run.spec, args.unshared, L, args.graph, world),
            "clocks": r["clocks"],
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps,
                    # host<->device copies of one step alone (up and down overlapped): the
                    # end-to-end step is bound by them whenever they take longer than the compute
                    "copies_only_ms": copy_ms,
                    "copies_only_gbs": (h2d + d2h) / (copy_ms * 1e-3) / 1e9},
            "gpu_launches": r["launches"],
            "roofline": {
                "bound": "hbm", "achieved": head["achieved_gbs"], "peak": peak, "unit": "GB/s",
                "frac": head["achieved_gbs"] / peak, "traffic": traffic,
                "traffic_source": traffic_src,
                "peak_kind": f"of {peak_kind} copy bandwidth",
                # the same achieved rate against two other ceilings: this library's read-only
                # streaming probe, run just now on this GPU, and the nominal HBM3e figure
                "peak_read_only": read_peak,
                "frac_of_read_only": head["achieved_gbs"] / read_peak,
                "peak_nominal": 8000.0, "frac_of_nominal": head["achieved_gbs"] / 8000.0,
                "unique_kv_frac_of_nominal": head["unique_kv_frac_of_nominal"],
                "attention_ms_median": head["attention_ms_median"],
                "attention_ms_min": head["attention_ms_min"],
                "kernel": "the attention kernels of apar_decode_step (tcgen05 + warp-stream + single-row + merge launches), between events the library records on the stream",
                "algorithmic_bytes": head["algorithmic_bytes"], "attention_ms": head["attention_ms"],
            },
            "kv_bytes": {"unique_per_step": head["unique_kv_bytes_per_step"],
                         "unshared_per_step": head["unshared_kv_bytes_per_step"],
                         "sharing_ratio": head["sharing_ratio"],
                         "attended_tokens_per_thread": head["attended_tokens"] / T,
                         "unique_tokens": head["unique_tokens"],
                         "note": "means over the timed steps (threads grow one token per step)"},
            "plan": {"work_items": r["stats"]["attn_work_items"],
                     "vec_items": r["stats"]["attn_vec_items"],
                     "mma_items": r["stats"]["attn_mma_items"],
                     "partials": r["stats"]["attn_partials"],
                     "reused_last_step": r["stats"]["attn_plan_reused"],
                     "host_issue_ms_per_step": head["host_issue_ms_per_step"],
                     "host_calls_ms_per_step": head["host_calls_ms_per_step"],
                     "host_calls_ms": head["host_calls_ms"]},
            "setup_s": t_setup,
        }
        line.update(extras)
        if world == 1 and not args.skip_cpu_baseline:
            pool = OraclePool()
            cpu_rate, cpu_threads, cores = pool.sample(cfg_id, run.spec.seed, args.requests,
                                                       args.unshared, 10.0)
            pool.close()
            line["cpu_baseline"] = {
                "value": cpu_rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"{cpu_threads} live threads of {args.workload} on {cores} host cores "
                          f"(one single-threaded process per core, about 10 s of checker time "
                          f"each), one thread at a time: fp64 chain materialisation + dense "
                          f"attention, all query heads"}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--requests", type=int, default=None,
                    help="shrink the workload to this many requests (profiling captures)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true",
                    help="only the headline workload: no sustained run, no other configurations")
    ap.add_argument("--sustained-steps", type=int, default=300,
                    help="steps of the longer run of the headline workload (default line only)")
    ap.add_argument("--sweep-steps", type=int, default=50,
                    help="timed steps of each of the other configurations (at least 30)")
    ap.add_argument("--unshared", action="store_true",
                    help="same live threads, but every thread owns a private copy of its whole "
                         "chain (the copy-the-prefix-on-fork policy); for comparison with the tree")
    ap.add_argument("--graph", action="store_true",
                    help="with --layers >= 2: layers 1.. of a step are replayed from a CUDA graph "
                         "(device arm only)")
    ap.add_argument("--layers", type=int, default=1,
                    help="attention layers per step (layers > 0 replay the plan; default 1)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.workload == "prefill":
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable":
                              "the prefill workload is timed on the GPU arm only"}))
        else:
            run_prefill(args)
    elif args.impl == "reference":
        run_reference(args, parse_workload(args.workload))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

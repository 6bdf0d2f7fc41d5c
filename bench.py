#!/usr/bin/env python
"""Benchmark of the APAR decode hot path on B200: one step = (the step's fork, if the workload
has one) + KV append of one token per live thread + tree decode attention over all live
threads, for one attention layer.  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

With N > 1 (under torchrun) every rank runs its own shard of requests (a different seed of the
same workload) on its own GPU; there is no exchange between shards.
"""
from __future__ import annotations

import argparse
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
                 "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
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
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def parse_workload(name: str) -> int:
    if not (name.startswith("cfg") and name[3:].isdigit() and int(name[3:]) in synth.LAYER_SHAPES):
        raise SystemExit(f"unknown workload {name}; use cfg1..cfg5")
    return int(name[3:])


# ------------------------------------------------------------------------------ CPU baseline
def oracle_sample(spec, budget_s: float, min_threads: int = 2):
    """Times the fp64 checker, as it stands, on live threads of `spec` until the budget is used.
    Returns (thread-tokens per second, threads done, cores used)."""
    import numpy as np
    from oracle import Forest, tree_decode_attention
    torch.set_num_threads(1)
    live = spec.live_nodes()
    order = list(range(0, len(live), max(1, len(live) // 64))) + list(range(len(live)))
    scale = spec.shape.head_dim ** -0.5
    q_all = synth.queries(spec, len(live), "cpu").to(torch.float64).numpy()
    done, spent = 0, 0.0
    for i in order:
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
        if spent >= budget_s and done >= min_threads:
            break
    return done / spent, done, 1


def run_reference(args, cfg_id):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = synth.forest_spec(cfg_id)
    # about a minute of timed oracle work over the whole run (input generation, untimed, takes
    # about as long again)
    per_step = max(0.5, min(20.0, 60.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(spec, per_step / 4)
    rates, threads = [], 0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        r, n, cores = oracle_sample(spec, per_step)
        rates.append(r); threads += n
    wall = time.perf_counter() - t0
    value = statistics.mean(rates)
    sample = (f"{threads} live threads of {args.workload} over {args.steps} steps, one thread "
              f"at a time: chain materialised in fp64 + dense softmax attention, all "
              f"{spec.shape.num_q_heads} query heads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wall / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": args.workload},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------ GPU arm
def run_ours(args, cfg_id):
    from paper_2401_06761_b200 import build
    build.build()
    from paper_2401_06761_b200.session import PagedSession, pool_requirements

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

    # shard = the same workload with a rank-specific seed: independent requests, no exchange
    spec = sharding.shard_spec(cfg_id, rank, n_requests=args.requests)
    if args.unshared:
        spec = synth.unshared_spec(spec)
    shape = spec.shape
    steps_total = args.warmup + args.steps
    nb, nt, mb = pool_requirements(spec)
    n_live = len(spec.live_nodes())
    n_step_forks = sum(1 for n in spec.nodes if n.step_fork)
    grow_blocks = (n_live + n_step_forks) * (2 * steps_total // 16 + 2) + 2 * n_step_forks
    L = max(1, args.layers)
    from paper_2401_06761_b200 import binding as B

    class S:      # the session in use: the end-to-end arm rebuilds it, see below
        sess = step0 = base_live = base_live_arr = None
        setup_s = 0.0
        graph = graph_in = graph_ptrs = None

    def make_session():
        if S.sess is not None:
            S.sess.close()
            S.sess = S.step0 = S.graph = None
            torch.cuda.empty_cache()
        t0 = time.perf_counter()
        S.sess = PagedSession(shape, nb + grow_blocks, nt + n_step_forks,
                              mb + 2 * steps_total // 16 + 2, device=dev, num_layers=L)
        S.step0 = synth.build_forest(spec, S.sess, device=dev)
        if L > 1:      # give the other layers the same rows as layer 0 (setup, untimed)
            for pool in (S.sess.k_pool, S.sess.v_pool):
                per = pool.shape[0] // L
                for l in range(1, L):
                    pool[l * per:(l + 1) * per].copy_(pool[:per])
        torch.cuda.synchronize()
        S.setup_s = time.perf_counter() - t0
        S.base_live = [h for h, n in zip(S.step0.live_handles, S.step0.live_nodes)
                       if not n.step_fork]
        S.base_live_arr = B.int32_array(S.base_live)

    make_session()
    t_setup = S.setup_s
    stream = torch.cuda.current_stream().cuda_stream
    T = n_live
    g = torch.Generator(device=dev).manual_seed(spec.seed + 99)
    row_shape = (T, shape.num_kv_heads, shape.head_dim)
    q_shape = (T, shape.num_q_heads, shape.head_dim)

    def fresh(shp):
        return torch.randn(shp, generator=g, device=dev).to(torch.bfloat16)

    out = torch.empty(q_shape, dtype=torch.bfloat16, device=dev)
    attn_events = []

    def one_step(q, k_new, v_new, record, stream=stream, out=out):
        """fork (if the workload has one) + append + attention [+ release of the step's forks]."""
        sess, step0 = S.sess, S.step0
        kids = B.apar_fork(sess.ctx, step0.fork_parents, stream) if step0.fork_parents else []
        live = B.int32_array(S.base_live + kids) if kids else S.base_live_arr
        B.apar_append_kv(sess.ctx, live, None, k_new.data_ptr(), v_new.data_ptr(), stream)
        if record:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        B.apar_tree_decode_attention(sess.ctx, live, q.data_ptr(), out.data_ptr(), sess.sm_scale,
                                     stream)
        if record:
            e1.record()
            attn_events.append((e0, e1))
        if S.graph is not None:        # the other layers, replayed from the captured graph
            if (q.data_ptr(), k_new.data_ptr(), out.data_ptr()) != S.graph_ptrs:
                S.graph_in[0].copy_(q); S.graph_in[1].copy_(k_new); S.graph_in[2].copy_(v_new)
            S.graph.replay()
        else:
            for l in range(1, L):      # the other layers: scatter + attention launches only
                B.apar_append_kv_layer(sess.ctx, l, k_new.data_ptr(), v_new.data_ptr(), stream)
                B.apar_tree_decode_attention_layer(sess.ctx, l, q.data_ptr(), out.data_ptr(),
                                                   sess.sm_scale, stream)
        if kids:
            B.apar_release(sess.ctx, kids)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return sharding.reduce_timing(ms, 0.0, dist, dev)[0]

    # ---------------- device-resident arm
    inputs = [(fresh(q_shape), fresh(row_shape), fresh(row_shape)) for _ in range(min(4, steps_total))]
    for i in range(args.warmup):
        one_step(*inputs[i % len(inputs)], record=False)
    barrier()

    def capture_layer_loop(out_buf):
        """Layers 1.. of a step only launch kernels whose sizes the cached plan fixes: capture
        them once; valid while the plan is reused (threads only grow)."""
        S.graph_in = [torch.empty_like(inputs[0][0]), torch.empty_like(inputs[0][1]),
                      torch.empty_like(inputs[0][2])]
        for dst, src in zip(S.graph_in, inputs[0]):
            dst.copy_(src)
        gq, gk, gv = S.graph_in
        S.graph_ptrs = (gq.data_ptr(), gk.data_ptr(), out_buf.data_ptr())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            cs = torch.cuda.current_stream().cuda_stream
            for l in range(1, L):
                B.apar_append_kv_layer(S.sess.ctx, l, gk.data_ptr(), gv.data_ptr(), cs)
                B.apar_tree_decode_attention_layer(S.sess.ctx, l, gq.data_ptr(), out_buf.data_ptr(),
                                                   S.sess.sm_scale, cs)
        S.graph = graph

    if args.graph:
        if L < 2 or S.step0.fork_parents:
            raise SystemExit("--graph needs --layers >= 2 and a workload without forks in the step")
        capture_layer_loop(out)
        one_step(*inputs[0], record=False)
        barrier()
    k0 = S.sess.stats()["kernels_total"]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    host_t0 = time.perf_counter()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # A workload whose KV fits in the L2 cache would be timed on cache hits: for those, every
    # step is timed on its own and a buffer larger than L2 is written between the steps.
    small = spec.unique_tokens() * shape.bytes_per_token < 4 * 126e6
    if small:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        step_events = []
        for i in range(args.steps):
            flush.fill_(i & 0xff)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            one_step(*inputs[i % len(inputs)], record=True)
            b.record()
            step_events.append((a, b))
        host_issue_ms = 1e3 * (time.perf_counter() - host_t0)
        barrier()
        total_ms = max_over_ranks(sum(a.elapsed_time(b) for a, b in step_events))
        del flush
    else:
        ev0.record()
        for i in range(args.steps):
            one_step(*inputs[i % len(inputs)], record=True)
        ev1.record()
        host_issue_ms = 1e3 * (time.perf_counter() - host_t0)
        barrier()
        total_ms = max_over_ranks(ev0.elapsed_time(ev1))
    clocks = sampler.stop() if rank == 0 else None
    launches = S.sess.stats()["kernels_total"] - k0
    attn_ms = statistics.mean(a.elapsed_time(b) for a, b in attn_events)
    st = S.sess.stats()
    n_base_live, has_fork = len(S.base_live), bool(S.step0.fork_parents)
    if st["device_wait_timeouts"]:
        raise SystemExit(f"a kernel gave up a bounded wait (code {st['device_wait_timeouts']}): "
                         "the timed results are invalid")

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
        one_step(dq[b], dk[b], dv[b], record=False, out=dout[b])
        ev_cmp[b].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[b])
            hout.copy_(dout[b], non_blocking=True)
            ev_out[b].record(s_out)

    # The end-to-end arm starts from the same forest as the device arm did (every step makes
    # each thread one token longer, so carrying on would time a larger problem): rebuild it,
    # then the same number of warm-up steps, untimed.
    make_session()
    e2e_steps = args.steps
    for i in range(args.warmup):
        e2e_step(i)
    barrier()
    ev0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    s_cmp.wait_event(ev_out[(e2e_steps - 1) % 2])
    if e2e_steps >= 2:
        s_cmp.wait_event(ev_out[e2e_steps % 2])
    ev1.record()
    barrier()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1))
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

    # ---------------- numbers
    total_T = sharding.reduce_timing(0.0, float(T), dist, dev)[1]
    value = total_T * L * args.steps / (total_ms * 1e-3)
    e2e_value = total_T * L * e2e_steps / (e2e_ms * 1e-3)
    bpt = shape.bytes_per_token
    # every persistent thread grows by one token per step: the counters of the last timed step
    # are brought back to their mean over the timed steps
    grow = n_base_live * (args.steps - 1) / 2.0
    unique_tokens = st["attn_unique_tokens"] - grow
    attended_tokens = st["attn_attended_tokens"] - grow
    unique_bytes = unique_tokens * bpt
    unshared_bytes = attended_tokens * bpt
    qo_bytes = 2 * T * shape.num_q_heads * shape.head_dim * 2
    algo_bytes = unique_bytes + qo_bytes
    peak, peak_kind = measured_peaks()
    achieved = algo_bytes / (attn_ms * 1e-3) / 1e9
    attn_all = sorted(a.elapsed_time(b) for a, b in attn_events)
    read_peak = read_only_rate(dev) if rank == 0 else None
    # DRAM bytes (read + write) of the attention kernels of one call, from the ncu captures
    # summarised under profiles/ (taken on a 64-request case of the same kernels and scaled by
    # the requests processed; DRAM traffic is proportional to them).  Only for the full cfg4.
    traffic = None
    if cfg_id == 4 and args.requests is None and not args.unshared and L == 1:
        traffic = ((546.5 + 30.8) + (735.6 + 12.8)) * 1e6 * (512 / 64)

    if rank == 0:
        cpu_rate, cpu_threads, cores = (oracle_sample(spec, 12.0)
                                        if world == 1 and not args.skip_cpu_baseline
                                        else (None, 0, 0))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {
                "workload": args.workload + ("-unshared" if args.unshared else ""),
                "threads_per_gpu": T, "requests": args.requests or synth.DEFAULT_REQUESTS[cfg_id],
                "num_q_heads": shape.num_q_heads, "num_kv_heads": shape.num_kv_heads,
                "head_dim": shape.head_dim, "block_size": shape.block_size,
                "step": ("fork+" if has_fork else "") + "append+attention, " +
                        ("one layer" if L == 1 else f"{L} layers (value counts thread-tokens "
                                                    f"per layer)") +
                        (", layers 1.. replayed from a CUDA graph" if args.graph else ""),
                "l2": "inputs larger than L2 (unique KV bytes per step >> 126 MB)"
                      if not small else "KV fits in L2: 256 MB written between steps, each step "
                                        "timed on its own (device arm)",
                "parallelism": f"{world} independent shard(s), no collective",
            },
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps,
                    # host<->device copies of one step alone (up and down overlapped): the
                    # end-to-end step is bound by them whenever they take longer than the compute
                    "copies_only_ms": copy_ms,
                    "copies_only_gbs": (h2d + d2h) / (copy_ms * 1e-3) / 1e9},
            "gpu_launches": launches,
            "roofline": {
                "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic,
                "peak_kind": f"of {peak_kind} copy bandwidth",
                # the same achieved rate against two other ceilings: this library's read-only
                # streaming probe, run just now on this GPU, and the nominal HBM3e figure
                "peak_read_only": read_peak, "frac_of_read_only": achieved / read_peak,
                "peak_nominal": 8000.0, "frac_of_nominal": achieved / 8000.0,
                "attention_ms_median": attn_all[len(attn_all) // 2],
                "attention_ms_min": attn_all[0],
                "kernel": "apar_tree_decode_attention call (table sync + attention + merge launches)",
                "algorithmic_bytes": algo_bytes, "attention_ms": attn_ms,
            },
            "kv_bytes": {"unique_per_step": unique_bytes, "unshared_per_step": unshared_bytes,
                         "sharing_ratio": unshared_bytes / max(1, unique_bytes),
                         "attended_tokens_per_thread": attended_tokens / T,
                         "unique_tokens": unique_tokens,
                         "note": "means over the timed steps (threads grow one token per step)"},
            "plan": {"work_items": st["attn_work_items"], "vec_items": st["attn_vec_items"],
                     "mma_items": st["attn_mma_items"], "partials": st["attn_partials"],
                     "reused_last_step": st["attn_plan_reused"],
                     "host_issue_ms_per_step": host_issue_ms / args.steps},
            "setup_s": t_setup,
        }
        if cpu_rate is not None:
            line["cpu_baseline"] = {
                "value": cpu_rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"{cpu_threads} live threads of {args.workload}, one at a time "
                          f"(fp64 chain materialisation + dense attention, all query heads)"}
        print(json.dumps(line))
    S.sess.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--requests", type=int, default=None,
                    help="shrink the workload to this many requests (profiling captures)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
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
    cfg_id = parse_workload(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg_id)
    else:
        run_ours(args, cfg_id)


if __name__ == "__main__":
    main()

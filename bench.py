#!/usr/bin/env python
"""Benchmark of the fused sampling / verification path on B200.

A "step" is one fused call (sonic_sample on the heterogeneous-batch workload c2
by default) over one batch of seeded synthetic input.  Inputs rotate over enough
distinct copies that their total footprint exceeds twice the L2 capacity, so
every call reads its logits from HBM.  Calls are captured in CUDA graphs and
timed with CUDA events on the launching stream: a timed block is exactly
`--steps` calls, and blocks are repeated until `--min-time-ms` of device time has
been measured (mean and minimum over the blocks are printed).  With N > 1
(torchrun) every rank runs an independent replica on its own GPU and the slowest
rank's time counts.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_20475_b200 import workloads as wl  # noqa: E402

METRIC = "us_per_fused_sample_call"
L2_BYTES = 126 * 1024 * 1024
PROFILE_TRAFFIC = os.path.join(ROOT, "profiles", "dram_traffic_per_call.txt")


def profiled_traffic(name: str):
    """DRAM bytes (read + write) of one call's kernels and their serialised times, from the ncu summary committed
    under profiles/ (lines `<workload> total <bytes>` and `<workload> kernel <name> <launches per call> <us> <bytes>`).
    Returns (bytes or None, {kernel: {...}}, source file or None)."""
    if not os.path.exists(PROFILE_TRAFFIC):
        return None, {}, None
    total, kernels = None, {}
    for ln in open(PROFILE_TRAFFIC):
        f = ln.split()
        if len(f) >= 3 and f[0] == name and f[1] == "total":
            total = float(f[2])
        elif len(f) >= 6 and f[0] == name and f[1] == "kernel":
            kernels[f[2]] = {"launches_per_call": float(f[3]), "us_per_call_under_ncu": float(f[4]), "dram_bytes_per_call": float(f[5])}
    return total, kernels, os.path.relpath(PROFILE_TRAFFIC, ROOT)


def launches_per_call(name: str, w) -> int:
    """Kernels one call enqueues.  Sampling: streaming, merge, histogram pass, collect pass, row finish, cluster kernel.
    Verification adds the residual pass, the residual draw and the combine kernel.  (sonic_topk: streaming, merge,
    cluster kernel.)"""
    if name == "c4":
        return 9 if w.K > 0 else 7
    if name.startswith("c5"):
        return 3
    return 6


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def make_workload(name: str, copy: int = 0):
    """Workload `name`; `copy` > 0 gives an independent draw of the same recipe."""
    if name == "c1":
        return wl.config1()
    if name == "c2":
        return wl.config2(data_seed=wl.BASE_SEED + 2 + 1000 * copy)
    if name == "c3":
        return wl.config3(data_seed=wl.BASE_SEED + 3 + 1000 * copy)
    if name == "c4":
        return wl.config4(data_seed=wl.BASE_SEED + 4 + 1000 * copy)
    raise ValueError(name)


def algorithmic_bytes(name: str, w) -> int:
    """Bytes a call must read at least once: logits, grammar words, sparse lists (verification: target logits)."""
    if name == "c4":
        return w.sample.input_bytes()
    return w.input_bytes()


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nme, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_time(name: str, w, budget_s: float):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload.  Returns (us per call, description,
    rows of the sample, rows of the sample whose decision margin is below 1e-6)."""
    from oracle import oracle
    import copy as _copy
    if name == "c4":
        vw = w
        nreq = max(1, min(vw.B, 4))
        sub = _copy.copy(vw)
        sub.B = nreq
        sub.sample = _slice_sample(vw.sample, nreq, rows=nreq * (vw.K + 1))
        sub.draft_tokens = vw.draft_tokens[:nreq]
        sub.draft_probs = vw.draft_probs[:nreq]
        t0 = time.perf_counter(); ref = oracle.verify(sub); dt = time.perf_counter() - t0
        near = int((ref["margin"] < 1e-6).sum())
        reps = max(1, int(budget_s / max(dt, 1e-3)) - 1)
        t0 = time.perf_counter()
        for _ in range(reps):
            oracle.verify(sub)
        dt = (time.perf_counter() - t0) / reps if reps else dt
        return dt * vw.B / nreq * 1e6, f"{nreq} of {vw.B} requests x {reps} repetitions, scaled to the full batch", nreq, near
    n = max(1, min(w.B, 8))
    sub = _slice_sample(w, n, rows=n)
    t0 = time.perf_counter(); oracle.sample(sub); dt = time.perf_counter() - t0
    per_row = dt / n
    n2 = int(max(1, min(w.B, budget_s / max(per_row, 1e-6))))
    sub = _slice_sample(w, n2, rows=n2)
    t0 = time.perf_counter(); ref = oracle.sample(sub); dt = time.perf_counter() - t0
    near = int((ref["margin"] < 1e-6).sum())
    return dt * w.B / n2 * 1e6, f"first {n2} of {w.B} rows, one pass, scaled to the full batch", n2, near


def _slice_sample(w, n, rows, start=0):
    import copy as _copy
    s = _copy.copy(w)
    s.B = n
    s.logits = w.logits[start:start + rows]
    for f in ("mode", "temperature", "top_k", "top_p", "min_p", "rep_penalty", "freq_penalty", "pres_penalty", "seed",
              "offset", "hist_ids", "hist_counts", "hist_len", "bias_ids", "bias_vals", "bias_len"):
        v = getattr(w, f)
        setattr(s, f, None if v is None else v[start:start + n])
    if w.bitmask is not None:
        s.bitmask = w.bitmask[start:start + rows]
    return s


def oracle_time_all_cores(name: str, w, budget_s: float):
    """The same oracle with the rows of a singular-mode workload dealt to one thread per host core (the C routine
    releases the interpreter lock).  Returns (us per call scaled to the full batch, threads, description) or None."""
    if name == "c4":
        return None
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle
    cores = len(os.sched_getaffinity(0))
    t0 = time.perf_counter(); oracle.sample(_slice_sample(w, 1, 1)); per_row = time.perf_counter() - t0
    per_thread = int(max(1, min(w.B // max(1, cores), budget_s / max(per_row, 1e-6))))
    threads = min(cores, max(1, w.B // per_thread))
    parts = [_slice_sample(w, per_thread, per_thread, start=i * per_thread) for i in range(threads)]
    with ThreadPoolExecutor(threads) as pool:
        t0 = time.perf_counter()
        list(pool.map(oracle.sample, parts))
        dt = time.perf_counter() - t0
    rows = per_thread * threads
    return dt * w.B / rows * 1e6, threads, f"{rows} of {w.B} rows, {per_thread} per thread, one pass, scaled to the full batch"


def read_probe(gib: float = 1.0, reps: int = 10):
    """Read-only streaming rate of this GPU (the path is read-dominated, the measured peak is a copy): a library
    reduction over a buffer far larger than L2, best of `reps`, CUDA events.  A second denominator, not the target."""
    import torch
    x = torch.empty(int(gib * (1 << 30)) // 4, dtype=torch.float32, device="cuda").fill_(1.0)
    best = float("inf")
    for _ in range(3):
        x.sum()
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); x.sum(); e1.record(); torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) * 1e-3)
    gbs = x.numel() * 4 / best / 1e9
    del x
    return {"gbs": gbs, "bytes": int(gib * (1 << 30)), "how": "torch.sum over fp32, best of %d, CUDA events" % reps}


def config_dict(name, w0, copies=None, bytes_call=None, world=1):
    """The same description of the workload in both arms."""
    B = w0.B
    dt = w0.sample.dtype if hasattr(w0, "sample") else w0.dtype
    cfg = {"workload": f"{name}: B={B}, V={w0.V}, {'bf16' if dt == wl.DTYPE_BF16 else 'fp32'} logits"
                       + (f", K={w0.K}" if name == "c4" else ""),
           "replicas": world}
    if copies is not None:
        cfg["l2"] = f"inputs rotate over {copies} distinct copies ({copies * bytes_call / 1e6:.0f} MB > 2x L2)"
        cfg["timing"] = "CUDA-graph replays, CUDA events on the launching stream"
    else:
        cfg["l2"] = "n/a (host run)"
        cfg["timing"] = "host wall clock"
    return cfg


def run_reference(args, rank, world):
    if rank != 0:
        return
    name = args.workload
    w = make_workload(name)
    B = w.B
    budget = 120.0 / max(1, args.steps + args.warmup)
    times = []
    desc = ""
    for i in range(args.warmup + args.steps):
        us, desc, _, _ = oracle_time(name, w, budget_s=max(0.05, budget))
        if i >= args.warmup:
            times.append(us)
    us = float(np.mean(times))
    out = {
        "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": us / 1000.0, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "impl": "reference",
        "config": config_dict(name, w, world=max(1, args.gpus)),
        "cpu_baseline": {"value": us, "unit": "us", "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def build_device_copies(name, copies, binding):
    import torch
    devs = []
    ws = None
    for c in range(copies):
        w = make_workload(name, copy=c)
        if name == "c4":
            if ws is None:
                ws = binding.new_workspace(w.B * (w.K + 1), w.V)
            devs.append(binding.DeviceVerify(w, ws=ws))
        else:
            if ws is None:
                ws = binding.new_workspace(w.B, w.V)
            devs.append(binding.DeviceSample(w, ws=ws))
    # one eager call per copy: results exist for the row counts, and nothing of the library is set up for the
    # first time inside a capture
    for d in devs:
        d.run()
    torch.cuda.synchronize()
    return devs


def capture(devs, calls):
    """One CUDA graph of `calls` back-to-back fused calls over rotating input copies."""
    import torch
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(calls):
            devs[i % len(devs)].run()
    return g


def time_graph_steps(graph_full, per_graph, graph_rem, rem, steps):
    """Device time (s) of exactly `steps` calls: CUDA events on the launching stream, synchronised on both sides."""
    import torch
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for _ in range(steps // per_graph):
        graph_full.replay()
    if rem:
        graph_rem.replay()
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / 1000.0


def time_blocks(graph_full, per_graph, graph_rem, rem, steps, min_time_s, max_blocks=400):
    """Timed blocks of exactly `steps` calls each, repeated until their device time adds up to `min_time_s`.
    Returns the list of block times (s)."""
    blocks = [time_graph_steps(graph_full, per_graph, graph_rem, rem, steps)]
    while sum(blocks) < min_time_s and len(blocks) < max_blocks:
        blocks.append(time_graph_steps(graph_full, per_graph, graph_rem, rem, steps))
    return blocks


def time_graph_min(graph, per_graph, reps=12):
    """Fastest replay of the graph, per call (CUDA events around every replay)."""
    import torch
    best = float("inf")
    for _ in range(reps):
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        graph.replay()
        e.record()
        torch.cuda.synchronize()
        best = min(best, s.elapsed_time(e) * 1000.0 / per_graph)
    return best


def time_warm_l2(dev, calls=8, reps=12):
    """The same call back to back on ONE input copy (the input stays in L2 when it fits): us per call."""
    import torch
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(calls):
            dev.run()
    for _ in range(3):
        g.replay()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s.record()
    for _ in range(reps):
        g.replay()
    e.record()
    torch.cuda.synchronize()
    return s.elapsed_time(e) * 1000.0 / (calls * reps)


def fallback_rows(name, devs):
    """Rows (requests for c4) per call, over the input copies, that report the cluster kernel (diagnostic flag bit 2)
    and the histogram path (bit 3)."""
    out = {}
    for key, bit in (("cluster", 4), ("dense", 8)):
        per_copy = [int((d.results()["flags"][:(d.vw.B if name == "c4" else None)] & bit).astype(bool).sum()) for d in devs]
        out[key] = {"mean_per_call": float(np.mean(per_copy)), "max_per_call": int(max(per_copy)),
                    "unit": "requests" if name == "c4" else "rows"}
    return out


def measure_floor(calls=64, reps=20):
    """Device time per node of a graph of trivial kernels: the launch floor small calls are compared with."""
    import torch
    x = torch.zeros(1, device="cuda")
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(calls):
            x.add_(1.0)
    for _ in range(3):
        g.replay()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s.record()
    for _ in range(reps):
        g.replay()
    e.record()
    torch.cuda.synchronize()
    return s.elapsed_time(e) * 1000.0 / (calls * reps)


def e2e_measure(name, dev, steps):
    """Same call through the public API from HOST buffers: every step copies the step's inputs host->device from
    pinned memory, runs the fused call and reads the result back."""
    import torch
    s = dev.s if name == "c4" else dev
    pairs = []
    for key, t in s.t.items():
        if t is None:
            continue
        h = t.detach().cpu().pin_memory()
        pairs.append((t, h))
    if name == "c4":
        for t in (dev.draft_tokens, dev.draft_probs):
            pairs.append((t, t.detach().cpu().pin_memory()))
        outs = [dev.out_tokens, dev.out_accept, dev.out_p_draft, s.out_flags]
    else:
        outs = [s.out_token, s.out_prob, s.out_flags, s.out_support]
    houts = [torch.empty_like(o, device="cpu").pin_memory() for o in outs]
    h2d = sum(h.numel() * h.element_size() for _, h in pairs)
    d2h = sum(h.numel() * h.element_size() for h in houts)

    def one():
        for t, h in pairs:
            t.copy_(h, non_blocking=True)
        dev.run()
        for o, h in zip(outs, houts):
            h.copy_(o, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    for _ in range(3):
        one()
    st, en = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    st.record()
    for _ in range(steps):
        one()
    en.record()
    torch.cuda.synchronize()
    return st.elapsed_time(en) * 1000.0 / steps, h2d, d2h


def max_over_ranks(value: float, world: int, device) -> float:
    """Replicas are independent; the job's time is the slowest rank's (all-reduce MAX, NCCL on GPUs, gloo on CPU)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(us_per_call_per_replica: float, world: int) -> float:
    """Whole-job metric: `world` replicas each finish one call per us_per_call, so the job finishes one call every
    us_per_call / world (weak scaling, no data-path collective)."""
    return us_per_call_per_replica / max(1, world)


def run_sonic(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    from paper_2607_20475_b200 import harness as binding

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.lib()
    name = args.workload
    w0 = make_workload(name)
    bytes_call = algorithmic_bytes(name, w0)
    copies = max(2, int(np.ceil(2.0 * L2_BYTES / bytes_call)))
    copies = min(copies, 24)
    devs = build_device_copies(name, copies, binding)
    per_graph = copies
    steps = max(1, args.steps)
    g_full = capture(devs, per_graph)
    rem = steps % per_graph
    g_rem = capture(devs, rem) if rem else None
    # warm-up: at least 3 calls, in whole graphs
    for _ in range(max(1, int(np.ceil(max(3, args.warmup) / per_graph)))):
        g_full.replay()
    if g_rem is not None:
        g_rem.replay()
    torch.cuda.synchronize()

    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else local_rank)
    if rank == 0:
        sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    if args.profile_run:
        args.min_time_ms = 0.0
    blocks = time_blocks(g_full, per_graph, g_rem, rem, steps, args.min_time_ms / 1000.0)
    # keep the sampler busy long enough to see clocks under load
    t_end = time.time() + (0.3 if args.min_time_ms > 0 else 0.0)
    while rank == 0 and time.time() < t_end:
        g_full.replay()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    # every rank's mean over its blocks; the job's time is the slowest rank's
    elapsed = max_over_ranks(float(np.mean(blocks)), world, "cuda")
    clocks = sampler.stop() if rank == 0 else None

    us_call = elapsed / steps * 1e6                     # per replica, mean over the blocks
    us_call_best_block = min(blocks) / steps * 1e6
    if args.profile_run:
        # under a profiler: the timed calls only (no end-to-end leg, probes or CPU baseline), a short line
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": job_value(us_call, world), "unit": "us", "steps": steps,
                              "profile_run": True, "config": config_dict(name, w0, copies, bytes_call, world)}))
        if world > 1:
            dist.destroy_process_group()
        return
    e2e_us, h2d, d2h = e2e_measure(name, devs[0], steps=min(steps, 40))
    e2e_us = max_over_ranks(e2e_us, world, "cuda")
    floor_us = measure_floor() if rank == 0 else None
    min_us = time_graph_min(g_full, per_graph) if rank == 0 else None
    warm_us = time_warm_l2(devs[0]) if rank == 0 else None
    fb = fallback_rows(name, devs) if rank == 0 else None

    extra = {}
    if rank == 0 and args.also:
        for other in [n for n in args.also.split(",") if n and n != name]:
            extra[other] = quick_measure(other, binding)

    if rank == 0:
        peak, which = peaks()
        B = w0.B
        rows = B * (w0.K + 1) if name == "c4" else B
        achieved = bytes_call / (us_call * 1e-6) / 1e9
        n_launch = launches_per_call(name, w0)
        traffic, per_kernel, traffic_src = profiled_traffic(name)
        in_dtype = "bf16" if w0_dtype(w0) == wl.DTYPE_BF16 else "f32"
        cpu_us, cpu_desc, cpu_rows, cpu_near = oracle_time(name, w0, budget_s=15.0)
        cpu_all = oracle_time_all_cores(name, w0, budget_s=6.0)
        probe = read_probe()
        out = {
            "metric": METRIC, "value": job_value(us_call, world), "unit": "us", "n_gpus": world, "steps": steps,
            "warmup": max(3, args.warmup), "ms_per_step": us_call / 1000.0, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "input_dtype": in_dtype, "data": "synthetic",
            "config": config_dict(name, w0, copies, bytes_call, world),
            "timed": {"blocks": len(blocks), "calls_per_block": steps, "device_ms_total": sum(blocks) * 1e3,
                      "us_per_call_mean": us_call, "us_per_call_min_block": us_call_best_block,
                      "note": "value is the mean over the blocks; every block is exactly `steps` calls between two CUDA events"},
            "rows_per_s": rows * world / (us_call * 1e-6),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "algorithmic_bytes": int(bytes_call), "measured_dram_bytes": traffic,
                         "measured_dram_bytes_source": traffic_src, "peak_source": which, "kernel": "whole call",
                         "dominant_kernel": "sonic_stream_kernel",
                         "per_kernel": per_kernel,
                         "note": "achieved = algorithmic bytes of the call (logits + mask words + lists, read once) / CUDA-event "
                                 "time of the whole call: the streaming kernel moves the bytes, the merges and the histogram "
                                 "passes of the same call run behind it, partly beside each other on a forked stream, "
                                 "so a call has no single kernel's duration.  per_kernel: serialised "
                                 "times and DRAM bytes under ncu from the committed profile (compare shares)."},
            "cpu_baseline": {"value": cpu_us, "unit": "us", "cores": 1, "kind": "oracle", "sample": cpu_desc},
            "cpu_baseline_all_cores": None if cpu_all is None else
                {"value": cpu_all[0], "unit": "us", "cores": cpu_all[1], "kind": "oracle", "sample": cpu_all[2]},
            "read_probe": dict(probe, frac_of_read_probe=achieved / probe["gbs"]),
            "e2e": {"value": job_value(e2e_us, world), "unit": "us", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": n_launch * steps * len(blocks),
            "gpu_launches_per_call": n_launch,
            "empty_graph_node_us": floor_us,
            "us_per_call_min": min_us,
            "warm_l2": {"us_per_call": warm_us, "input_fits_l2": bool(bytes_call < L2_BYTES),
                        "note": "one input copy replayed back to back"},
            "rows": {"per_call": rows, "cluster_kernel": fb["cluster"], "histogram_path": fb["dense"],
                     "near_margin": {"count": cpu_near, "of": cpu_rows, "unit": fb["cluster"]["unit"],
                                     "note": "decision margin below 1e-6 in the oracle, on the cpu_baseline sample"}},
            "clocks": clocks,
            "also": extra,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def w0_dtype(w):
    return w.sample.dtype if hasattr(w, "sample") else w.dtype


def quick_topk(k, binding, reps=10):
    """sonic_topk on the c5 'normal' regime (B=256, V=262144, fp32), two input copies (> 2x L2), one k."""
    import torch
    tw = wl.config5("normal")
    ws = binding.new_workspace(tw.B, tw.V)
    devs = [binding.DeviceTopK(tw, k, ws=ws), binding.DeviceTopK(tw, k, ws=ws)]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for d in devs:
            d.run()
    for _ in range(2):
        g.replay()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s.record()
    for _ in range(reps):
        g.replay()
    e.record()
    torch.cuda.synchronize()
    us = s.elapsed_time(e) * 1000.0 / (reps * 2)
    peak, _ = peaks()
    nbytes = tw.logits.nbytes
    del devs, g
    torch.cuda.empty_cache()
    return {"us_per_call": us, "algorithmic_bytes": int(nbytes), "achieved_gbs": nbytes / us / 1e3,
            "frac": nbytes / us / 1e3 / peak, "copies": 2, "k": k}


def topk_all(binding, min_time_s=0.05):
    """sonic_topk on all of configuration 5: three regimes x six k (B=256, V=262144, fp32; two input copies > 2x L2)."""
    import torch
    peak, _ = peaks()
    table = {}
    for regime in wl.TOPK_REGIMES:
        tw = wl.config5(regime)
        ws = binding.new_workspace(tw.B, tw.V)
        first = binding.DeviceTopK(tw, 1, ws=ws)
        second_logits = first.logits.clone()
        nbytes = tw.logits.nbytes
        for k in wl.TOPK_KS:
            devs = [binding.DeviceTopK(tw, k, ws=ws, logits=first.logits), binding.DeviceTopK(tw, k, ws=ws, logits=second_logits)]
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for d in devs:
                    d.run()
            for _ in range(3):
                g.replay()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps, total = 0, 0.0
            torch.cuda.synchronize()
            while total < min_time_s and reps < 400:
                s.record()
                for _ in range(5):
                    g.replay()
                e.record()
                torch.cuda.synchronize()
                total += s.elapsed_time(e) * 1e-3
                reps += 5
            us = total * 1e6 / (reps * 2)
            table[f"{regime}_k{k}"] = {"us_per_call": round(us, 2), "achieved_gbs": round(nbytes / us / 1e3, 1),
                                       "frac": round(nbytes / us / 1e3 / peak, 4)}
            del devs, g
        del first, second_logits, ws
        torch.cuda.empty_cache()
    return {"workload": "c5: sonic_topk, B=256, V=262144, fp32, regimes x k", "algorithmic_bytes": int(nbytes),
            "copies": 2, "table": table}


def quick_measure(name, binding, reps=30):
    """Short cold-input timing of another configuration (not the headline line)."""
    import torch
    if name == "c5":
        return topk_all(binding)
    if name.startswith("c5k"):
        return quick_topk(int(name[3:]), binding)
    w0 = make_workload(name)
    bytes_call = algorithmic_bytes(name, w0)
    copies = int(min(8, max(2, np.ceil(2.0 * L2_BYTES / bytes_call))))
    devs = build_device_copies(name, copies, binding)
    g = capture(devs, copies)
    for _ in range(3):
        g.replay()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    blocks = []
    torch.cuda.synchronize()
    while sum(blocks) < 0.1 and len(blocks) < 200:           # >= 100 ms of device time
        s.record()
        for _ in range(reps):
            g.replay()
        e.record()
        torch.cuda.synchronize()
        blocks.append(s.elapsed_time(e) * 1e-3)
    us = float(np.mean(blocks)) * 1e6 / (reps * copies)
    peak, which = peaks()
    gbs = bytes_call / (us * 1e-6) / 1e9
    traffic, per_kernel, src = profiled_traffic(name)
    del devs, g
    torch.cuda.empty_cache()
    return {"us_per_call": us, "us_per_call_min_block": min(blocks) * 1e6 / (reps * copies), "blocks": len(blocks),
            "algorithmic_bytes": int(bytes_call), "measured_dram_bytes": traffic, "achieved_gbs": gbs, "frac": gbs / peak,
            "copies": copies, "gpu_launches_per_call": launches_per_call(name, w0)}


def run_sweep():
    """Throughput sweep beyond the five configurations (one GPU): fused sample call on B rows of vocabulary V, all
    rows low-entropy ("spiked") or high-entropy ("flat"), fp32 and bf16.  Prints one JSON line with the table."""
    import torch
    from paper_2607_20475_b200 import harness as binding
    binding.lib()
    peak, which = peaks()
    table = []
    for dtype, dname in ((wl.DTYPE_F32, "f32"), (wl.DTYPE_BF16, "bf16")):
        for V in (1 << 15, 1 << 16, 1 << 17, 1 << 18):
            for B in (1, 8, 64, 256):
                for regime in ("spiked", "flat"):
                    nbytes = B * V * (2 if dtype == wl.DTYPE_BF16 else 4)
                    copies = int(min(16, max(2, np.ceil(2.0 * L2_BYTES / nbytes))))
                    ws = binding.new_workspace(B, V)
                    devs = [binding.DeviceSample(wl.sweep_case(B, V, dtype, regime, c), ws=ws) for c in range(copies)]
                    g = capture(devs, copies)
                    for _ in range(3):
                        g.replay()
                    reps = int(max(5, min(200, 2000 // copies)))
                    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    torch.cuda.synchronize()
                    s.record()
                    for _ in range(reps):
                        g.replay()
                    e.record()
                    torch.cuda.synchronize()
                    us = s.elapsed_time(e) * 1000.0 / (reps * copies)
                    fb = int(np.mean([int((d.results()["flags"] & 4).astype(bool).sum()) for d in devs]))
                    table.append({"dtype": dname, "V": V, "B": B, "rows": regime, "us_per_call": round(us, 2),
                                  "gbs": round(nbytes / us / 1e3, 1), "frac": round(nbytes / us / 1e3 / peak, 4),
                                  "cold": bool(copies * nbytes > 2 * L2_BYTES), "exact_rows": fb})
                    del devs, g, ws
                    torch.cuda.empty_cache()
    print(json.dumps({"sweep": "fused sample call, temperature 0.8, top-k 50, top-p 0.9", "peak_gbs": peak,
                      "peak_source": which, "table": table}))


TIMELINE_KERNELS = {0: "sonic_stream_kernel", 1: "sonic_merge_kernel", 6: "sonic_dense_stage2_kernel",
                    3: "sonic_dense_collect_kernel", 8: "sonic_dense_finish_kernel", 4: "sonic_dense_resid_kernel",
                    9: "sonic_dense_resid_finish_kernel", 2: "sonic_exact_kernel", 5: "sonic_verify_combine_kernel"}


def run_timeline(names, reps=5):
    """Per-kernel timeline of ONE call inside a replayed CUDA graph, from the trace variant of the library (every kernel
    leaves the earliest start and the latest end of its CTAs, globaltimer, in the workspace header).  One input copy
    (warm L2 where it fits); the figures show how the kernels of a call overlap, they are not a bench value.
    Prints one JSON line: {workload: {kernel: [start_us, end_us] (median of `reps` replays, from the first start)}}."""
    import torch
    from paper_2607_20475_b200 import build as _build
    _build.LIB = _build.build_trace()               # before the binding loads a library: this process uses the trace variant
    from paper_2607_20475_b200 import harness as binding
    binding.lib()
    out = {}
    for name in names:
        if name.startswith("c5k"):
            dev = binding.DeviceTopK(wl.config5("normal"), int(name[3:]))
        elif name == "c4":
            dev = binding.DeviceVerify(make_workload(name))
        else:
            dev = binding.DeviceSample(make_workload(name))
        hdr = dev.ws[:512].view(torch.int32)
        dev.run()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            dev.run()
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        runs = []
        for _ in range(reps):
            init = torch.zeros(24, dtype=torch.int32, device="cuda")
            init[0::2] = -1                                     # starts take a minimum, ends a maximum
            hdr[48:72] = init
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            h = hdr.cpu().numpy().astype(np.int64) & 0xFFFFFFFF
            t0 = min(int(h[48 + 2 * k]) for k in TIMELINE_KERNELS if h[48 + 2 * k] != 0xFFFFFFFF)
            runs.append({nm: [((int(h[48 + 2 * k]) - t0) & 0xFFFFFFFF) / 1000.0, ((int(h[49 + 2 * k]) - t0) & 0xFFFFFFFF) / 1000.0]
                         for k, nm in TIMELINE_KERNELS.items() if h[48 + 2 * k] != 0xFFFFFFFF and h[49 + 2 * k] != 0})
        kernels = {}
        for nm in runs[0]:
            if all(nm in r for r in runs):
                kernels[nm] = [round(float(np.median([r[nm][0] for r in runs])), 2), round(float(np.median([r[nm][1] for r in runs])), 2)]
        out[name] = {"kernels": kernels, "call_end_us": max(v[1] for v in kernels.values())}
        del dev, g
        torch.cuda.empty_cache()
    print(json.dumps({"timeline": out, "unit": "us from the first kernel's start", "build": "-DSONIC_TRACE variant, one input copy"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="sonic", choices=["sonic", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c1", "c2", "c3", "c4"])
    ap.add_argument("--sweep", action="store_true", help="time the V x B x entropy x dtype sweep instead (one GPU)")
    ap.add_argument("--min-time-ms", type=float, default=500.0,
                    help="repeat the timed block of --steps calls until this much device time is measured (0: one block)")
    ap.add_argument("--profile-run", action="store_true",
                    help="run the warm-up and one timed block only and print a short line (for use under ncu; never a bench value)")
    ap.add_argument("--timeline", default=None,
                    help="print the per-kernel timeline of one call of the given workloads (comma separated: c1..c4, c5k<k>) "
                         "from the trace variant of the library, instead of a bench line (one GPU)")
    ap.add_argument("--also", default="c1,c3,c4,c5", help="other configurations to time briefly (comma separated, '' for none; "
                    "c5 = sonic_topk over all regimes and k, c5k<k> = one k of the 'normal' regime)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if args.steps == 2000:
            args.steps = 5
        if args.warmup == 16:
            args.warmup = 1
        run_reference(args, rank, world)
        return
    if args.timeline:
        if rank == 0:
            run_timeline([n for n in args.timeline.split(",") if n])
        return
    if args.sweep:
        if rank == 0:
            run_sweep()
        return
    run_sonic(args, rank, world, local_rank)


if __name__ == "__main__":
    main()

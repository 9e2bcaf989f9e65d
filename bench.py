#!/usr/bin/env python
"""Benchmark of the quantised linear layer on B200: decode weight GB/s and prefill TFLOP/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Default workload: the Llama3.1-8B-shaped decode layer set at M = 1 (seven projections: q/k/v/o int8
per-channel, gate/up/down int4 group-32), 4 weight copies rotated so that every timed pass streams
its 141 MB of weights from HBM, launched as a CUDA graph with programmatic dependent launch.  One
step = one pass over the layer set.  The same run also times the prefill layer set (M = 2048) and
reports it under "prefill".  One JSON line is printed by rank 0.

With N > 1 (torchrun) every rank runs an independent replica on its own GPU (the path has no
exchange step); the value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import configs as C  # noqa: E402

L2_BYTES_FALLBACK = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# DRAM traffic per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum, one ncu
# capture each, summarised with its command under profiles/), averaged over the launches this file times.
NCU_TRAFFIC_BYTES = {
    ("llama31_8b_decode", 1): (66.095104e6 + 0.455936e6 + 33.085440e6) / 2,     # gate+up and down launches
    ("llama31_8b_prefill", 2048): (73.6e6 + 73.6e6 + 95.9e6) / 3,            # gate, up, down (reads + y write-back)
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period, self.samples, self.reasons = index, period_s, [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": int(statistics.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------ set-up
def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


class LayerSet:
    """`copies` independent weight copies of every layer of a workload, resident on one GPU."""

    def __init__(self, workload, M, copies, device, distinct_copies=True):
        import torch
        import paper_2505_00232_b200 as P
        self.P, self.torch, self.workload, self.M, self.copies = P, torch, workload, M, copies
        self.layers = workload.layers
        self.lin = [[None] * len(self.layers) for _ in range(copies)]
        self.x_host, self.x, self.y, self.y_host = [], [], [], []
        for li, layer in enumerate(self.layers):
            desc = P.Desc(layer.N, layer.K, layer.bits, layer.group)
            blob0 = None
            for cp in range(copies):
                if cp == 0 or distinct_copies:
                    q, s = C.layer_weights(workload.seed, layer, li, cp)
                    blob = torch.from_numpy(P.qlinear_pack(desc, q, s)).to(device)
                    blob0 = blob if cp == 0 else blob0
                else:
                    blob = blob0.clone()          # same bytes, separate HBM: still streamed from DRAM
                self.lin[cp][li] = P.QLinear(desc, blob)
            xh = torch.from_numpy(C.layer_activations(workload.seed, layer, M, li)).pin_memory()
            self.x_host.append(xh)
            self.x.append(xh.to(device))
            self.y.append(torch.empty((M, layer.N), dtype=torch.float16, device=device))
            self.y_host.append(torch.empty((M, layer.N), dtype=torch.float16).pin_memory())
        self.weight_bytes = sum(l.weight_bytes for l in self.layers)
        self.flops = sum(l.flops(M) for l in self.layers)

    def step(self, cp, only=None):
        for li in range(len(self.layers)):
            if only is None or li in only:
                self.lin[cp][li].forward_raw(self.x[li].data_ptr(), self.y[li].data_ptr(), self.M)

    _STAGE = {"q": 0, "k": 0, "v": 0, "o": 1, "gate": 2, "up": 2, "down": 3}

    def _groups(self):
        """Consecutive layers that read the same input (q, k, v; gate, up), as lists of layer indices."""
        groups, prev = [], None
        for li, l in enumerate(self.layers):
            st = self._STAGE.get(l.name, 100 + li)
            same = st == prev and groups and all(
                (self.layers[j].K, self.layers[j].bits, self.layers[j].group) == (l.K, l.bits, l.group) for j in groups[-1])
            if same:
                groups[-1].append(li)
            else:
                groups.append([li])
            prev = st
        return groups

    def step_grouped(self, cp, only=None):
        """One pass with the data flow of a transformer layer: q, k, v read the same input and go out as ONE
        grouped call, then o; gate and up likewise, then down.  Same seven layers, same bytes, four launches."""
        P = self.P
        for grp in self._groups():
            if only is not None and not all(li in only for li in grp):
                continue
            if len(grp) == 1:
                li = grp[0]
                self.lin[cp][li].forward_raw(self.x[li].data_ptr(), self.y[li].data_ptr(), self.M)
            else:
                P.qlinear_forward_group_raw([self.lin[cp][li] for li in grp], self.x[grp[0]].data_ptr(),
                                            [self.y[li].data_ptr() for li in grp], self.M)

    @property
    def launches_grouped(self):
        return len(self._groups())

    def step_e2e(self, cp, grouped=False):
        """Host buffers in, host buffers out: H2D of every input, the forwards, D2H of every y."""
        groups = self._groups() if grouped else [[li] for li in range(len(self.layers))]
        for grp in groups:
            li0 = grp[0]
            self.x[li0].copy_(self.x_host[li0], non_blocking=True)
            if len(grp) == 1:
                self.lin[cp][li0].forward_raw(self.x[li0].data_ptr(), self.y[li0].data_ptr(), self.M)
            else:
                self.P.qlinear_forward_group_raw([self.lin[cp][li] for li in grp], self.x[li0].data_ptr(),
                                                 [self.y[li].data_ptr() for li in grp], self.M)
            for li in grp:
                self.y_host[li].copy_(self.y[li], non_blocking=True)
        self.torch.cuda.current_stream().synchronize()

    def h2d_bytes(self, grouped=False):
        groups = self._groups() if grouped else [[li] for li in range(len(self.layers))]
        return sum(2 * self.M * self.layers[g[0]].K for g in groups)

    @property
    def d2h_bytes(self):
        return sum(2 * self.M * l.N for l in self.layers)


def max_over_ranks(local_value: float, device) -> float:
    """Slowest rank's value (all-reduce MAX); identity when no process group is up."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_value)
    t = torch.tensor([local_value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_step: float, steps: int, ms: float, world: int) -> float:
    """Replicas only: every rank processes the same units; the job's rate uses the slowest rank's time."""
    return world * units_per_step * steps / (ms / 1e3)


def time_events(torch, fn, iters):
    """Device time of fn() repeated `iters` times on the current stream (CUDA events), in ms."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for i in range(iters):
        fn(i)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b)


def capture_graph(torch, fn, n_steps):
    """Captures fn(0..n_steps-1) on a side stream into one CUDA graph."""
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for i in range(n_steps):
            fn(i)                       # warm, uncaptured
        torch.cuda.current_stream().synchronize()
        with torch.cuda.graph(g, stream=s):
            for i in range(n_steps):
                fn(i)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    return g


# ------------------------------------------------------------------------------------ CPU oracle legs
def oracle_sample_pass(workload, M, rows_cap, threads=0, reps=1):
    """`reps` passes of the CPU oracle (C triple loop, as it stands) over the first `rows_cap` output
    channels of every layer of the workload.  Returns (seconds, weight bytes, flops, cores), summed over
    the passes; the synthetic tensors are generated outside the timed region."""
    from oracle import qlinear_oracle as O
    total_t, wbytes, flops = 0.0, 0, 0
    for li, layer in enumerate(workload.layers):
        n = min(layer.N, rows_cap)
        sub = C.LayerSpec(layer.name, n, layer.K, layer.bits, layer.group, layer.lo, layer.hi)
        q, s = C.layer_weights(workload.seed, sub, li)
        x = C.layer_activations(workload.seed, sub, M, li)
        for _ in range(reps):
            t0 = time.perf_counter()
            O.linear_loops(x, q, s, layer.group, threads)
            total_t += time.perf_counter() - t0
            wbytes += sub.weight_bytes
            flops += sub.flops(M)
    return total_t, wbytes, flops, O.threads()


def calibrate_rows(workload, M, budget_s):
    """Rows per layer such that one oracle pass takes about budget_s seconds."""
    rows = 64
    t, _, _, _ = oracle_sample_pass(workload, M, rows)
    full_rows = max(l.N for l in workload.layers)
    while rows < full_rows and t < budget_s / 2.5:
        rows = min(full_rows, rows * 2)
        t, _, _, _ = oracle_sample_pass(workload, M, rows)
    return rows


def metric_of(stage):
    return ("decode_weight_gbs", "GB/s") if stage == "decode" else ("prefill_tflops", "TFLOP/s")


def units_of(stage, wbytes, flops):
    return wbytes / 1e9 if stage == "decode" else flops / 1e12


def run_reference(args, workload, M):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    metric, unit = metric_of(workload.stage)
    per_step_budget = max(0.05, min(2.0, 150.0 / max(1, args.steps + args.warmup)))
    rows = calibrate_rows(workload, M, per_step_budget)
    for _ in range(args.warmup):
        oracle_sample_pass(workload, M, rows)
    t_total, units = 0.0, 0.0
    cores = 1
    for _ in range(args.steps):
        t, wb, fl, cores = oracle_sample_pass(workload, M, rows)
        t_total += t
        units += units_of(workload.stage, wb, fl)
    value = units / t_total
    sample = f"first {rows} output channels of each of the {len(workload.layers)} layers, M={M}, per step"
    line = {
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload.name, "M": M, "note": "CPU oracle (fp64 triple loop) on host cores"},
        "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------ GPU legs
def bench_stage(torch, ls, stage, steps, warmup, use_graph, sampler_index, grouped=False):
    """Times `steps` passes over the layer set; returns dict with ms_per_step, clocks, launches."""
    copies = ls.copies
    per_step = ls.launches_grouped if grouped else len(ls.layers)
    step_fn = ls.step_grouped if grouped else ls.step
    if use_graph:
        graph = capture_graph(torch, lambda i: step_fn(i % copies), copies)
        n_replays = max(1, steps // copies)
        steps = n_replays * copies
        for _ in range(max(1, warmup // copies)):
            graph.replay()
        run = lambda: time_events(torch, lambda i: graph.replay(), n_replays)
    else:
        for i in range(warmup):
            step_fn(i % copies)
        run = lambda: time_events(torch, lambda i: step_fn(i % copies), steps)
    with ClockSampler(sampler_index) as cs:
        ms = run()
    return {"ms": ms, "steps": steps, "clocks": cs.summary(), "launches": steps * per_step}


def dominant_kernel_time(torch, ls, layer_ids, launches, use_graph, grouped=False):
    """Average device time per launch of the listed layers' kernel, rotated over the weight copies.
    Returns (ms per launch, launches per pass): with grouped calls a pass over the listed layers is
    fewer launches than layers."""
    copies = ls.copies
    step_fn = (lambda cp: ls.step_grouped(cp, only=layer_ids)) if grouped else (lambda cp: ls.step(cp, only=layer_ids))
    per_pass = len([g for g in ls._groups() if all(li in layer_ids for li in g)]) if grouped else len(layer_ids)
    if use_graph:
        graph = capture_graph(torch, lambda i: step_fn(i % copies), copies)
        per_replay = copies * per_pass
        n = max(1, launches // per_replay)
        for _ in range(3):
            graph.replay()
        ms = time_events(torch, lambda i: graph.replay(), n)
        return ms / (n * per_replay), per_pass
    n = max(1, launches // per_pass)
    for i in range(copies):
        step_fn(i % copies)
    ms = time_events(torch, lambda i: step_fn(i % copies), n)
    return ms / (n * per_pass), per_pass


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=40)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama31_8b_decode")
    ap.add_argument("--M", type=int, default=0, help="tokens (default: the workload's first M)")
    ap.add_argument("--copies", type=int, default=0, help="weight copies rotated (default: decode 3x L2 and >= 4, prefill 1.5x L2)")
    ap.add_argument("--no-graph", action="store_true", help="plain stream launches instead of CUDA-graph replay")
    ap.add_argument("--no-groups", action="store_true",
                    help="decode graph: one launch per layer (default: layers that read the same input, q/k/v and "
                         "gate/up, go out as one grouped call each, the data flow of a transformer layer)")
    ap.add_argument("--no-prefill", action="store_true", help="skip the prefill sub-measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--prefill-steps", type=int, default=20)
    ap.add_argument("--quick", action="store_true",
                    help="main timed region only (no e2e, per-kernel, prefill or CPU legs): the command to profile")
    args = ap.parse_args()

    workload = C.by_name(args.workload)
    M = args.M or workload.Ms[0]
    if args.impl == "reference":
        run_reference(args, workload, M)
        return

    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    peaks = load_peaks()
    stage = workload.stage
    metric, unit = metric_of(stage)
    l2 = torch.cuda.get_device_properties(local).L2_cache_size or L2_BYTES_FALLBACK

    layer_bytes = sum(l.weight_bytes for l in workload.layers)
    if stage == "decode":
        copies = args.copies or max(4, -(-3 * l2 // layer_bytes))
    else:
        copies = args.copies or max(1, -(-3 * l2 // (2 * layer_bytes)))
    ls = LayerSet(workload, M, copies, device, distinct_copies=True)
    use_graph = (stage == "decode") and not args.no_graph

    # ---- main timed region: K steps, barrier + synchronize on both sides, max over ranks
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    grouped = not args.no_groups
    res = bench_stage(torch, ls, stage, args.steps, args.warmup, use_graph, physical_gpu_index(local), grouped)
    if world > 1:
        dist.barrier()
        res["ms"] = max_over_ranks(res["ms"], device)
    steps = res["steps"]
    units_per_step = units_of(stage, ls.weight_bytes, ls.flops)
    value = whole_job_value(units_per_step, steps, res["ms"], world)

    if args.quick:
        if rank == 0:
            print(json.dumps({"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": steps,
                              "warmup": args.warmup, "ms_per_step": res["ms"] / steps, "quick": True,
                              "config": {"workload": workload.name, "M": M, "weight_copies": copies},
                              "gpu_launches": res["launches"]}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end to end through the public API with host buffers (H2D + forwards + D2H per step)
    e2e_steps = max(8, min(200, steps // 10))
    for i in range(3):
        ls.step_e2e(i % copies, grouped)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        ls.step_e2e(i % copies, grouped)
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, device)
    e2e_value = whole_job_value(units_per_step, e2e_steps, e2e_s * 1e3, world)

    # ---- roofline of the dominant kernel (live CUDA-event timing of that kernel's launches alone)
    if stage == "decode":
        dom_ids = [i for i, l in enumerate(workload.layers) if l.bits == 4] or list(range(len(workload.layers)))
        dom_name = "gemv_kernel<int4, grouped>" if workload.layers[dom_ids[0]].bits == 4 else "gemv_kernel<int8>"
        dom_ms, dom_launches = dominant_kernel_time(torch, ls, dom_ids, 1200, use_graph, grouped)
        dom_bytes = sum(workload.layers[i].weight_bytes for i in dom_ids) / dom_launches
        achieved = dom_bytes / 1e9 / (dom_ms / 1e3)
        roof = {"bound": "hbm", "kernel": dom_name, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get((workload.name, M)),
                "peak_source": peaks["source"],
                "bytes_per_launch": dom_bytes, "us_per_launch": dom_ms * 1e3,
                "frac_of_nominal_8tbs": achieved / 8000.0}
    else:
        dom_ids = [i for i, l in enumerate(workload.layers) if l.bits == 4] or list(range(len(workload.layers)))
        dom_ms, _ = dominant_kernel_time(torch, ls, dom_ids, 30 * len(dom_ids), False)
        dom_flops = sum(workload.layers[i].flops(M) for i in dom_ids) / len(dom_ids)
        achieved = dom_flops / 1e12 / (dom_ms / 1e3)
        peak = peaks["bf16_tflops"]
        roof = {"bound": "tensor", "kernel": "gemm_pair_kernel<int4, grouped>", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES.get((workload.name, M)),
                "peak_source": peaks["source"],
                "flops_per_launch": dom_flops, "us_per_launch": dom_ms * 1e3,
                "frac_of_nominal_2250": achieved / 2250.0}

    line = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": steps, "warmup": args.warmup,
        "ms_per_step": res["ms"] / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "dtype_detail": "int4/int8 weights unpacked to f16, f16 activations, f32 accumulate", "data": "synthetic",
        "config": {"workload": workload.name, "M": M, "layers": [f"{l.name}:{l.N}x{l.K}:int{l.bits}" for l in workload.layers],
                   "weight_copies": copies, "weight_bytes_per_step": ls.weight_bytes,
                   "l2": f"{copies} weight copies ({copies * layer_bytes / 1e6:.0f} MB) rotated per step; no flush",
                   "launch": ("cuda graph + programmatic dependent launch" if use_graph else "stream launches")
                             + (", q/k/v and gate/up as one grouped call each" if grouped else ""),
                   "parallelism": "replicas only" if world > 1 else "single gpu"},
        "clocks": res["clocks"], "gpu_launches": res["launches"],
        "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": ls.h2d_bytes(grouped), "d2h_bytes_per_step": ls.d2h_bytes,
                "steps": e2e_steps},
        "roofline": roof,
        "frac_of_measured_peak": value / world / (peaks["hbm_gbs"] if stage == "decode" else peaks["bf16_tflops"]),
    }

    if rank == 0 and world == 1:
        # ---- second stage of the hot path, measured in the same run
        if stage == "decode" and not args.no_prefill:
            line["prefill"] = prefill_sub(torch, device, peaks, args.prefill_steps, local)
        # ---- CPU oracle beside it (bounded sample)
        if not args.no_cpu_baseline:
            rows = calibrate_rows(workload, M, 8.0)
            t1, _, _, _ = oracle_sample_pass(workload, M, rows)
            reps = max(1, min(16, int(round(12.0 / max(t1, 1e-3)))))     # about 12 s of CPU work in all
            t, wb, fl, cores = oracle_sample_pass(workload, M, rows, reps=reps)
            line["cpu_baseline"] = {"value": units_of(stage, wb, fl) / t, "unit": unit, "cores": cores, "kind": "oracle",
                                    "sample": f"first {rows} output channels of each layer, {reps} passes, {t:.1f} s"}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def prefill_sub(torch, device, peaks, steps, local):
    import paper_2505_00232_b200 as P
    w = C.by_name("llama31_8b_prefill")
    M = w.Ms[0]
    try:
        ls = LayerSet(w, M, 2, device)
        res = bench_stage(torch, ls, "prefill", steps, 3, False, physical_gpu_index(local), grouped=True)
    except P.QLinearError as e:
        return {"unavailable": str(e)}
    tf = ls.flops * res["steps"] / 1e12 / (res["ms"] / 1e3)
    dom_ids = [i for i, l in enumerate(w.layers) if l.bits == 4]
    dom_ms, _ = dominant_kernel_time(torch, ls, dom_ids, 30, False)
    dom_flops = sum(w.layers[i].flops(M) for i in dom_ids) / len(dom_ids)
    ach = dom_flops / 1e12 / (dom_ms / 1e3)
    return {"metric": "prefill_tflops", "value": tf, "unit": "TFLOP/s", "steps": res["steps"],
            "ms_per_step": res["ms"] / res["steps"], "config": {"workload": w.name, "M": M},
            "clocks": res["clocks"], "gpu_launches": res["launches"],
            "roofline": {"bound": "tensor", "kernel": "gemm_pair_kernel<int4, grouped>", "achieved": ach,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
                         "traffic": NCU_TRAFFIC_BYTES.get((w.name, M)), "peak_source": peaks["source"],
                         "frac_of_nominal_2250": ach / 2250.0}}


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the quantised linear layer on B200: decode weight GB/s and prefill TFLOP/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Default workload: the Llama3.1-8B-shaped decode layer set at M = 1 (seven projections: q/k/v/o int8
per-channel, gate/up/down int4 group-32), 4 weight copies rotated so that every timed pass streams
its 141 MB of weights from HBM, launched as a CUDA graph with programmatic dependent launch.  One
step = one pass over the layer set.  The same run also times the prefill layer set (M = 2048) and
reports it under "prefill".  One JSON line is printed by rank 0.

Every timed leg runs the K steps it was asked for, `repeats` times back to back, inside ONE pair of CUDA
events, so that the region lasts at least half a second: long enough for the NVML sampler to see the
clocks the kernels really ran at.  "configs" carries one entry per benchmark workload (configs 1-5, the LM
head, and the paper's q8 and per-channel 8/4/4 schemes), each measured the same way.

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
    # gemm_pair_ta_kernel: gate + up grouped (83.06 + 82.21 MB, halved per layer) and down (146.67 + 12.78 MB)
    ("llama31_8b_prefill", 2048): (82.64e6 + 82.64e6 + 159.44e6) / 3,
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

    def __init__(self, workload, M, copies, device, distinct_copies=True, blobs=None, act="fp16"):
        """blobs: optional {layer index: packed device tensor} to bind copy 0 to weights that are already
        resident (the paper's point: one resident copy serves both stages)."""
        import torch
        import paper_2505_00232_b200 as P
        self.P, self.torch, self.workload, self.M, self.copies = P, torch, workload, M, copies
        self.act = act                        # "fp16": qlinear_forward; "int8": qlinear_forward_a8 (one call per layer)
        self.layers = workload.layers
        self.lin = [[None] * len(self.layers) for _ in range(copies)]
        self.blob0 = {}
        for li, layer in enumerate(self.layers):
            desc = P.Desc(layer.N, layer.K, layer.bits, layer.group)
            blob0 = None
            for cp in range(copies):
                if cp == 0 and blobs is not None:
                    blob = blobs[li]
                elif cp == 0 or distinct_copies:
                    q, s = C.layer_weights(workload.seed, layer, li, cp)
                    blob = torch.from_numpy(P.qlinear_pack(desc, q, s)).to(device)
                else:
                    blob = blob0.clone()          # same bytes, separate HBM: still streamed from DRAM
                blob0 = blob if cp == 0 else blob0
                self.lin[cp][li] = P.QLinear(desc, blob)
            self.blob0[li] = blob0
        # Inputs and outputs of all layers live in ONE host buffer and ONE device buffer each, so that the
        # end-to-end step moves them with a single copy per direction; per-layer tensors are views.
        x_np = [C.layer_activations(workload.seed, layer, M, li) for li, layer in enumerate(self.layers)]
        nx, ny = sum(a.size for a in x_np), sum(M * l.N for l in self.layers)
        self.x_host_all = torch.empty(nx, dtype=torch.float16).pin_memory()
        self.y_host_all = torch.empty(ny, dtype=torch.float16).pin_memory()
        self.x_all = torch.empty(nx, dtype=torch.float16, device=device)
        self.y_all = torch.empty(ny, dtype=torch.float16, device=device)
        self.x_host, self.x, self.y, self.y_host = [], [], [], []
        ox = oy = 0
        for a, layer in zip(x_np, self.layers):
            self.x_host.append(self.x_host_all[ox:ox + a.size].view(M, layer.K))
            self.x_host[-1].copy_(torch.from_numpy(a))
            self.x.append(self.x_all[ox:ox + a.size].view(M, layer.K))
            self.y.append(self.y_all[oy:oy + M * layer.N].view(M, layer.N))
            self.y_host.append(self.y_host_all[oy:oy + M * layer.N].view(M, layer.N))
            ox += a.size
            oy += M * layer.N
        self.x_all.copy_(self.x_host_all)
        self.weight_bytes = sum(l.weight_bytes for l in self.layers)
        self.flops = sum(l.flops(M) for l in self.layers)

    def step(self, cp, only=None):
        for li in range(len(self.layers)):
            if only is None or li in only:
                fwd = self.lin[cp][li].forward_a8_raw if self.act == "int8" else self.lin[cp][li].forward_raw
                fwd(self.x[li].data_ptr(), self.y[li].data_ptr(), self.M)

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
        """Host buffers in, host buffers out: one H2D copy of all inputs from pinned memory, the forwards
        through the C-ABI, one D2H copy of all outputs, synchronise."""
        self.x_all.copy_(self.x_host_all, non_blocking=True)
        (self.step_grouped if grouped else self.step)(cp)
        self.y_host_all.copy_(self.y_all, non_blocking=True)
        self.torch.cuda.current_stream().synchronize()

    def e2e_graphs(self, grouped=False):
        """The same end-to-end step captured once per weight copy as a CUDA graph (copy in, forwards, copy out):
        what a serving loop that replays a fixed step does.  Returns one replay-and-synchronise callable per copy."""
        torch = self.torch
        graphs = []
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for cp in range(self.copies):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    self.x_all.copy_(self.x_host_all, non_blocking=True)
                    (self.step_grouped if grouped else self.step)(cp)
                    self.y_host_all.copy_(self.y_all, non_blocking=True)
                graphs.append(g)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

        def run(cp):
            graphs[cp].replay()
            torch.cuda.current_stream().synchronize()
        return run

    @property
    def h2d_bytes(self):
        return 2 * self.x_host_all.numel()

    @property
    def d2h_bytes(self):
        return 2 * self.y_host_all.numel()


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
MIN_REGION_S = 0.5      # every timed region lasts at least this long (enough NVML samples for a clock record)


def timed_region(torch, block, steps_per_block, sampler_index, min_s=MIN_REGION_S):
    """Times `repeats` runs of block() (each = steps_per_block steps) between one pair of CUDA events, with
    repeats chosen so that the region lasts at least min_s.  Returns ms, repeats and the clock record."""
    probe = time_events(torch, lambda i: block(), 1)                      # also a last warm-up
    repeats = max(1, int(np.ceil(min_s * 1e3 / max(probe, 1e-3))))
    with ClockSampler(sampler_index) as cs:
        ms = time_events(torch, lambda i: block(), repeats)
    clocks = cs.summary()
    if clocks["sm_mhz"]:
        clocks["ms_per_step_x_mhz"] = ms / (repeats * steps_per_block) * clocks["sm_mhz"]
    return ms, repeats, clocks


def bench_stage(torch, ls, stage, steps, warmup, use_graph, sampler_index, grouped=False, min_s=MIN_REGION_S):
    """Times `steps` passes over the layer set, repeated back to back; returns ms per step and the record."""
    copies = ls.copies
    per_step = ls.launches_grouped if grouped else len(ls.layers)
    step_fn = ls.step_grouped if grouped else ls.step
    if use_graph:
        graph = capture_graph(torch, lambda i: step_fn(i % copies), copies)
        n_replays = max(1, steps // copies)
        steps = n_replays * copies
        for _ in range(max(1, warmup // copies)):
            graph.replay()

        def block():
            for _ in range(n_replays):
                graph.replay()
    else:
        for i in range(max(warmup, copies)):
            step_fn(i % copies)

        def block():
            for i in range(steps):
                step_fn(i % copies)
    ms, repeats, clocks = timed_region(torch, block, steps, sampler_index, min_s)
    return {"ms": ms, "steps": steps, "repeats": repeats, "ms_per_step": ms / (repeats * steps), "clocks": clocks,
            "launches": repeats * steps * per_step}


def kernel_time(torch, ls, layer_ids, use_graph, grouped, sampler_index, min_s=0.25):
    """Device time per launch of the launch(es) that serve the listed layers alone, rotated over the weight
    copies (CUDA events on the launching stream).  Returns (ms per launch, launches per pass)."""
    copies = ls.copies
    step_fn = (lambda cp: ls.step_grouped(cp, only=layer_ids)) if grouped else (lambda cp: ls.step(cp, only=layer_ids))
    per_pass = len([g for g in ls._groups() if all(li in layer_ids for li in g)]) if grouped else len(layer_ids)
    if use_graph:
        graph = capture_graph(torch, lambda i: step_fn(i % copies), copies)
        for _ in range(3):
            graph.replay()
        block = graph.replay
    else:
        def block():
            for i in range(copies):
                step_fn(i)
        block()
    ms, repeats, _ = timed_region(torch, block, copies, sampler_index, min_s)
    return ms / (repeats * copies * per_pass), per_pass


def decode_roofline(torch, ls, workload, M, peaks, use_graph, grouped, sampler_index):
    """The dominant decode kernel on its own: each launch shape of the int4 layers (as the step issues them: gate
    and up in one grouped launch, down alone) timed separately; the headline figure is their bytes over their time."""
    ids4 = [i for i, l in enumerate(workload.layers) if l.bits == 4]
    dom_ids = ids4 or list(range(len(workload.layers)))
    groups = [g for g in (ls._groups() if grouped else [[i] for i in range(len(workload.layers))]) if all(i in dom_ids for i in g)]
    per_launch, tot_bytes, tot_ms = [], 0.0, 0.0
    for g in groups:
        ms, _ = kernel_time(torch, ls, g, use_graph, grouped, sampler_index)
        nbytes = sum(workload.layers[i].weight_bytes for i in g)
        per_launch.append({"layers": "+".join(workload.layers[i].name for i in g), "bytes": nbytes, "us": ms * 1e3,
                           "gbs": nbytes / 1e9 / (ms / 1e3), "frac": nbytes / 1e9 / (ms / 1e3) / peaks["hbm_gbs"]})
        tot_bytes += nbytes
        tot_ms += ms
    achieved = tot_bytes / 1e9 / (tot_ms / 1e3)
    name = "gemv_kernel<int4, grouped>" if ids4 else "gemv_kernel<int8>"
    return {"bound": "hbm", "kernel": name + ": the launches listed under 'launches', each timed alone; achieved = their bytes / their time",
            "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
            "traffic": NCU_TRAFFIC_BYTES.get((workload.name, M)), "peak_source": peaks["source"],
            "bytes_per_launch": tot_bytes / len(groups), "us_per_launch": tot_ms * 1e3 / len(groups),
            "launches": per_launch, "frac_of_nominal_8tbs": achieved / 8000.0}


def prefill_roofline(torch, ls, workload, M, peaks, sampler_index, kernel_name="gemm_pair_ta_kernel<int4, grouped>"):
    ids4 = [i for i, l in enumerate(workload.layers) if l.bits == 4] or list(range(len(workload.layers)))
    ms, _ = kernel_time(torch, ls, ids4, False, False, sampler_index)
    flops = sum(workload.layers[i].flops(M) for i in ids4) / len(ids4)
    ach = flops / 1e12 / (ms / 1e3)
    return {"bound": "tensor", "kernel": kernel_name + ": the int4 layers as single launches, average", "achieved": ach,
            "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
            "traffic": NCU_TRAFFIC_BYTES.get((workload.name, M)), "peak_source": peaks["source"],
            "flops_per_launch": flops, "us_per_launch": ms * 1e3, "frac_of_nominal_2250": ach / 2250.0,
            # the launches are timed back to back for at least a quarter of a second, i.e. under the power limit: next to
            # the burst peak (the denominator of `frac`) the peak of a seconds-long cuBLAS loop on the same part
            "peak_sustained": peaks.get("bf16_tflops_sustained"),
            "frac_of_sustained_peak": ach / peaks["bf16_tflops_sustained"] if peaks.get("bf16_tflops_sustained") else None}


def config_entry(torch, device, peaks, sampler_index, name, M, copies=0, blobs=None, ls=None, steps=0):
    """One workload of the benchmark measured like the headline: value, time per step, fraction of the measured peak."""
    w = C.by_name(name)
    stage = w.stage
    l2 = torch.cuda.get_device_properties(device).L2_cache_size or L2_BYTES_FALLBACK
    layer_bytes = sum(l.weight_bytes for l in w.layers)
    if not copies:
        copies = max(4, -(-3 * l2 // layer_bytes)) if stage == "decode" else max(1, -(-3 * l2 // (2 * layer_bytes)))
    own = ls is None
    if own:
        ls = LayerSet(w, M, copies, device, distinct_copies=False, blobs=blobs)
    res = bench_stage(torch, ls, stage, steps or (4 * ls.copies if stage == "decode" else 2), max(3, ls.copies),
                      stage == "decode", sampler_index, grouped=True)
    metric, unit = metric_of(stage)
    value = units_of(stage, ls.weight_bytes, ls.flops) / (res["ms_per_step"] / 1e3)
    peak = peaks["hbm_gbs"] if stage == "decode" else peaks["bf16_tflops"]
    entry = {"workload": name, "M": M, "metric": metric, "value": value, "unit": unit, "us_per_step": res["ms_per_step"] * 1e3,
             "frac_of_measured_peak": value / peak, "weight_bytes_per_step": ls.weight_bytes, "weight_copies": ls.copies,
             "launches_per_step": ls.launches_grouped, "steps": res["steps"], "repeats": res["repeats"],
             "timed_region_ms": res["ms"], "clocks": res["clocks"], "gpu_launches": res["launches"]}
    if own:
        del ls
        torch.cuda.empty_cache()
    return entry


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
    ap.add_argument("--act", default="fp16", choices=["fp16", "int8"],
                    help="int8: the int8-activation entry point (paper Section 3.7), one call per layer")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-workload record (configs 1-5, LM head, q8, 8/4/4)")
    ap.add_argument("--prefill-steps", type=int, default=20)
    ap.add_argument("--records", default="", help="comma-separated names of the auxiliary records to run (default: all), e.g. kv_attention")
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
    ls = LayerSet(workload, M, copies, device, distinct_copies=True, act=args.act)
    if args.act == "int8":
        args.no_groups = True
    use_graph = (stage == "decode") and not args.no_graph

    # ---- main timed region: K steps (repeated back to back, see timed_region), barrier + synchronize on both
    # sides, max over ranks
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    grouped = not args.no_groups
    sidx = physical_gpu_index(local)
    res = bench_stage(torch, ls, stage, args.steps, args.warmup, use_graph, sidx, grouped,
                      min_s=0.0 if args.quick else MIN_REGION_S)
    if world > 1:
        dist.barrier()
        res["ms"] = max_over_ranks(res["ms"], device)
        res["ms_per_step"] = res["ms"] / (res["repeats"] * res["steps"])
    steps = res["steps"]
    units_per_step = units_of(stage, ls.weight_bytes, ls.flops)
    value = whole_job_value(units_per_step, 1, res["ms_per_step"], world)

    if args.quick:
        if rank == 0:
            print(json.dumps({"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": steps,
                              "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "repeats": res["repeats"], "quick": True,
                              "config": {"workload": workload.name, "M": M, "weight_copies": copies},
                              "gpu_launches": res["launches"]}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end to end through the public API with host buffers: per step ONE H2D copy of all inputs from pinned
    # memory, the forwards, ONE D2H copy of all outputs, synchronise
    def time_e2e(step):
        for i in range(3):
            step(i % copies)
        torch.cuda.synchronize()
        n, dt = 0, 0.0
        t0 = time.perf_counter()
        while dt < MIN_REGION_S / 2 or n < 8:
            step(n % copies)
            n += 1
            dt = time.perf_counter() - t0
        return n, max_over_ranks(dt, device)
    # plain calls (every step issues its copies and launches), and the same step replayed as one CUDA graph
    e2e_steps_plain, e2e_s_plain = time_e2e(lambda cp: ls.step_e2e(cp, grouped))
    e2e_plain = whole_job_value(units_per_step, e2e_steps_plain, e2e_s_plain * 1e3, world)
    e2e_steps, e2e_s = time_e2e(ls.e2e_graphs(grouped)) if stage == "decode" else (e2e_steps_plain, e2e_s_plain)
    e2e_value = whole_job_value(units_per_step, e2e_steps, e2e_s * 1e3, world)

    # ---- roofline of the dominant kernel (live CUDA-event timing of that kernel's launches alone)
    if stage == "decode":
        roof = decode_roofline(torch, ls, workload, M, peaks, use_graph, grouped, sidx)
    else:
        roof = prefill_roofline(torch, ls, workload, M, peaks, sidx)

    line = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": steps, "warmup": args.warmup,
        "ms_per_step": res["ms_per_step"], "repeats": res["repeats"], "timed_region_ms": res["ms"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "dtype_detail": "int4/int8 weights unpacked to f16, f16 activations, f32 accumulate", "data": "synthetic",
        "config": {"workload": workload.name, "M": M, "layers": [f"{l.name}:{l.N}x{l.K}:int{l.bits}" for l in workload.layers],
                   "weight_copies": copies, "weight_bytes_per_step": ls.weight_bytes,
                   "l2": f"{copies} weight copies ({copies * layer_bytes / 1e6:.0f} MB) rotated per step; no flush",
                   "launch": ("cuda graph + programmatic dependent launch" if use_graph else "stream launches")
                             + (", q/k/v and gate/up as one grouped call each" if grouped else ""),
                   "timing": f"the {steps} steps are run {res['repeats']} times back to back inside one CUDA-event pair "
                             f"(at least {MIN_REGION_S} s, so that the clock record has samples)",
                   "parallelism": "replicas only" if world > 1 else "single gpu"},
        "clocks": res["clocks"], "gpu_launches": res["launches"],
        "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": ls.h2d_bytes, "d2h_bytes_per_step": ls.d2h_bytes,
                "steps": e2e_steps, "us_per_step": e2e_s / e2e_steps * 1e6,
                "copies": "one pinned host buffer each way: 1 H2D + 1 D2H per step, host synchronises after every step",
                "launch": "the step (copy in, forwards, copy out) replayed as one CUDA graph" if stage == "decode" else "stream launches",
                "plain_calls": {"value": e2e_plain, "us_per_step": e2e_s_plain / e2e_steps_plain * 1e6, "steps": e2e_steps_plain}},
        "roofline": roof,
        "frac_of_measured_peak": value / world / (peaks["hbm_gbs"] if stage == "decode" else peaks["bf16_tflops"]),
    }

    if rank == 0 and world == 1:
        wanted = {r for r in args.records.split(",") if r}

        def extra(name, fn, append=False):
            """An auxiliary record must not cost the line: on failure its place holds the error."""
            if wanted and name not in wanted:
                return
            try:
                rec = fn()
                line[name] = line[name] + rec if append else rec
            except Exception as e:                                        # noqa: BLE001 (reported in the line)
                torch.cuda.synchronize()
                ls.lin[0][0].device_status()                              # reads and clears an expired-wait report
                err = {"error": f"{type(e).__name__}: {e}"}
                line[name] = line[name] + [err] if append else err
        if stage == "decode" and workload.name == "llama31_8b_decode":
            # ---- every decode workload of the benchmark first, measured like the headline (the tensor-core legs
            # that follow heat the part and would lower the clocks of whatever runs after them)
            if not args.no_configs:
                extra("configs", lambda: decode_configs(torch, device, peaks, sidx, ls, line))
                extra("decoder_block", lambda: block_record(torch, device, peaks, sidx, ls))
                extra("launch_floor", lambda: floor_record(torch, sidx, ls))
            # ---- second stage of the hot path on the SAME resident weights (copy 0), measured in the same run
            if not args.no_prefill:
                extra("prefill", lambda: prefill_sub(torch, device, peaks, args.prefill_steps, sidx, ls.blob0))
            if not args.no_configs:
                if not isinstance(line.get("configs"), list):
                    line["configs"] = [line["configs"]] if "configs" in line else []
                extra("configs", lambda: prefill_configs(torch, device, peaks, sidx, line), append=True)
                extra("fused_gating", lambda: gated_record(torch, device, peaks, sidx, ls))
                extra("residual_rmsnorm", lambda: norm_record(torch, device, peaks, sidx))
                extra("rope_qkv", lambda: rope_record(torch, device, peaks, sidx))
                extra("kv_attention", lambda: kv_record(torch, device, peaks, sidx))
                extra("int8_activations", lambda: a8_record(torch, device, peaks, sidx))
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


def prefill_sub(torch, device, peaks, steps, sidx, blobs):
    import paper_2505_00232_b200 as P
    w = C.by_name("llama31_8b_prefill")
    M = w.Ms[0]
    try:
        ls = LayerSet(w, M, 2, device, distinct_copies=False, blobs=blobs)
        res = bench_stage(torch, ls, "prefill", steps, 3, False, sidx, grouped=True)
        # the same layer set back to back for at least two seconds: the sustained figure, under the power cap
        sus = bench_stage(torch, ls, "prefill", steps, 0, False, sidx, grouped=True, min_s=2.0)
    except P.QLinearError as e:
        return {"unavailable": str(e)}
    tf = ls.flops / 1e12 / (res["ms_per_step"] / 1e3)
    tf_sus = ls.flops / 1e12 / (sus["ms_per_step"] / 1e3)
    out = {"metric": "prefill_tflops", "value": tf, "unit": "TFLOP/s", "steps": res["steps"], "repeats": res["repeats"],
           "timed_region_ms": res["ms"], "ms_per_step": res["ms_per_step"], "config": {"workload": w.name, "M": M,
           "weights": "copy 0 is the decode leg's resident blob; 1 more copy rotated"},
           "clocks": res["clocks"], "gpu_launches": res["launches"],
           "frac_of_measured_peak": tf / peaks["bf16_tflops"],
           "sustained": {"value": tf_sus, "unit": "TFLOP/s", "seconds": sus["ms"] / 1e3, "peak": peaks.get("bf16_tflops_sustained"),
                         "frac": tf_sus / peaks["bf16_tflops_sustained"] if peaks.get("bf16_tflops_sustained") else None,
                         "clocks": sus["clocks"]},
           "roofline": prefill_roofline(torch, ls, w, M, peaks, sidx)}
    del ls
    torch.cuda.empty_cache()
    return out


def norm_record(torch, device, peaks, sidx):
    """Residual connection + RMS normalisation (paper Section 3.6), the operator that produces the linear layer's
    input, at the Llama width: prefill (M = 2048; 8 rotated buffer sets = 537 MB, past L2) and one decode token."""
    import paper_2505_00232_b200 as P
    K, out = 4096, {"K": 4096, "bytes_per_token": 4 * 4096 * 2}
    rng = np.random.default_rng(3)
    g = torch.from_numpy((rng.standard_normal(K) / 4).astype(np.float16)).to(device)
    for stage, M, sets in (("prefill", 2048, 8), ("decode", 1, 64)):
        xs = [torch.from_numpy(rng.standard_normal((M, K)).astype(np.float16)).to(device) for _ in range(sets)]
        rs = [torch.from_numpy(rng.standard_normal((M, K)).astype(np.float16)).to(device) for _ in range(sets)]
        hs = [torch.empty_like(xs[0]) for _ in range(sets)]
        ys = [torch.empty_like(xs[0]) for _ in range(sets)]
        graph = capture_graph(torch, lambda i: P.qlinear_residual_rmsnorm(xs[i], rs[i], g, 1e-5, 0.0, h_out=hs[i], y_out=ys[i]), sets)
        for _ in range(3):
            graph.replay()
        ms, repeats, clocks = timed_region(torch, graph.replay, sets, sidx, 0.25)
        us = ms * 1e3 / (repeats * sets)
        gbs = 4 * M * K * 2 / 1e3 / us
        out[stage] = {"M": M, "us": us, "gbs": gbs, "frac_of_measured_peak": gbs / peaks["hbm_gbs"], "sm_mhz": clocks["sm_mhz"]}
    return out


def rope_record(torch, device, peaks, sidx):
    """Rotary embedding + Q/K/V layout transformation (paper Section 3.6) at the Llama3.1-8B head shape (32 / 8 heads of
    128): prefill (S = 2048; 10 rotated buffer sets = 503 MB, past L2) and one decode token."""
    import paper_2505_00232_b200 as P
    h_q, h_kv, d_h, n_pos = 32, 8, 128, 4096
    rng = np.random.default_rng(4)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * (500000.0 ** (-np.arange(d_h // 2) * 2.0 / d_h))[None, :]
    cos, sin = (torch.from_numpy(f(ang).astype(np.float32)).to(device) for f in (np.cos, np.sin))
    out = {"h_q": h_q, "h_kv": h_kv, "d_h": d_h, "bytes_per_token": 2 * 2 * (h_q + 2 * h_kv) * d_h}
    for stage, S, sets in (("prefill", 2048, 10), ("decode", 1, 64)):
        mk = lambda heads: [torch.from_numpy(rng.standard_normal((S, heads * d_h)).astype(np.float16)).to(device) for _ in range(sets)]
        qs, ks, vs = mk(h_q), mk(h_kv), mk(h_kv)
        pos = torch.arange(S, dtype=torch.int32, device=device)
        graph = capture_graph(torch, lambda i: P.qlinear_rope_qkv(qs[i], ks[i], vs[i], pos, cos, sin, 1, S, h_q, h_kv, d_h), sets)
        for _ in range(3):
            graph.replay()
        ms, repeats, clocks = timed_region(torch, graph.replay, sets, sidx, 0.25)
        us = ms * 1e3 / (repeats * sets)
        gbs = out["bytes_per_token"] * S / 1e3 / us
        out[stage] = {"S": S, "us": us, "gbs": gbs, "frac_of_measured_peak": gbs / peaks["hbm_gbs"], "sm_mhz": clocks["sm_mhz"]}
    return out


def floor_record(torch, sidx, ls_main):
    """What a dependent launch costs on this machine: a kernel that does nothing, launched like every kernel of the
    library, 64 of them chained in a CUDA graph -- one warp, and a grid the size of a decode launch (4 CTAs of 256
    threads per SM).  The floor under every small layer (config 1 is a single 5.3 MB launch)."""
    lin = ls_main.lin[0][0]
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    out = {}
    for name, grid, block in (("one_warp", 1, 32), ("decode_sized_grid", 4 * sms, 256)):
        graph = capture_graph(torch, lambda i: lin.debug_null_launch(grid, block), 64)
        for _ in range(3):
            graph.replay()
        ms, repeats, clocks = timed_region(torch, graph.replay, 64, sidx, 0.2)
        out[name + "_us"] = ms * 1e3 / (repeats * 64)
    return out


def kv_record(torch, device, peaks, sidx):
    """The attention products over the KV cache held as weights (paper Section 3.8) for one decode token of a
    Llama3.1-8B attention layer (8 KV heads of 128, 4 query rows each): append of the token's keys and values, scores
    and output for all heads, one launch each (the softmax between them is the caller's and not in the region).  At
    the paper's protocol length (1024 + 256 positions) and at 32768 positions, where the caches of 4 layers (268 MB)
    are rotated so that they come from HBM."""
    import paper_2505_00232_b200 as P
    h_kv, g, d_h = 8, 4, 128
    rng = np.random.default_rng(5)
    out = {"h_kv": h_kv, "q_rows_per_head": g, "d_h": d_h, "launches_per_step": 3}
    for T, layers in ((1280, 4), (32768, 4)):
        caches = [P.KVHeads(h_kv, T, d_h, device) for _ in range(layers)]
        kv = torch.from_numpy(rng.standard_normal((h_kv, T, d_h)).astype(np.float16)).to(device)
        for c in caches:
            c.append(kv[:, :T - 1].contiguous(), kv[:, :T - 1].contiguous())
        q = torch.from_numpy(rng.standard_normal((h_kv, g, d_h)).astype(np.float16)).to(device)
        prob = torch.full((h_kv, g, T), 1.0 / T, dtype=torch.float16, device=device)
        sc = torch.empty((h_kv, g, T), dtype=torch.float16, device=device)
        o = torch.empty((h_kv, g, d_h), dtype=torch.float16, device=device)
        new = kv[:, T - 1:].contiguous()

        def step(i, what=("append", "scores", "output")):
            c = caches[i % layers]
            if "append" in what:
                c.length = T - 1                                          # the same last position every time
                c.append_raw(new.data_ptr(), new.data_ptr(), d_h, d_h, 1)
            if "scores" in what:
                c.scores_raw(q.data_ptr(), sc.data_ptr(), g)
            if "output" in what:
                c.output_raw(prob.data_ptr(), o.data_ptr(), g)
        rec = {"positions": T, "cache_bytes_read": 2 * h_kv * T * d_h}
        for name, what in (("step", ("append", "scores", "output")), ("append", ("append",)), ("scores", ("scores",)), ("output", ("output",))):
            graph = capture_graph(torch, lambda i: step(i, what), layers)
            for _ in range(3):
                graph.replay()
            ms, repeats, clocks = timed_region(torch, graph.replay, layers, sidx, 0.2)
            rec[name + "_us"] = ms * 1e3 / (repeats * layers)
        rec["gbs"] = rec["cache_bytes_read"] / 1e3 / rec["step_us"]
        rec["frac_of_measured_peak"] = rec["gbs"] / peaks["hbm_gbs"]
        out[f"T{T}"] = rec
        del caches
        torch.cuda.empty_cache()
    return out


def block_record(torch, device, peaks, sidx, ls_main):
    """The linear hot path of ONE Llama3.1-8B transformer block at the headline's M with the operators of Section 3.6
    around it, chained on one stream the way a decoder issues them (the attention core itself is not part of this
    library and is left out: the o projection reads a buffer of the right shape):
      residual + rmsnorm -> q/k/v (one grouped launch) -> rotary + QKV layout -> o -> residual + rmsnorm
      -> gate/up with the gating fused -> down.
    8 kernels, replayed as one CUDA graph over the rotated weight copies; value = weight bytes over time."""
    import paper_2505_00232_b200 as P
    w, M, copies = ls_main.workload, ls_main.M, ls_main.copies
    idx = {l.name: i for i, l in enumerate(w.layers)}
    D, h_q, h_kv, d_h = w.layers[idx["q"]].K, 32, 8, 128
    rng = np.random.default_rng(11)
    f16 = lambda *shape: torch.from_numpy(rng.standard_normal(shape).astype(np.float16)).to(device)
    x, res, gam = f16(M, D), f16(M, D), f16(D)
    a, attn = torch.empty_like(x), f16(M, h_q * d_h)
    yq, yk, yv = (torch.empty((M, n), dtype=torch.float16, device=device) for n in (h_q * d_h, h_kv * d_h, h_kv * d_h))
    x2 = torch.empty_like(x)
    ff = torch.empty((M, w.layers[idx["gate"]].N), dtype=torch.float16, device=device)
    pos = torch.arange(M, dtype=torch.int32, device=device)
    ang = np.arange(64, dtype=np.float64)[:, None] * (500000.0 ** (-np.arange(d_h // 2) * 2.0 / d_h))[None, :]
    cos, sin = (torch.from_numpy(f(ang).astype(np.float32)).to(device) for f in (np.cos, np.sin))

    def block(cp):
        L = ls_main.lin[cp]
        P.qlinear_residual_rmsnorm(x, res, gam, 1e-5, 0.0, h_out=res, y_out=a)
        P.qlinear_forward_group_raw([L[idx["q"]], L[idx["k"]], L[idx["v"]]], a.data_ptr(), [yq.data_ptr(), yk.data_ptr(), yv.data_ptr()], M)
        P.qlinear_rope_qkv(yq, yk, yv, pos, cos, sin, 1, M, h_q, h_kv, d_h)
        L[idx["o"]].forward_raw(attn.data_ptr(), x2.data_ptr(), M)
        P.qlinear_residual_rmsnorm(x2, res, gam, 1e-5, 0.0, h_out=res, y_out=a)
        P.qlinear_forward_gated_raw(L[idx["gate"]], L[idx["up"]], a.data_ptr(), ff.data_ptr(), M, "silu")
        L[idx["down"]].forward_raw(ff.data_ptr(), x.data_ptr(), M)

    graph = capture_graph(torch, lambda i: block(i % copies), copies)
    for _ in range(3):
        graph.replay()
    ms, repeats, clocks = timed_region(torch, graph.replay, copies, sidx, 0.25)
    us = ms * 1e3 / (repeats * copies)
    gbs = ls_main.weight_bytes / 1e3 / us
    return {"M": M, "kernels": 8, "us": us, "weight_gbs": gbs, "frac_of_measured_peak": gbs / peaks["hbm_gbs"], "sm_mhz": clocks["sm_mhz"],
            "note": "residual+rmsnorm, q/k/v grouped, rope+layout, o, residual+rmsnorm, gated gate/up, down; attention core not included"}


def gated_record(torch, device, peaks, sidx, ls_main):
    """The fused gating epilogue of the feed-forward block (paper Section 3.6) on the Llama gate / up layers,
    next to the same two layers as one grouped call that writes both projections: decode at the headline's M,
    prefill at M = 2048.  Same weights (the decode leg's resident copies), same x."""
    import paper_2505_00232_b200 as P
    w = ls_main.workload
    ig = [i for i, l in enumerate(w.layers) if l.name == "gate"][0]
    iu = [i for i, l in enumerate(w.layers) if l.name == "up"][0]
    layer, act = w.layers[ig], "silu"
    wbytes = layer.weight_bytes + w.layers[iu].weight_bytes
    out = {"layers": f"gate, up {layer.N}x{layer.K} int{layer.bits} group {layer.group}", "act": act}
    for stage, M in (("decode", ls_main.M), ("prefill", 2048)):
        x = torch.from_numpy(C.layer_activations(w.seed, layer, M, ig)).to(device)
        y = torch.empty((M, layer.N), dtype=torch.float16, device=device)
        y2 = torch.empty((M, layer.N), dtype=torch.float16, device=device)
        pairs = [(ls_main.lin[cp][ig], ls_main.lin[cp][iu]) for cp in range(ls_main.copies)]
        fused = lambda cp: P.qlinear_forward_gated_raw(pairs[cp][0], pairs[cp][1], x.data_ptr(), y.data_ptr(), M, act)
        plain = lambda cp: P.qlinear_forward_group_raw(list(pairs[cp]), x.data_ptr(), [y.data_ptr(), y2.data_ptr()], M)
        rec = {"M": M}
        for name, fn in (("gated", fused), ("grouped", plain)):
            if stage == "decode":
                graph = capture_graph(torch, lambda i: fn(i % ls_main.copies), ls_main.copies)
                for _ in range(3):
                    graph.replay()
                ms, repeats, clocks = timed_region(torch, graph.replay, ls_main.copies, sidx, 0.25)
            else:
                def block():
                    for cp in range(ls_main.copies):
                        fn(cp)
                block()
                ms, repeats, clocks = timed_region(torch, block, ls_main.copies, sidx, 0.25)
            rec[name + "_us"] = ms * 1e3 / (repeats * ls_main.copies)
            rec[name + "_sm_mhz"] = clocks["sm_mhz"]
        if stage == "decode":
            rec["gated_gbs"] = wbytes / 1e3 / rec["gated_us"]
            rec["gated_frac_of_measured_peak"] = rec["gated_gbs"] / peaks["hbm_gbs"]
        else:
            fl = layer.flops(M) + w.layers[iu].flops(M)
            rec["gated_tflops"] = fl / 1e6 / rec["gated_us"]
            rec["grouped_tflops"] = fl / 1e6 / rec["grouped_us"]
            rec["y_bytes_written"] = {"gated": 2 * M * layer.N, "grouped": 4 * M * layer.N}
        out[stage] = rec
    return out


def a8_record(torch, device, peaks, sidx):
    """Int8 activations (paper Section 3.7) next to the fp16-activation kernels on the same weights: decode on the LM
    head (quantisation fused into the kernel), prefill at M = 2048 on the Llama shapes in the paper's per-channel 8/4/4
    scheme (quantisation kernel + integer tensor-core matmul; the times include the quantisation kernel)."""
    import paper_2505_00232_b200 as P
    out = {}
    # ---- decode, LM head
    w = C.CONFIG_5B
    layer = w.layers[0]
    desc = P.Desc(layer.N, layer.K, layer.bits, layer.group)
    blob = torch.from_numpy(P.qlinear_pack(desc, *C.layer_weights(w.seed, layer, 0))).to(device)
    lins = [P.QLinear(desc, blob), P.QLinear(desc, blob.clone())]
    x = torch.from_numpy(C.layer_activations(w.seed, layer, 1, 0)).to(device)
    y = torch.empty((1, layer.N), dtype=torch.float16, device=device)
    rec = {"layer": f"lm_head {layer.N}x{layer.K} int4 group 32", "M": 1}
    for name in ("f16", "a8"):
        fn = (lambda cp: lins[cp].forward_raw(x.data_ptr(), y.data_ptr(), 1)) if name == "f16" else \
             (lambda cp: lins[cp].forward_a8_raw(x.data_ptr(), y.data_ptr(), 1))
        graph = capture_graph(torch, lambda i: fn(i % 2), 2)
        for _ in range(3):
            graph.replay()
        ms, repeats, clocks = timed_region(torch, graph.replay, 2, sidx, 0.25)
        us = ms * 1e3 / (2 * repeats)
        rec[name] = {"us": us, "gbs": layer.weight_bytes / 1e3 / us, "frac_of_measured_peak": layer.weight_bytes / 1e3 / us / peaks["hbm_gbs"],
                     "sm_mhz": clocks["sm_mhz"]}
    out["decode"] = rec
    del lins, blob
    torch.cuda.empty_cache()
    # ---- prefill, Llama shapes, per-channel 8/4/4
    wl = C.by_name("llama31_8b_decode_pc4")
    M = 2048
    rows = []
    tot = {"f16": 0.0, "a8": 0.0}
    flops = 0
    for li, layer in enumerate(wl.layers):
        if layer.name in ("k", "v", "up"):
            continue                                                      # same shapes as q / gate; k and v alone have too few tiles for this kernel
        desc = P.Desc(layer.N, layer.K, layer.bits, layer.group)
        blob = torch.from_numpy(P.qlinear_pack(desc, *C.layer_weights(wl.seed, layer, li))).to(device)
        lins = [P.QLinear(desc, blob), P.QLinear(desc, blob.clone())]
        x = torch.from_numpy(C.layer_activations(wl.seed, layer, M, li)).to(device)
        y = torch.empty((M, layer.N), dtype=torch.float16, device=device)
        r = {"layer": f"{layer.name} {layer.N}x{layer.K} int{layer.bits} per channel"}
        for name in ("f16", "a8"):
            fn = (lambda cp: lins[cp].forward_raw(x.data_ptr(), y.data_ptr(), M)) if name == "f16" else \
                 (lambda cp: lins[cp].forward_a8_raw(x.data_ptr(), y.data_ptr(), M))

            def block():
                fn(0)
                fn(1)
            block()
            ms, repeats, clocks = timed_region(torch, block, 2, sidx, 0.25)
            us = ms * 1e3 / (2 * repeats)
            r[name] = {"us": us, "tera_ops": layer.flops(M) / 1e6 / us, "sm_mhz": clocks["sm_mhz"]}
            tot[name] += us
        flops += layer.flops(M)
        rows.append(r)
        del lins, blob
        torch.cuda.empty_cache()
    out["prefill"] = {"M": M, "layers": rows, "sum": {k: {"us": v, "tera_ops": flops / 1e6 / v} for k, v in tot.items()},
                      "note": "a8 = quantisation kernel + kind::i8 matmul; tera_ops counts 2*M*N*K for both"}
    return out


def decode_configs(torch, device, peaks, sidx, ls_main, line):
    """One entry per decode workload of the benchmark: the benchmark's configs 1-3 (config 3 at M = 1 and M = 4), the
    LM head (5b), and the two schemes of the paper's Section 4.2 on the Llama shapes (q8; 8/4/4 per channel)."""
    main = {"workload": line["config"]["workload"], "M": line["config"]["M"], "metric": line["metric"], "value": line["value"],
            "unit": line["unit"], "us_per_step": line["ms_per_step"] * 1e3, "frac_of_measured_peak": line["frac_of_measured_peak"],
            "weight_bytes_per_step": ls_main.weight_bytes, "weight_copies": ls_main.copies, "launches_per_step": ls_main.launches_grouped,
            "steps": line["steps"], "repeats": line["repeats"], "timed_region_ms": line["timed_region_ms"], "clocks": line["clocks"],
            "gpu_launches": line["gpu_launches"], "note": "the headline of this line"}
    out = [config_entry(torch, device, peaks, sidx, "int8_gemv_2304", 1), config_entry(torch, device, peaks, sidx, "gemma2_2b_decode", 1), main,
           config_entry(torch, device, peaks, sidx, "llama31_8b_decode", 4, copies=ls_main.copies, blobs=ls_main.blob0),
           config_entry(torch, device, peaks, sidx, "llama31_8b_lm_head", 1)]
    # the paper's schemes: bytes ratio and time ratio next to its "up to 1.9x" for decode (Section 4.2)
    q8 = config_entry(torch, device, peaks, sidx, "llama31_8b_decode_q8", 1)
    pc4 = config_entry(torch, device, peaks, sidx, "llama31_8b_decode_pc4", 1)
    for e in (main, q8, pc4):
        e["vs_q8"] = {"bytes_ratio": q8["weight_bytes_per_step"] / e["weight_bytes_per_step"],
                      "time_ratio": q8["us_per_step"] / e["us_per_step"],
                      "paper": "decode up to 1.9x faster with 8/4/4 than with q8 (Section 4.2; other hardware)"}
    return out + [q8, pc4]


def prefill_configs(torch, device, peaks, sidx, line):
    """The prefill workloads: config 4 (Gemma2-2B FFN, M = 1024) and config 5 (the 'prefill' record of this line)."""
    out = [config_entry(torch, device, peaks, sidx, "gemma2_2b_prefill", 1024)]
    if "prefill" in line and "value" in line["prefill"]:
        pf = line["prefill"]
        out.append({"workload": "llama31_8b_prefill", "M": pf["config"]["M"], "metric": pf["metric"], "value": pf["value"], "unit": pf["unit"],
                    "us_per_step": pf["ms_per_step"] * 1e3, "frac_of_measured_peak": pf["frac_of_measured_peak"],
                    "steps": pf["steps"], "repeats": pf["repeats"], "timed_region_ms": pf["timed_region_ms"], "clocks": pf["clocks"],
                    "gpu_launches": pf["gpu_launches"], "note": "same record as 'prefill'"})
    return out


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the multi-Bulyan aggregation path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--d D] [--quick] [--impl reference]

A step is one whole aggregation GAR(f, [G_1..G_n]) (distances -> selection ->
coordinate phase) of one synthetic workload resident in HBM.  One JSON line is
printed by rank 0: the headline on the chosen workload (default: the largest,
n = 15, d = 1e9), `per_config` with the same measurement on the three workloads
of the d >= 1e7 regime, the CPU oracle timed on a sample, and the end-to-end
figure through the host entry point.  `--quick --d D` runs a workload's recipe at
another dimension and prints the device-side numbers only (the command line the
profiler captures under profiles/ are taken on).  With N > 1 (torchrun) the workload's
coordinates are sharded over the N GPUs and a step is one aggregation by all of them
(paper_1905_04374_b200/sharded.py): strong scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "multi_bulyan_aggregations_per_sec"
UNIT = "aggregations/s"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) per coordinate of the dominant kernels, from the ncu captures under
# profiles/ (kernel, n) -> bytes; a kernel that changed since its capture has no entry.
NCU_DRAM_BYTES_PER_COORD = {
    ("k1_distances", 39): 1313.0e6 / 8388608, ("k3_coordinate", 39): 1041.5e6 / 8388608,     # k1_umma (packed) / k3_bulk<19, V=2>
    ("k1_distances", 51): 1718.0e6 / 8388608, ("k3_coordinate", 51): 1680.0e6 / 8388608,     # k1_umma (wide) / k3_bulk<25, V=2>
    ("k1_distances", 15): 1010.8e6 / 16777216, ("k3_coordinate", 15): 731.8e6 / 16777216,    # k1_direct_bulk / k3_bulk<7, V=4>
}


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    def __init__(self, index: int, period: float = 0.002):
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None

    def _run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
            }
            while not self._stop.is_set():
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                    for bit, name in names.items():
                        if mask & bit:
                            self.reasons.add(name)
                except Exception:
                    pass
                time.sleep(self.period)
        except Exception as exc:  # pragma: no cover
            self.reasons.add(f"sampler_error:{type(exc).__name__}")

    def __enter__(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thr.join(timeout=2)

    def summary(self):
        s = sorted(self.samples)
        med = s[len(s) // 2] if s else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(s)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# columns of the CPU-baseline sample per workload: about 10 to 30 s of the numpy oracle on one core
CPU_SAMPLE = {1: 100_000, 2: 1 << 20, 3: 1 << 22, 4: 1 << 21, 5: 1 << 25}
REF_SAMPLE = {1: 100_000, 2: 1 << 18, 3: 1 << 18, 4: 1 << 17, 5: 1 << 21}


def oracle_sample_time(cfg: int, d_sample: int):
    """Times the CPU oracle, as it stands, on a d_sample-column sample of the workload."""
    import numpy as np
    from oracle import gar_oracle as O
    from paper_1905_04374_b200 import workloads
    wl = workloads.WORKLOADS[cfg]
    d_sample = min(d_sample, wl.d)
    G, _ = workloads.make_gradients(cfg, d=d_sample, device="cpu")
    Gh = G.numpy()
    t0 = time.perf_counter()
    out, _, _ = O.multi_bulyan(Gh, wl.f)
    dt = time.perf_counter() - t0
    assert np.all(np.isfinite(out))
    return dt, wl, d_sample


def cpu_baseline(cfg: int, d_sample: int):
    dt, wl, d_sample = oracle_sample_time(cfg, d_sample)
    per_full = dt * (wl.d / d_sample)
    return {"value": 1.0 / per_full, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"numpy fp64 oracle on the first {d_sample} of {wl.d} coordinates of {wl.name} "
                      f"({dt:.2f} s), scaled by d/sample", "seconds_sample": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_1905_04374_b200 import workloads
    wl = workloads.WORKLOADS[args.config]
    d_sample = min(args.ref_sample or REF_SAMPLE[args.config], wl.d)
    times = []
    for i in range(args.warmup + args.steps):
        dt, _, _ = oracle_sample_time(args.config, d_sample)
        if i >= args.warmup:
            times.append(dt)
    per_step_full = (sum(times) / len(times)) * (wl.d / d_sample)
    value = 1.0 / per_step_full
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step_full * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "n": wl.n, "f": wl.f, "d": wl.d, "rule": "multi_bulyan"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"each step: numpy fp64 oracle on the first {d_sample} of {wl.d} coordinates, "
                                   f"scaled by d/sample"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def event_time_ms(fn, reps, stream):
    import torch
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record(stream)
    for _ in range(reps):
        fn()
    stop.record(stream)
    torch.cuda.synchronize()
    return start.elapsed_time(stop) / reps


def max_over_ranks(elapsed_ms: float, world: int, device=None) -> float:
    """Slowest rank's time (every rank must call it): the job is only as fast as that rank."""
    if world <= 1:
        return elapsed_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def launches_per_aggregation(n: int, d: int, theta: int) -> int:
    """Kernels of this library one multi-Bulyan call launches on 16-byte aligned rows: the distance
    kernel (for n > 16 and d >= 32768 the tensor-core kernel plus the gated difference-form kernel
    behind it), the selection kernel, the staged coordinate kernel (from 400000 coordinates on) and
    the register kernel for what is left after the last whole tile."""
    k1 = 2 if (n > 16 and d >= 32768) else 1
    if d >= 400_000:
        tile = 512 if theta <= 12 else 256
        k3 = 1 + (1 if d % tile else 0)
    else:
        k3 = 1
    return k1 + 1 + k3


def measure_workload(pkg, cfg, dev, steps, warmup, world, local, d=None, variant=True, distance_mode="auto",
                     dtype="f32"):
    """Device-side measurement of one workload resident in HBM: `steps` whole aggregations timed
    with CUDA events on the launch stream (max over ranks), then each stage alone."""
    import torch
    import torch.distributed as dist
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f = wl.n, wl.f
    d = d or wl.d
    theta_a = pkg.gar_theta("multi_bulyan", n, f)
    theta_b = pkg.gar_theta("bulyan", n, f)
    G, _ = pkg.workloads.make_gradients(cfg, d=d, device=dev)
    out = torch.empty(d, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    if dtype != "f32":
        # 16-bit gradients: the same draw rounded to bfloat16 / binary16; only the whole call is timed
        # (the stage calls of the C ABI take fp32 gradients)
        G16 = torch.empty(n, d, dtype=torch.bfloat16 if dtype == "bf16" else torch.float16, device=dev)
        for c0 in range(0, d, 1 << 24):
            G16[:, c0:c0 + (1 << 24)] = G[:, c0:c0 + (1 << 24)]
        del G
        torch.cuda.empty_cache()
        for _ in range(max(warmup, 3)):
            pkg.gar_aggregate_ex("multi_bulyan", G16, f, out=out)
        torch.cuda.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(physical_gpu_index(local), period=0.002) as clocks:
            start.record(stream)
            for _ in range(steps):
                pkg.gar_aggregate_ex("multi_bulyan", G16, f, out=out)
            stop.record(stream)
            torch.cuda.synchronize()
        ms = start.elapsed_time(stop) / steps
        peak, _ = measured_hbm_peak()
        bytes16 = 2.0 * d * (n + theta_b) + 4.0 * d
        return {"workload": f"{wl.name} recipe at d={d}, {dtype} gradients", "n": n, "f": f, "d": d, "theta": theta_a,
                "ms_per_aggregation": ms, "aggregations_per_sec": 1e3 / ms, "steps": steps, "kernels": {},
                "roofline": None, "path": {"bytes_min_16bit_rows": bytes16, "effective_gbs": bytes16 / (ms * 1e-3) / 1e9,
                                           "frac_of_measured_peak": bytes16 / (ms * 1e-3) / 1e9 / peak},
                "clocks": clocks.summary(), "elapsed_ms": ms * steps}, G16

    def step():
        if distance_mode == "auto":
            pkg.gar_aggregate("multi_bulyan", G, f, out=out)
        else:
            pkg.gar_aggregate_ex("multi_bulyan", G, f, out=out, distance_mode=distance_mode)

    for _ in range(max(warmup, 3)):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(physical_gpu_index(local), period=0.002) as clocks:
        torch.cuda.synchronize()
        start.record(stream)
        for _ in range(steps):
            step()
        stop.record(stream)
        torch.cuda.synchronize()
    elapsed_ms = max_over_ranks(start.elapsed_time(stop), world, dev)
    if world > 1:
        dist.barrier()
    ms_per_step = elapsed_ms / steps

    # ---- per-kernel durations, measured live with CUDA events on the launch stream
    reps = max(5, min(50, steps))
    ws = torch.zeros(pkg.gar_workspace_bytes("multi_bulyan", n, f, d), dtype=torch.uint8, device=dev)
    dmat = torch.empty(n, n, dtype=torch.float64, device=dev)
    sel = pkg.new_selection(dev)
    pkg.gar_pairwise_distances(G, dist=dmat, workspace=ws, distance_mode=distance_mode)
    pkg.gar_select("multi_bulyan", dmat, n, f, sel=sel)
    k1_ms = event_time_ms(lambda: pkg.gar_pairwise_distances(G, dist=dmat, workspace=ws, distance_mode=distance_mode),
                          reps, stream)
    k2_ms = event_time_ms(lambda: pkg.gar_select("multi_bulyan", dmat, n, f, sel=sel), reps, stream)
    k3_ms = event_time_ms(lambda: pkg.gar_coordinate_phase(G, sel, theta_a, 1, out=out), reps, stream)
    selh = pkg.read_selection(sel)
    rows_k3 = int(selh.nu)
    peak, peak_kind = measured_hbm_peak()
    k1_bytes = 4.0 * n * d
    k3_bytes = 4.0 * d * ((rows_k3 if rows_k3 else theta_a) + 1)
    kernels = {
        "k1_distances": {"ms": k1_ms, "algorithmic_bytes": k1_bytes, "gbs": k1_bytes / (k1_ms * 1e-3) / 1e9,
                         "frac_of_measured_peak": k1_bytes / (k1_ms * 1e-3) / 1e9 / peak,
                         "path": pkg.distance_path(ws)},
        "k2_select": {"ms": k2_ms},
        "k3_coordinate": {"ms": k3_ms, "algorithmic_bytes": k3_bytes, "gbs": k3_bytes / (k3_ms * 1e-3) / 1e9,
                          "frac_of_measured_peak": k3_bytes / (k3_ms * 1e-3) / 1e9 / peak, "rows_read": rows_k3},
    }
    dom = "k1_distances" if k1_ms >= k3_ms else "k3_coordinate"
    achieved = kernels[dom]["gbs"]
    per_coord = NCU_DRAM_BYTES_PER_COORD.get((dom, n))
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": peak_kind,
                "traffic": per_coord * d if per_coord else None,
                "algorithmic_bytes": kernels[dom]["algorithmic_bytes"]}
    # whole-path effective bandwidth against the minimum traffic (n + theta + 1) * 4 d with
    # theta = n - 2f, and against this rule's own minimum (n + |U| + 1) * 4 d
    bytes_formula = 4.0 * d * (n + theta_b + 1)
    bytes_own = 4.0 * d * (n + (rows_k3 if rows_k3 else theta_a) + 1)
    path = {
        "bytes_min_n_plus_theta_plus_1": bytes_formula,
        "bytes_min_this_rule": bytes_own,
        "effective_gbs": bytes_formula / (ms_per_step * 1e-3) / 1e9,
        "effective_gbs_this_rule": bytes_own / (ms_per_step * 1e-3) / 1e9,
    }
    path["frac_of_nominal_8TBs"] = path["effective_gbs"] / NOMINAL_HBM_GBS
    path["frac_of_measured_peak"] = path["effective_gbs"] / peak
    path["frac_of_measured_peak_this_rule"] = path["effective_gbs_this_rule"] / peak
    res = {"workload": wl.name if d == wl.d else f"{wl.name} recipe at d={d}", "n": n, "f": f, "d": d,
           "theta": theta_a, "ms_per_aggregation": ms_per_step, "aggregations_per_sec": 1e3 / ms_per_step,
           "steps": steps, "kernels": kernels, "roofline": roofline, "path": path, "clocks": clocks.summary(),
           "elapsed_ms": elapsed_ms}
    if variant:
        # the same workload under the rule whose three-part summary speaks of theta = n - 2f iterated
        # Krum winners and beta = theta - 2f, no pre-aggregation: GAR_BULYAN
        k3b_sel = pkg.new_selection(dev)
        pkg.gar_select("bulyan", dmat, n, f, sel=k3b_sel)
        k3b_ms = event_time_ms(lambda: pkg.gar_coordinate_phase(G, k3b_sel, theta_b, 0, out=out), reps, stream)
        bulyan_ms = event_time_ms(lambda: pkg.gar_aggregate("bulyan", G, f, out=out), reps, stream)
        res["variant_bulyan"] = {
            "rule": "bulyan", "theta": theta_b, "beta": pkg.gar_beta("bulyan", n, f), "ms_per_aggregation": bulyan_ms,
            "aggregations_per_sec": 1e3 / bulyan_ms, "k3_coordinate_ms": k3b_ms,
            "effective_gbs": bytes_formula / (bulyan_ms * 1e-3) / 1e9,
            "frac_of_measured_peak": bytes_formula / (bulyan_ms * 1e-3) / 1e9 / peak,
            "frac_of_nominal_8TBs": bytes_formula / (bulyan_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS}
    return res, G


def resnet18_lengths():
    """Parameter-tensor lengths of an 18-layer residual network with 1000 outputs (62 tensors,
    11,689,512 parameters): convolution weights, the two vectors of every normalisation layer,
    the final linear layer."""
    out = [64 * 3 * 7 * 7, 64, 64]
    cin = 64
    for cout in (64, 128, 256, 512):
        for block in range(2):
            first = block == 0 and cout != 64
            out += [cout * cin * 9, cout, cout, cout * cout * 9, cout, cout]
            if first:
                out += [cout * cin, cout, cout]
            cin = cout
    return out + [512 * 1000, 1000]


# Per-layer mixes the batched call is timed on: (n, f, tensor lengths).
LAYER_MIXES = {
    # a network of two convolutions and two linear layers with d = 431,080 parameters (the size of
    # the model in Section 5), as weight and bias tensors: 5x5 kernels, 1 -> 20 -> 50 channels,
    # 800 -> 500 -> 10 units
    "cnn_d431080": (11, 2, [500, 20, 25_000, 50, 400_000, 500, 5_000, 10]),
    "resnet18_lengths": (15, 3, resnet18_lengths()),
}


def measure_multi(pkg, dev, reps=20):
    """gar_aggregate_multi (independent problems, and the tensors as one gradient) against one
    gar_aggregate_ex per tensor, on per-layer tensors; CUDA events, inputs resident."""
    import torch
    results = []
    for name, (n, f, dims) in LAYER_MIXES.items():
        gen = torch.Generator(device=dev)
        gen.manual_seed(workloads_seed(name))
        parts = [torch.randn(n, d, generator=gen, device=dev, dtype=torch.float32) for d in dims]
        for g in parts:
            g[n - f:] += 20.0
        count = len(parts)
        outs = [torch.empty(d, dtype=torch.float32, device=dev) for d in dims]
        ws = torch.empty(pkg.gar_multi_workspace_bytes("multi_bulyan", n, f, count), dtype=torch.uint8, device=dev)
        entry = {"mix": name, "n": n, "f": f, "tensors": count, "d_total": int(sum(dims)), "rule": "multi_bulyan"}

        def timed(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps

        entry["ms_multi_independent"] = timed(lambda: pkg.gar_aggregate_multi("multi_bulyan", parts, f, outs=outs, workspace=ws))
        entry["ms_multi_joint"] = timed(lambda: pkg.gar_aggregate_multi("multi_bulyan", parts, f, outs=outs, workspace=ws, joint=True))
        entry["ms_one_call_per_tensor"] = timed(lambda: [pkg.gar_aggregate_ex("multi_bulyan", g, f, out=o) for g, o in zip(parts, outs)])
        flat = torch.cat(parts, dim=1).contiguous()
        flat_out = torch.empty(flat.shape[1], dtype=torch.float32, device=dev)
        entry["ms_one_call_on_the_concatenation"] = timed(lambda: pkg.gar_aggregate_ex("multi_bulyan", flat, f, out=flat_out))
        entry["hbm_floor_ms"] = 4.0 * sum(dims) * (2 * n + 1) / (measured_hbm_peak()[0] * 1e9) * 1e3
        results.append(entry)
        del parts, outs, flat, flat_out, ws
        torch.cuda.empty_cache()
    return results


def measure_small(pkg, dev, reps=200):
    """Workloads 1 and 2 (d = 1e5, 1e6): three dependent launches, latency-bound.  Time per
    aggregation of plain calls and of a CUDA graph of the same three launches replayed."""
    import torch
    out = []
    for cfg in (1, 2):
        wl = pkg.workloads.WORKLOADS[cfg]
        G, _ = pkg.workloads.make_gradients(cfg, device=dev)
        res = torch.empty(wl.d, dtype=torch.float32, device=dev)
        ws = torch.zeros(pkg.gar_workspace_bytes("multi_bulyan", wl.n, wl.f, wl.d), dtype=torch.uint8, device=dev)
        call = lambda: pkg.gar_aggregate_ex("multi_bulyan", G, wl.f, out=res, workspace=ws)
        for _ in range(5):
            call()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            call()

        def timed(fn):
            for _ in range(5):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps

        out.append({"workload": wl.name, "n": wl.n, "f": wl.f, "d": wl.d,
                    "bound": "latency (three dependent launches)",
                    "ms_per_aggregation": timed(call), "ms_per_aggregation_graph_replay": timed(graph.replay),
                    "hbm_floor_ms": 4.0 * wl.d * (2 * wl.n + 1) / (measured_hbm_peak()[0] * 1e9) * 1e3})
        del graph, G, res, ws
        torch.cuda.empty_cache()
    return out


def workloads_seed(name):
    return 20_190_509 + sum(ord(c) for c in name)


def run_e2e(pkg, cfg, G, steps):
    """The same aggregation through the host entry point: pinned host buffers, both copies inside
    the timed region."""
    import torch
    n, d = G.shape
    f = pkg.workloads.WORKLOADS[cfg].f
    host = torch.empty(n, d, dtype=torch.float32, pin_memory=True)
    host.copy_(G)
    hout = torch.empty(d, dtype=torch.float32, pin_memory=True)
    pkg.gar_aggregate_host("multi_bulyan", host, f, out=hout)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        pkg.gar_aggregate_host("multi_bulyan", host, f, out=hout)
    t1 = time.perf_counter()
    return {"value": steps / (t1 - t0), "unit": UNIT, "h2d_bytes_per_step": int(4 * n * d),
            "d2h_bytes_per_step": int(4 * d) + 4, "steps": steps,
            "api": "gar_aggregate_host (pinned host buffers, synchronous)"}


def run_sharded(pkg, args, dev, world, rank, local):
    """N > 1: ONE aggregation spread over the N GPUs.  The workload's coordinates are split into
    contiguous column ranges, one per rank (whole generator chunks); a step is
    paper_1905_04374_b200.sharded.sharded_aggregate: local distance partials, one all-gather of
    n*n fp64 values per rank (NCCL), the sum in rank order, the replicated selection and the local
    coordinate phase.  Total work is fixed as N grows: strong scaling."""
    import torch
    import torch.distributed as dist
    from paper_1905_04374_b200 import sharded
    cfg = args.config
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f = wl.n, wl.f
    d = args.d or wl.d
    c0, c1 = pkg.workloads.shard_columns(d, world, rank)
    if c1 > c0:
        G, _ = pkg.workloads.make_gradients(cfg, d=d, device=dev, columns=(c0, c1))
    else:
        G = torch.empty(n, 0, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        return sharded.sharded_aggregate("multi_bulyan", G, f)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    dist.barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(physical_gpu_index(local), period=0.002) as clocks:
        torch.cuda.synchronize()
        start.record(stream)
        for _ in range(args.steps):
            step()
        stop.record(stream)
        torch.cuda.synchronize()
    elapsed_ms = max_over_ranks(start.elapsed_time(stop), world, dev)
    dist.barrier()
    # end to end: this rank's slice from pinned host memory, the sharded call, its slice of the result back
    e2e_steps = max(2, min(args.steps, args.e2e_steps))
    host = torch.empty(G.shape, dtype=torch.float32, pin_memory=True)
    host.copy_(G)
    hout = torch.empty(c1 - c0, dtype=torch.float32, pin_memory=True)
    stage = torch.empty_like(G)

    def e2e_step():
        stage.copy_(host, non_blocking=True)
        out, _, _ = sharded.sharded_aggregate("multi_bulyan", stage, f)
        hout.copy_(out, non_blocking=True)
        torch.cuda.synchronize()

    e2e_step()
    dist.barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    dist.barrier()
    e2e_s = time.perf_counter() - t0
    e2e_ms = max_over_ranks(e2e_s * 1e3, world, dev)
    if rank != 0:
        return
    ms_per_step = elapsed_ms / args.steps
    theta_b = pkg.gar_theta("bulyan", n, f)
    peak, peak_kind = measured_hbm_peak()
    bytes_formula = 4.0 * d * (n + theta_b + 1)
    line = {
        "metric": METRIC, "value": args.steps / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name if d == wl.d else f"{wl.name} recipe at d={d}", "n": n, "f": f, "d": d,
                   "rule": "multi_bulyan", "theta": pkg.gar_theta("multi_bulyan", n, f),
                   "beta": pkg.gar_beta("multi_bulyan", n, f),
                   "parallelism": f"coordinates sharded over {world} GPUs; one all-gather of n*n fp64 per aggregation",
                   "l2": "every rank's slice is larger than L2; no flush"},
        "roofline": None,
        "path": {"bytes_min_n_plus_theta_plus_1": bytes_formula,
                 "effective_gbs": bytes_formula / (ms_per_step * 1e-3) / 1e9,
                 "frac_of_measured_peak_all_gpus": bytes_formula / (ms_per_step * 1e-3) / 1e9 / (peak * world)},
        "cpu_baseline": None,
        "e2e": {"value": e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(4 * n * d),
                "d2h_bytes_per_step": int(4 * d), "steps": e2e_steps,
                "api": "sharded_aggregate on slices copied from pinned host memory, result slices copied back"},
        "gpu_launches": (launches_per_aggregation(n, max(c1 - c0, 1), pkg.gar_theta("multi_bulyan", n, f)) + 1) * args.steps,
        "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_1905_04374_b200 as pkg

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1 or args.force_sharded:
        os.environ.setdefault("NCCL_DEBUG", "WARN")     # keep NCCL's version banner off stdout: one JSON line
        dist.init_process_group("nccl", device_id=dev)

    cfg = args.config
    if args.multi_only:
        if rank == 0:
            print(json.dumps({"multi_tensor": measure_multi(pkg, dev), "small_d": measure_small(pkg, dev)}), flush=True)
        return
    if world > 1 or args.force_sharded:
        run_sharded(pkg, args, dev, world, rank, local)
        dist.destroy_process_group()
        return
    main, G = measure_workload(pkg, cfg, dev, args.steps, args.warmup, world, local, d=args.d,
                               distance_mode=args.distance_mode, dtype=args.dtype)
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f, d = main["n"], main["f"], main["d"]
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    value = world * args.steps / (main["elapsed_ms"] * 1e-3)

    e2e = None
    if not args.no_e2e:
        try:
            e2e = run_e2e(pkg, cfg, G, max(2, min(args.steps, args.e2e_steps)))
        except Exception as exc:                      # e.g. the host cannot pin a 60 GB buffer
            e2e = {"value": None, "unit": UNIT, "error": f"{type(exc).__name__}: {exc}"[:200]}
        pkg.gar_shutdown()                            # give the host path's staging copy back
    del G
    torch.cuda.empty_cache()

    # the other single-GPU workloads of the d >= 1e7 regime, same measurement, same run
    per_config = []
    if not args.no_per_config and args.d is None:
        for other in (3, 4, 5):
            if other == cfg:
                entry = {k: main[k] for k in main if k != "elapsed_ms"}
            else:
                owl = pkg.workloads.WORKLOADS[other]
                approx_ms = {3: 1.6, 4: 10.0, 5: 19.0}[other]
                osteps = max(20, int(1000.0 / approx_ms))          # about a second of timed work
                entry, Go = measure_workload(pkg, other, dev, osteps, 3, 1, local)
                del Go
                torch.cuda.empty_cache()
                entry.pop("elapsed_ms")
            per_config.append(entry)

    multi = None if args.no_multi else measure_multi(pkg, dev)
    small = None if args.no_multi else measure_small(pkg, dev)
    cpu = None if args.no_cpu_baseline else cpu_baseline(cfg, args.cpu_sample or CPU_SAMPLE[cfg])

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": main["ms_per_aggregation"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": main["workload"], "n": n, "f": f, "d": d, "rule": "multi_bulyan", "theta": main["theta"],
                   "beta": pkg.gar_beta("multi_bulyan", n, f), "parallelism": f"replicas x{world}",
                   "grads_dtype": args.dtype,
                   "why_this_workload": "the largest of the five configurations; it fits one GPU (60 GB of 180)",
                   "l2": "input (%.2f GB) larger than L2; no flush" % (4e-9 * n * d) if 4 * n * d > 2.6e8
                   else "input fits L2; not flushed between steps"},
        "roofline": main["roofline"], "path": main["path"], "kernels": main["kernels"],
        "variant_bulyan": main.get("variant_bulyan"), "per_config": per_config, "small_d": small, "multi_tensor": multi, "cpu_baseline": cpu, "e2e": e2e,
        "gpu_launches": launches_per_aggregation(n, d, main["theta"]) * args.steps, "clocks": main["clocks"],
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=5,
                    help="workload 1..5 (default 5: n=15, f=3, d=1e9, the largest single-GPU configuration)")
    ap.add_argument("--d", type=int, default=None, help="another dimension for the workload's recipe (profiling)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-sample", type=int, default=0, help="columns of the CPU-baseline sample (0: per workload)")
    ap.add_argument("--ref-sample", type=int, default=0, help="columns per step of --impl reference (0: per workload)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--no-multi", action="store_true", help="skip the timing of the batched per-layer call")
    ap.add_argument("--multi-only", action="store_true", help="print the batched per-layer call's timings and exit")
    ap.add_argument("--quick", action="store_true", help="device-side numbers of the chosen workload only")
    ap.add_argument("--distance-mode", default="auto", choices=["auto", "difference"],
                    help="difference: the fp32 difference-form distance kernels instead of the tensor-core one")
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16", "f16"],
                    help="element type of the gradients (16-bit: whole-call timing only, implies --quick)")
    ap.add_argument("--force-sharded", action="store_true",
                    help="run the sharded (N > 1) code path even with one rank (under torchrun, for checking it)")
    args = ap.parse_args()
    if args.dtype != "f32":
        args.quick = True
    if args.quick:
        args.no_e2e = args.no_cpu_baseline = args.no_per_config = args.no_multi = True
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

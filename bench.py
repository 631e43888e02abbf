#!/usr/bin/env python
"""Benchmark of Y = act(A.B + bias) on B200 through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

A step is one pass of the whole hot path (dispatch, operand staging, contraction,
split-K reduce where used, fused epilogue, store) over one synthetic problem.  The
headline line is for one workload (default c2, the bf16 GEMV-like shape); the same JSON
line carries a `per_shape` list with all five workloads, each with TFLOP/s, GB/s and its
roofline fraction.  Inputs are seeded and synthetic.  One JSON line goes to stdout.

Timing: W untimed warm-up steps, then exactly K steps between a barrier + synchronize on
both sides, CUDA events on the launching stream, max over ranks.  Consecutive steps use
different buffer sets whose total size is several times the L2 cache, so no step finds
its operands in L2 from the step before.  SM clocks and throttle reasons are sampled
through NVML while the timed region runs.

N > 1: the path does not shard; every rank runs an independent replica on its own GPU
(no data-path collective) and the aggregate is reported ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2602_12305_b200 import replicas, synth  # noqa: E402

METRIC = "TFLOP/s and HBM GB/s per shape on 1 B200, as % of roofline"
L2_BYTES = 126 * 1024 * 1024
# Roofline each workload is bounded by: plain FMA pipes (fp32, no tensor cores), HBM, tensor cores.
BOUND = {"c1": "alu", "c2": "hbm", "c3": "hbm", "c4": "tensor", "c5": "tensor"}
# FMA-pipe peak: 148 SMs x 128 fp32 lanes x 2 flop x 1.965 GHz (maximum SM clock).
FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel,
# from the ncu captures summarised under profiles/; None = not captured for the current kernel.
NCU_TRAFFIC_BYTES = {"c1": 545792, "c2": 138099712, "c3": 121091072, "c4": 107639552, "c5": 4376021872,
                     "sum": 272239616, "dot": 540065280, "mse": None, "a2": 250073088, "a3": 118124032}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# ---------------------------------------------------------------- clocks (NVML, read-only)

_REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
            0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
            0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
_BAD = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}


class ClockSampler(threading.Thread):
    """Samples SM clock, power and clock-event reasons every few milliseconds."""

    def __init__(self, device_index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples = []          # (time, sm_mhz, power_w, reason mask)
        self.ok = False
        self.max_mhz = None
        self._halt = threading.Event()
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def _reasons(self):
        for name in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            fn = getattr(self.nv, name, None)
            if fn is not None:
                try:
                    return int(fn(self.h))
                except Exception:
                    continue
        return 0

    def run(self):
        if not self.ok:
            return
        while not self._halt.is_set():
            try:
                mhz = float(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                try:
                    pw = self.nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                except Exception:
                    pw = float("nan")
                self.samples.append((time.perf_counter(), mhz, pw, self._reasons()))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()

    def window(self, t0: float, t1: float):
        return [s for s in self.samples if t0 <= s[0] <= t1]


def summarise_clocks(samples, max_mhz, how: str):
    if not samples:
        return {"sm_mhz": None, "sm_max_mhz": max_mhz, "reasons": [], "samples": 0, "sampled": "unavailable"}
    mask = 0
    for s in samples:
        mask |= s[3]
    reasons = sorted(n for b, n in _REASONS.items() if mask & b and n != "gpu_idle")
    pw = [s[2] for s in samples if not math.isnan(s[2])]
    return {"sm_mhz": statistics.median(s[1] for s in samples), "sm_max_mhz": max_mhz, "reasons": reasons,
            "samples": len(samples), "power_w_max": max(pw) if pw else None, "sampled": how}


# ---------------------------------------------------------------- device buffers

def to_device(arr, dtype, shape, device):
    if dtype == synth.F32:
        return torch.from_numpy(arr).view(*shape).to(device)
    return torch.from_numpy(arr.view(np.int16)).view(torch.bfloat16).view(*shape).to(device)


def to_pinned(arr, dtype, shape):
    if dtype == synth.F32:
        return torch.from_numpy(arr).view(*shape).pin_memory()
    return torch.from_numpy(arr.view(np.int16)).view(torch.bfloat16).view(*shape).pin_memory()


def make_sets(case, device):
    """Enough distinct (A, B, bias, Y) sets that a round over them moves >= 4 x L2."""
    n = max(2, min(1024, math.ceil(4 * L2_BYTES / case.algorithmic_bytes)))
    tdt = torch.float32 if case.dtype == synth.F32 else torch.bfloat16
    A0 = to_device(case.A, case.dtype, (case.M, case.K), device)
    B0 = to_device(case.B, case.dtype, (case.K, case.N), device)
    b0 = to_device(case.bias, case.dtype, (case.N,), device)
    sets = []
    for i in range(n):
        A, B, b = (A0, B0, b0) if i == 0 else (A0.clone(), B0.clone(), b0.clone())
        sets.append((A, B, b, torch.empty((case.M, case.N), dtype=tdt, device=device)))
    return sets


# ---------------------------------------------------------------- timing of one workload

def time_workload(handle, case, sets, steps, warmup, sampler, device):
    """W warm-up steps, then K timed steps; returns region time, per-launch times, clocks."""
    stream = torch.cuda.current_stream(device)

    # raw C-ABI calls with the device addresses taken once: the per-step host cost is the
    # ctypes call, not tensor bookkeeping
    raw = [(A.data_ptr(), B.data_ptr(), b.data_ptr(), Y.data_ptr()) for A, B, b, Y in sets]
    st = stream.cuda_stream

    def step(i):
        pa, pb, pbias, py = raw[i % len(raw)]
        rc = handle.gemm_epilogue_raw(pa, pb, pbias, py, case.M, case.N, case.K, case.dtype, case.act, st)
        if rc != 0:
            raise RuntimeError(f"optiml_gemm_epilogue returned {rc}")

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize(device)
    replicas.barrier()
    torch.cuda.synchronize(device)
    launches0 = handle.launch_count()
    # Two events bracket the K steps.  (An event record after every step would put 3-4 us of
    # idle time between consecutive kernels; the per-launch average is region / launches.)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(stream)
    for i in range(steps):
        step(warmup + i)
    e1.record(stream)
    torch.cuda.synchronize(device)
    t1 = time.perf_counter()
    replicas.barrier()
    torch.cuda.synchronize(device)
    region_ms = e0.elapsed_time(e1)
    launches = handle.launch_count() - launches0
    win = sampler.window(t0, t1) if sampler else []
    how = "during the timed region"
    if sampler and sampler.ok and len(win) < 3:
        # region too short for the sampling period: keep the same load running a little
        # longer (untimed) and sample the clocks under it
        t2 = time.perf_counter()
        i = 0
        while time.perf_counter() - t2 < 0.25:
            step(i)
            i += 1
            if i % 64 == 0:
                torch.cuda.synchronize(device)
        torch.cuda.synchronize(device)
        win = sampler.window(t2 + 0.05, time.perf_counter())
        how = "same load continued after the timed region (region shorter than the sampling period)"
    return {"region_ms": region_ms, "launches": launches,
            "clocks": summarise_clocks(win, sampler.max_mhz if sampler else None, how)}


def time_e2e(handle, case, steps, warmup, device):
    """The host entry point: pinned host inputs copied in, Y copied back, every step."""
    A = to_pinned(case.A, case.dtype, (case.M, case.K))
    B = to_pinned(case.B, case.dtype, (case.K, case.N))
    b = to_pinned(case.bias, case.dtype, (case.N,))
    tdt = torch.float32 if case.dtype == synth.F32 else torch.bfloat16
    Y = torch.empty((case.M, case.N), dtype=tdt).pin_memory()
    stream = torch.cuda.current_stream(device)
    for _ in range(warmup):
        handle.gemm_epilogue_host(A, B, b, Y, case.act, stream=stream)
    torch.cuda.synchronize(device)
    replicas.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        handle.gemm_epilogue_host(A, B, b, Y, case.act, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize(device)
    replicas.barrier()
    ms = e0.elapsed_time(e1) / steps
    es = 4 if case.dtype == synth.F32 else 2
    return ms, es * (case.M * case.K + case.K * case.N + case.N), es * case.M * case.N


_CASES = {}


def get_case(name):
    """Host arrays of a named workload, generated once per process."""
    if name not in _CASES:
        _CASES[name] = synth.make_case(name)
    return _CASES[name]


def headline_unit(name):
    return "GB/s" if BOUND[name] == "hbm" else "TFLOP/s"


def throughput(case, ms, unit):
    return (case.algorithmic_bytes / 1e9 if unit == "GB/s" else case.flops / 1e12) / (ms / 1e3)


def roofline(case, name, avg_launch_ms, region_s, peaks, peak_src):
    bound = BOUND[name]
    if bound == "hbm":
        ach, peak, unit, kind = case.algorithmic_bytes / 1e9 / (avg_launch_ms / 1e3), peaks["hbm_gbs"], "GB/s", "copy bandwidth"
    elif bound == "tensor":
        sustained = region_s >= 2.0
        peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
        ach, unit, kind = case.flops / 1e12 / (avg_launch_ms / 1e3), "TFLOP/s", "bf16 GEMM " + ("sustained" if sustained else "burst")
    else:
        ach, peak, unit, kind = case.flops / 1e12 / (avg_launch_ms / 1e3), FMA_PEAK_TFLOPS, "TFLOP/s", "fp32 FMA pipes at max clock (derived)"
    src = peak_src if bound != "alu" else "derived"
    extra = {}
    if bound == "tensor":
        # back-to-back launches run under the power cap; the fraction against the sustained
        # bf16 GEMM figure is given beside the one against the burst figure
        extra = {"frac_of_burst": ach / peaks["bf16_tflops"], "frac_of_sustained": ach / peaks["bf16_tflops_sustained"]}
    return {**extra, "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
            "traffic": NCU_TRAFFIC_BYTES.get(name), "peak_source": f"of {src}: {kind}",
            "algorithmic_bytes": case.algorithmic_bytes, "algorithmic_flops": case.flops,
            "avg_launch_ms": avg_launch_ms}


# ---------------------------------------------------------------- CPU baseline (the oracle, as it stands)

def oracle_sample(case, target_macs=2.0e9):
    """Time the oracle on a bounded sample of the workload: the first R rows (all of N and K)."""
    from oracle import oracle
    rows = max(1, min(case.M, int(target_macs // (case.N * case.K)) or 1))
    t0 = time.perf_counter()
    oracle.gemm_epilogue(case.A[:rows * case.K], case.B, case.bias, rows, case.N, case.K, case.dtype, case.act)
    dt = time.perf_counter() - t0
    threads = getattr(oracle.gemm_epilogue, "threads_used", 1)
    es = 4 if case.dtype == synth.F32 else 2
    nbytes = es * (rows * case.K + case.K * case.N + case.N + rows * case.N)
    return {"seconds": dt, "rows": rows, "flops": 2.0 * rows * case.N * case.K, "bytes": nbytes, "cores": threads,
            "sample": f"first {rows} of {case.M} rows, all {case.N} columns, K={case.K}, one pass"}


def cpu_baseline(case, unit):
    s = oracle_sample(case)
    v = (s["bytes"] / 1e9 if unit == "GB/s" else s["flops"] / 1e12) / s["seconds"]
    return {"value": v, "unit": unit, "cores": s["cores"], "kind": "oracle", "sample": s["sample"],
            "seconds": s["seconds"]}


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores, same config and metric."""
    rank, _, world = replicas.env_world()
    if rank != 0:
        return 0
    from oracle import oracle
    name = args.workload
    case = get_case(name)
    unit = headline_unit(name)
    # size the per-step sample so that the whole run stays within about two minutes
    probe_rows = 1
    t0 = time.perf_counter()
    cols = np.arange(min(case.N, 64))
    oracle.gemm_epilogue_sampled(case.A, case.B, case.bias, case.M, case.N, case.K, case.dtype, case.act,
                                 np.arange(probe_rows), cols)
    per_mac = (time.perf_counter() - t0) / (probe_rows * len(cols) * case.K)
    budget = 120.0 / (args.steps + args.warmup)
    n_out = max(8, int(budget / per_mac / case.K))
    rows = np.arange(max(1, min(case.M, n_out // case.N if n_out >= case.N else 1)))
    cols = np.arange(min(case.N, max(8, n_out // len(rows))))

    def step():
        oracle.gemm_epilogue_sampled(case.A, case.B, case.bias, case.M, case.N, case.K, case.dtype, case.act, rows, cols)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    ms = (time.perf_counter() - t0) * 1e3 / args.steps
    es = 4 if case.dtype == synth.F32 else 2
    nb = es * (len(rows) * case.K + case.K * len(cols) + len(cols) + len(rows) * len(cols))
    fl = 2.0 * len(rows) * len(cols) * case.K
    v = (nb / 1e9 if unit == "GB/s" else fl / 1e12) / (ms / 1e3)
    threads = getattr(oracle.gemm_epilogue_sampled, "threads_used", 1)
    sample = f"{len(rows)} rows x {len(cols)} columns of the {case.M}x{case.N} output, K={case.K}, per step"
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": workload_config(case, name, None),
            "cpu_baseline": {"value": v, "unit": unit, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)
    return 0


def workload_config(case, name, variant):
    cfg = {"workload": f"{name}: {'fp32' if case.dtype == synth.F32 else 'bf16'} {case.M}x{case.N}x{case.K} "
                       f"bias + {['none', 'ReLU', 'GELU(tanh)'][case.act]}",
           "arithmetic": "fp32 products and sums on the FMA pipes" if case.dtype == synth.F32
                         else "exact bf16 products, fp32 accumulation, one rounding to bf16 at the store",
           "M": case.M, "N": case.N, "K": case.K,
           "l2": "consecutive steps use different buffer sets; one round over the sets moves >= 4 x L2"}
    if variant is not None:
        cfg["variant"] = variant
    return cfg


# ---------------------------------------------------------------- main

def measure(handle, name, args, sampler, device, peaks, peak_src, steps, warmup, with_e2e=True):
    from paper_2602_12305_b200 import binding
    case = get_case(name)
    sets = make_sets(case, device)
    unit = headline_unit(name)
    res = time_workload(handle, case, sets, steps, warmup, sampler, device)
    bad = _BAD.intersection(res["clocks"]["reasons"])
    stuck = (res["clocks"]["sm_mhz"] is not None and res["clocks"]["sm_max_mhz"] and not res["clocks"]["reasons"]
             and res["clocks"]["sm_mhz"] < 0.6 * res["clocks"]["sm_max_mhz"])
    remeasured = False
    if bad or stuck:
        res = time_workload(handle, case, sets, steps, warmup, sampler, device)   # re-measure once
        remeasured = True
    timeouts = 0
    if handle.get_last_status() != binding.OK:
        # a bounded on-device wait gave up: the timing is void; measure once more and say so
        timeouts = 1
        res = time_workload(handle, case, sets, steps, warmup, sampler, device)
        if handle.get_last_status() != binding.OK:
            raise RuntimeError(f"{name}: device-side time-out reported twice in a row")
    ms = res["region_ms"] / steps
    avg_launch = res["region_ms"] / max(1, res["launches"])
    out = {"name": name, "case": case, "unit": unit, "ms_per_step": ms, "region_ms": res["region_ms"],
           "timeouts": timeouts,
           "launches": res["launches"], "clocks": res["clocks"], "remeasured": remeasured,
           "variant": binding.variant_name(handle.select_variant(case.M, case.N, case.K, case.dtype)),
           "roofline": roofline(case, name, avg_launch, res["region_ms"] / 1e3, peaks, peak_src)}
    del sets
    torch.cuda.empty_cache()
    if with_e2e:
        e_steps = max(1, min(steps, 20))
        e_ms, h2d, d2h = time_e2e(handle, case, e_steps, 2, device)
        out["e2e_ms"], out["h2d"], out["d2h"], out["e2e_steps"] = e_ms, h2d, d2h, e_steps
    return out


def measure_reductions(handle, device, peaks, peak_src, steps, warmup):
    """The stand-alone K reductions (sum, dot, MSE) over 2^26 fp32 elements: one pass over HBM."""
    n = 1 << 26
    x = torch.from_numpy(synth.uniform(0, 0, n, -1.0, 1.0, synth.F32)).to(device)
    y = torch.from_numpy(synth.uniform(0, 1, n, -1.0, 1.0, synth.F32)).to(device)
    out = torch.empty(1, dtype=torch.float32, device=device)
    stream = torch.cuda.current_stream(device)
    rows = []
    for kind, name, nvec in ((0, "sum", 1), (1, "dot", 2), (2, "mse", 2)):
        for _ in range(warmup):
            handle.reduce_f32(kind, x, y, out=out, stream=stream)
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            handle.reduce_f32(kind, x, y, out=out, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize(device)
        us = e0.elapsed_time(e1) * 1e3 / steps
        nbytes = 4 * n * nvec + 4
        gbs = nbytes / 1e9 / (us * 1e-6)
        rows.append({"kind": name, "n": n, "dtype": "f32", "us_per_step": us, "gbs": gbs,
                     "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                  "frac": gbs / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get(name), "algorithmic_bytes": nbytes,
                                  "peak_source": f"of {peak_src}: copy bandwidth"}})
    return rows


def measure_attention(handle, device, peaks, peak_src, steps, warmup):
    """Multi-head self-attention (bf16, tensor-core kernel) on the two large synthetic workloads:
    d_k = 128 and d_k = 64, 16384 rows, 16 heads.  Flops = 4 N^2 d_model (the two products)."""
    rows = []
    stream = torch.cuda.current_stream(device)
    for name in ("a2", "a3"):
        n, d_model, heads = synth.MHSA_WORKLOADS[name]
        q, k, v = synth.mhsa_inputs(n, d_model, synth.BF16)
        nsets = max(2, math.ceil(4 * L2_BYTES / (8 * n * d_model)))
        sets = []
        for _ in range(nsets):
            Q, K, V = (to_device(x, synth.BF16, (n, d_model), device) for x in (q, k, v))
            sets.append((Q, K, V, torch.empty_like(Q)))
        k_steps = max(5, min(steps, 100))
        for i in range(warmup):
            Q, K, V, Y = sets[i % nsets]
            handle.mhsa(Q, K, V, heads, Y=Y, stream=stream)
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(k_steps):
            Q, K, V, Y = sets[(warmup + i) % nsets]
            handle.mhsa(Q, K, V, heads, Y=Y, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize(device)
        from paper_2602_12305_b200 import binding
        if handle.get_last_status() != binding.OK:
            raise RuntimeError(f"attention {name}: device-side time-out reported")
        us = e0.elapsed_time(e1) * 1e3 / k_steps
        flops = 4.0 * n * n * d_model
        tf = flops / 1e12 / (us * 1e-6)
        rows.append({"workload": f"{name}: bf16 self-attention N={n} d_model={d_model} heads={heads} (d_k={d_model // heads})",
                     "us_per_step": us, "tflops": tf, "steps": k_steps,
                     "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                  "frac": tf / peaks["bf16_tflops"], "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                                  "traffic": NCU_TRAFFIC_BYTES.get(name), "algorithmic_flops": flops,
                                  "algorithmic_bytes": 8 * n * d_model,
                                  "peak_source": f"of {peak_src}: bf16 GEMM burst"}})
        del sets
        torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c2", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-per-shape", action="store_true", help="skip the other four workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    from paper_2602_12305_b200 import binding, build
    rank, local_rank, world = replicas.env_world()
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    if rank == 0:
        build.build_library()
    replicas.init("nccl", device)
    replicas.barrier()
    handle = binding.Handle(local_rank)
    peaks, peak_src = load_peaks()
    sampler = ClockSampler(local_rank)
    sampler.start()

    main_res = measure(handle, args.workload, args, sampler, device, peaks, peak_src, args.steps, args.warmup)
    case, unit = main_res["case"], main_res["unit"]
    region_ms, units = replicas.aggregate(main_res["region_ms"], throughput(case, 1.0, unit) * 1e-3 * args.steps, device)
    value = units / (region_ms / 1e3)          # units are GB or TFLOP done by all ranks
    e2e_ms, e2e_units = replicas.aggregate(main_res["e2e_ms"] * main_res["e2e_steps"],
                                           throughput(case, 1.0, unit) * 1e-3 * main_res["e2e_steps"], device)
    e2e_value = e2e_units / (e2e_ms / 1e3)

    per_shape = []
    if not args.no_per_shape:
        for name in sorted(synth.WORKLOADS):
            if name == args.workload:
                r = main_res
            else:
                # keep each region near a quarter of a second, but never more than --steps
                guess_ms = {"c1": 545792.01, "c2": 0.025, "c3": 121091072.025, "c4": 107639552.12, "c5": 4376021872.8}[name]
                k = max(10, min(args.steps, int(250.0 / guess_ms)))
                r = measure(handle, name, args, sampler, device, peaks, peak_src, k, args.warmup)
            c = r["case"]
            per_shape.append({
                "workload": name, "M": c.M, "N": c.N, "K": c.K, "variant": r["variant"],
                "us_per_step": r["ms_per_step"] * 1e3,
                "tflops": c.flops / 1e12 / (r["ms_per_step"] / 1e3),
                "gbs": c.algorithmic_bytes / 1e9 / (r["ms_per_step"] / 1e3),
                "roofline": r["roofline"], "clocks": r["clocks"],
                "e2e_us": r["e2e_ms"] * 1e3, "gpu_launches": r["launches"],
                "device_timeouts_remeasured": r["timeouts"]})

    reductions = [] if args.no_per_shape else measure_reductions(handle, device, peaks, peak_src, min(args.steps, 200),
                                                                 args.warmup)

    attention = [] if args.no_per_shape else measure_attention(handle, device, peaks, peak_src, args.steps, args.warmup)

    line = {"metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": region_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if case.dtype == synth.F32 else "bf16", "data": "synthetic",
            "config": workload_config(case, args.workload, main_res["variant"]),
            "tflops": case.flops / 1e12 * world / (region_ms / args.steps / 1e3),
            "gbs": case.algorithmic_bytes / 1e9 * world / (region_ms / args.steps / 1e3),
            "roofline": main_res["roofline"], "clocks": main_res["clocks"],
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": main_res["h2d"],
                    "d2h_bytes_per_step": main_res["d2h"], "ms_per_step": e2e_ms / main_res["e2e_steps"],
                    "steps": main_res["e2e_steps"]},
            "gpu_launches": main_res["launches"], "replicas": "independent replicas, no data-path collective",
            "per_shape": per_shape, "reductions": reductions, "attention": attention}
    sampler.stop()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(case, unit)
        for entry in per_shape:
            if entry["workload"] != args.workload:
                c = get_case(entry["workload"])
                entry["cpu_baseline"] = cpu_baseline(c, headline_unit(entry["workload"]))
            else:
                entry["cpu_baseline"] = line["cpu_baseline"]
    handle.destroy()
    replicas.barrier()
    if rank == 0:
        print(json.dumps(line), flush=True)
    replicas.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())

#!/usr/bin/env python
"""Benchmark of Y = act(A.B + bias) on B200 through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]
    python bench.py --crossover            # the dispatcher's M sweep (markdown tables), nothing else

A step is one pass of the whole hot path (dispatch, operand staging, contraction,
split-K reduce where used, fused epilogue, store) over one synthetic problem.  The
headline line is for one workload (default c2, the bf16 GEMV-like shape); the same JSON
line carries a `per_shape` list with all five workloads, the stand-alone reductions,
attention and a few further shapes, and ends with a compact `summary` of all of them.
Inputs are seeded and synthetic.  One JSON line goes to stdout.

Timing.  Headline: W untimed warm-up steps, then exactly K steps between a barrier +
synchronize on both sides, CUDA events on the launching stream, max over ranks.  Every
workload is in addition timed by a fixed protocol that does not depend on --steps: at least
20 warm-up launches, then REGIONS regions of back-to-back launches (one pair of events per
region; at least 200 launches in total for c1-c3, 50 for c4, 20 for c5), from which the
median and the minimum time per call are reported beside the mean.  Tensor-core workloads get
two figures: the short regions (a burst, against the burst bf16 GEMM peak) and one region of
at least two seconds (sustained, under the power cap, against the sustained peak), each with
the SM clock sampled while it ran.  Bandwidth-bound workloads also get the time of an ISOLATED
call (a stream synchronisation between calls, so that no call overlaps its predecessor's
drain).  Consecutive calls use different buffer sets whose total size is several times the L2
cache, so no call finds its operands in L2 from the call before.  SM clocks and throttle
reasons are sampled through NVML while the timed regions run.

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
# FMA-pipe peak: 148 SMs x 128 fp32 lanes x 2 flop x SM clock; 1.965 GHz is the maximum SM clock.
FMA_FLOP_PER_MHZ = 148 * 128 * 2 * 1e6
FMA_PEAK_TFLOPS = FMA_FLOP_PER_MHZ * 1965 / 1e12
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# Timing protocol: launches per workload that do not depend on --steps.
PROTOCOL_WARMUP = 20
PROTOCOL_MIN_LAUNCHES = {"c1": 200, "c2": 200, "c3": 200, "c4": 50, "c5": 20}
REGIONS = 5
REGION_TARGET_MS = 5.0            # a region is at least this long (and at least min launches / REGIONS)
SUSTAINED_SECONDS = 2.0
SINGLE_CALLS = 200


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def load_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel
    of each workload, from the ncu captures summarised under profiles/; a missing or null entry
    means "not captured for the current kernel"."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            return {k: v for k, v in json.load(f)["dram_bytes_per_launch"].items()}
    except Exception:
        return {}


TRAFFIC = load_traffic()


# ---------------------------------------------------------------- clocks (NVML, read-only)

_REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
            0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
            0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
_BAD = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}


class ClockSampler(threading.Thread):
    """Samples SM clock, power and clock-event reasons every few milliseconds."""

    def __init__(self, device_index: int, period_s: float = 0.002):
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


def clocks_rejected(clk) -> bool:
    """A slowdown reason, or clocks stuck far below the maximum with no reason at all."""
    if _BAD.intersection(clk["reasons"]):
        return True
    return bool(clk["sm_mhz"] is not None and clk["sm_max_mhz"] and not clk["reasons"]
                and clk["sm_mhz"] < 0.6 * clk["sm_max_mhz"])


# ---------------------------------------------------------------- device buffers

def to_device(arr, dtype, shape, device):
    if dtype == synth.F32:
        return torch.from_numpy(arr).view(*shape).to(device)
    return torch.from_numpy(arr.view(np.int16)).view(torch.bfloat16).view(*shape).to(device)


def to_pinned(arr, dtype, shape):
    if dtype == synth.F32:
        return torch.from_numpy(arr).view(*shape).pin_memory()
    return torch.from_numpy(arr.view(np.int16)).view(torch.bfloat16).view(*shape).pin_memory()


def make_sets(case, device, cap=1024):
    """Enough distinct (A, B, bias, Y) sets that a round over them moves >= 4 x L2."""
    n = max(2, min(cap, math.ceil(4 * L2_BYTES / case.algorithmic_bytes)))
    tdt = torch.float32 if case.dtype == synth.F32 else torch.bfloat16
    A0 = to_device(case.A, case.dtype, (case.M, case.K), device)
    B0 = to_device(case.B, case.dtype, (case.K, case.N), device)
    b0 = to_device(case.bias, case.dtype, (case.N,), device)
    sets = []
    for i in range(n):
        A, B, b = (A0, B0, b0) if i == 0 else (A0.clone(), B0.clone(), b0.clone())
        sets.append((A, B, b, torch.empty((case.M, case.N), dtype=tdt, device=device)))
    return sets


# ---------------------------------------------------------------- timing primitives

class Timer:
    """Times calls of `step(i)` (which enqueues one launch on `stream`) in three ways."""

    def __init__(self, step, stream, device, sampler):
        self.step, self.stream, self.device, self.sampler = step, stream, device, sampler
        self.i = 0

    def warm(self, n):
        for _ in range(n):
            self.step(self.i)
            self.i += 1
        torch.cuda.synchronize(self.device)

    def region(self, launches, barrier=False, gate=None):
        """`launches` back-to-back calls between two events -> (milliseconds, host t0, host t1).
        (An event after every call would put 3-4 us of idle time between consecutive kernels.)
        With `gate` (a callable that enqueues a short busy kernel) the first event is recorded behind
        that kernel, so the first calls are already queued when the event completes: a region of a
        few launches then holds the launches and nothing of the host's start-up (about 10 us between
        an event record and the first launch reaching an idle GPU from Python)."""
        torch.cuda.synchronize(self.device)
        if barrier:
            replicas.barrier()
            torch.cuda.synchronize(self.device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        if gate is not None:
            gate()
        e0.record(self.stream)
        for _ in range(launches):
            self.step(self.i)
            self.i += 1
        e1.record(self.stream)
        torch.cuda.synchronize(self.device)
        t1 = time.perf_counter()
        if barrier:
            replicas.barrier()
            torch.cuda.synchronize(self.device)
        return e0.elapsed_time(e1), t0, t1

    def isolated(self, calls, gate=None):
        """One pair of events around every call, the stream synchronised between calls: no call
        overlaps the drain of the one before -> list of microseconds.  With `gate` (a callable that
        enqueues a short busy kernel on the stream) the event records and the call are enqueued while
        the GPU is still busy with the gate, so the time between the events holds no host latency:
        what remains is the call alone, from an idle, drained GPU."""
        out = []
        for _ in range(calls):
            torch.cuda.synchronize(self.device)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if gate is not None:
                gate()
            e0.record(self.stream)
            self.step(self.i)
            self.i += 1
            e1.record(self.stream)
            e1.synchronize()
            out.append(e0.elapsed_time(e1) * 1e3)
        return out

    def clocks(self, t0, t1, min_samples=3):
        """Clock summary of the host-time window; when it is too short for the sampling period the
        same load is continued (untimed) for a quarter of a second and sampled."""
        sm = self.sampler
        if sm is None or not sm.ok:
            return summarise_clocks([], sm.max_mhz if sm else None, "unavailable")
        win = sm.window(t0, t1)
        how = "during the timed region"
        if len(win) < min_samples:
            t2 = time.perf_counter()
            n = 0
            while time.perf_counter() - t2 < 0.25:
                self.step(self.i)
                self.i += 1
                n += 1
                if n % 64 == 0:
                    torch.cuda.synchronize(self.device)
            torch.cuda.synchronize(self.device)
            win = sm.window(t2 + 0.05, time.perf_counter())
            how = "same load continued after the timed region (region shorter than the sampling period)"
        return summarise_clocks(win, sm.max_mhz, how)


_GATE = {}


def make_gate(device):
    """A callable that enqueues a busy kernel of about 60 us on the current stream (the library's
    bounded-wait self-test on a handle of its own, whose status word nobody else reads)."""
    from paper_2602_12305_b200 import binding
    key = str(device)
    if key not in _GATE:
        _GATE[key] = binding.Handle(device.index if device.index is not None else 0)
    gh = _GATE[key]
    return lambda: gh.selftest_timeout(120000)


def close_gates():
    for gh in _GATE.values():
        gh.get_last_status()          # clears the recorded time-outs
        gh.destroy()
    _GATE.clear()


def protocol(timer, min_launches, est_ms):
    """The fixed protocol: warm-up, then REGIONS regions; per-call statistics in microseconds."""
    timer.warm(PROTOCOL_WARMUP)
    per_region = max(math.ceil(min_launches / REGIONS), math.ceil(REGION_TARGET_MS / max(est_ms, 1e-4)), 1)
    per_region = min(per_region, 2000)
    times, t_first, t_last = [], None, None
    for _ in range(REGIONS):
        ms, t0, t1 = timer.region(per_region)
        times.append(ms * 1e3 / per_region)
        t_first = t0 if t_first is None else t_first
        t_last = t1
    return {"median": statistics.median(times), "min": min(times), "mean": statistics.fmean(times),
            "max": max(times), "regions": REGIONS, "launches_per_region": per_region,
            "launches": REGIONS * per_region}, t_first, t_last


def sustained(timer, us_per_call):
    """One region of at least SUSTAINED_SECONDS of back-to-back launches."""
    launches = max(20, math.ceil(SUSTAINED_SECONDS * 1e6 / us_per_call * 1.05))
    ms, t0, t1 = timer.region(launches)
    clk = summarise_clocks(timer.sampler.window(t0 + 0.2, t1) if timer.sampler else [],
                           timer.sampler.max_mhz if timer.sampler else None, "during the sustained region, after its first 0.2 s")
    return {"us_per_call": ms * 1e3 / launches, "launches": launches, "region_s": ms / 1e3, "clocks": clk}


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


def estimate_ms(case, bound, peaks):
    """Rough time of one call from the roofline (used only to size the timed regions)."""
    t_mem = case.algorithmic_bytes / (peaks["hbm_gbs"] * 1e9)
    peak_tf = FMA_PEAK_TFLOPS if case.dtype == synth.F32 else peaks["bf16_tflops"]
    t_math = case.flops / (peak_tf * 1e12)
    return (max(t_mem, t_math) / 0.7 + 4e-6) * 1e3


def roofline(case, name, bound, us, peaks, peak_src, sustained_region=False, sm_mhz=None):
    """Roofline object for a call that took `us` microseconds."""
    s = us * 1e-6
    if bound == "hbm":
        ach, peak, unit, kind = case.algorithmic_bytes / 1e9 / s, peaks["hbm_gbs"], "GB/s", "copy bandwidth"
    elif bound == "tensor":
        peak = peaks["bf16_tflops_sustained"] if sustained_region else peaks["bf16_tflops"]
        ach, unit, kind = case.flops / 1e12 / s, "TFLOP/s", "bf16 GEMM " + ("sustained" if sustained_region else "burst")
    else:
        ach, peak, unit, kind = case.flops / 1e12 / s, FMA_PEAK_TFLOPS, "TFLOP/s", "fp32 FMA pipes at max clock (derived)"
    src = peak_src if bound != "alu" else "derived"
    out = {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
           "traffic": TRAFFIC.get(name), "peak_source": f"of {src}: {kind}",
           "algorithmic_bytes": case.algorithmic_bytes, "algorithmic_flops": case.flops, "avg_launch_ms": us / 1e3}
    if bound == "alu" and sm_mhz:
        # the FMA pipes' peak at the clock the kernel actually ran at
        out["frac_at_sampled_clock"] = ach / (FMA_FLOP_PER_MHZ * sm_mhz / 1e12)
    return out


# ---------------------------------------------------------------- one GEMM workload

def gemm_timer(handle, case, sets, device, sampler):
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

    return Timer(step, stream, device, sampler)


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


def measure_once(handle, name, case, bound, args, sampler, device, peaks, peak_src, contract_steps, quick):
    from paper_2602_12305_b200 import binding
    sets = make_sets(case, device)
    timer = gemm_timer(handle, case, sets, device, sampler)
    launches0 = handle.launch_count()
    out = {"name": name, "case": case, "bound": bound,
           "variant": binding.variant_name(handle.select_variant(case.M, case.N, case.K, case.dtype))}
    if contract_steps:
        # the headline region: W warm-up steps, exactly K steps, barrier + synchronize on both sides
        timer.warm(args.warmup)
        ms_host, _, _ = timer.region(contract_steps, barrier=True)
        ms, t0, t1 = timer.region(contract_steps, barrier=True, gate=make_gate(device))
        out["contract_ms"], out["contract_steps"] = ms, contract_steps
        out["contract_ms_host_started"] = ms_host
        out["contract_clocks"] = timer.clocks(t0, t1)
    min_l = PROTOCOL_MIN_LAUNCHES.get(name, 20)
    stats, t0, t1 = protocol(timer, min_l if not quick else min(min_l, 20), estimate_ms(case, bound, peaks))
    out["per_call_us"] = stats
    out["clocks"] = timer.clocks(t0, t1)
    if bound == "tensor" and not quick:
        out["sustained"] = sustained(timer, stats["median"])
    if bound != "tensor" and not quick:
        iso = timer.isolated(SINGLE_CALLS, gate=make_gate(device))
        host = timer.isolated(SINGLE_CALLS)
        out["single_call_us"] = {"median": statistics.median(iso), "min": min(iso), "calls": len(iso),
                                 "how": "one call between two events on a drained GPU; a short busy kernel ahead of the "
                                        "first event hides the host's enqueue latency",
                                 "with_host_latency_median": statistics.median(host)}
    out["launches"] = handle.launch_count() - launches0
    del sets, timer
    torch.cuda.empty_cache()
    return out


def measure(handle, name, case, bound, args, sampler, device, peaks, peak_src, contract_steps=0, with_e2e=True,
            quick=False):
    """All timings of one GEMM workload; re-measured once after rejected clocks or a device time-out."""
    from paper_2602_12305_b200 import binding
    res = measure_once(handle, name, case, bound, args, sampler, device, peaks, peak_src, contract_steps, quick)
    remeasured, timeouts = False, 0
    # (every rank takes the same decision: the contract region holds barriers)
    if replicas.any_rank(clocks_rejected(res["clocks"]) or bool(contract_steps and clocks_rejected(res["contract_clocks"])),
                         device):
        res = measure_once(handle, name, case, bound, args, sampler, device, peaks, peak_src, contract_steps, quick)
        remeasured = True
    if replicas.any_rank(handle.get_last_status() != binding.OK, device):
        # a bounded on-device wait gave up: the timing is void; measure once more and say so
        timeouts = 1
        res = measure_once(handle, name, case, bound, args, sampler, device, peaks, peak_src, contract_steps, quick)
        if handle.get_last_status() != binding.OK:
            raise RuntimeError(f"{name}: device-side time-out reported twice in a row")
    res["remeasured"], res["timeouts"] = remeasured, timeouts
    pc = res["per_call_us"]
    res["roofline"] = roofline(case, name, bound, pc["mean"], peaks, peak_src, sm_mhz=res["clocks"]["sm_mhz"])
    res["roofline"]["frac_median"] = res["roofline"]["frac"] * pc["mean"] / pc["median"]
    res["roofline"]["frac_best"] = res["roofline"]["frac"] * pc["mean"] / pc["min"]
    if bound == "tensor":
        res["roofline"]["peak_source"] += " (regions of a few milliseconds)"
        mhz = res["clocks"]["sm_mhz"]
        res["roofline"]["burst"] = {"us_per_call": pc["min"], "frac": res["roofline"]["frac_best"], "sm_mhz": mhz,
                                    "us_x_mhz": pc["min"] * mhz if mhz else None}
        if "sustained" in res:
            s = res["sustained"]
            r = roofline(case, name, bound, s["us_per_call"], peaks, peak_src, sustained_region=True)
            mhz = s["clocks"]["sm_mhz"]
            res["roofline"]["sustained"] = {"us_per_call": s["us_per_call"], "achieved": r["achieved"], "peak": r["peak"],
                                            "frac": r["frac"], "launches": s["launches"], "region_s": s["region_s"],
                                            "sm_mhz": mhz, "us_x_mhz": s["us_per_call"] * mhz if mhz else None,
                                            "reasons": s["clocks"]["reasons"], "peak_source": r["peak_source"]}
    if "single_call_us" in res and bound == "hbm":
        sc = res["single_call_us"]
        sc["gbs"] = case.algorithmic_bytes / 1e3 / sc["median"]
        sc["frac"] = sc["gbs"] / peaks["hbm_gbs"]
    if with_e2e:
        e_steps = max(1, min(args.steps, 20))
        e_ms, h2d, d2h = time_e2e(handle, case, e_steps, 2, device)
        res["e2e_ms"], res["h2d"], res["d2h"], res["e2e_steps"] = e_ms, h2d, d2h, e_steps
    return res


def isolated_floor_us(handle, device, sampler):
    """What the isolated-call protocol measures for a kernel that does next to nothing (a 4-element
    sum through the same C ABI): launch latency plus the two event records, the part of every
    `single_call_us` figure that is not the kernel's own work."""
    x = torch.ones(4, dtype=torch.float32, device=device)
    out = torch.empty(1, dtype=torch.float32, device=device)
    stream = torch.cuda.current_stream(device)
    timer = Timer(lambda i: handle.reduce_f32(0, x, None, out=out, stream=stream), stream, device, sampler)
    timer.warm(10)
    iso = timer.isolated(SINGLE_CALLS, gate=make_gate(device))
    host = timer.isolated(SINGLE_CALLS)
    return {"median": statistics.median(iso), "min": min(iso), "calls": len(iso),
            "with_host_latency_median": statistics.median(host),
            "what": "isolated call of a 4-element sum: kernel start-up + event records"}


def shape_entry(r):
    c, pc = r["case"], r["per_call_us"]
    e = {"workload": r["name"], "M": c.M, "N": c.N, "K": c.K, "variant": r["variant"],
         "us_per_step": pc["mean"], "per_call_us": pc,
         "tflops": c.flops / 1e6 / pc["mean"], "gbs": c.algorithmic_bytes / 1e3 / pc["mean"],
         "roofline": r["roofline"], "clocks": r["clocks"], "gpu_launches": r["launches"],
         "clocks_remeasured": r["remeasured"], "device_timeouts_remeasured": r["timeouts"]}
    if "single_call_us" in r:
        e["single_call_us"] = r["single_call_us"]
    if "e2e_ms" in r:
        e["e2e_us"] = r["e2e_ms"] * 1e3
    return e


# ---------------------------------------------------------------- further rows

# fp32 beyond c1 on the FMA tiles, and shapes whose N is not a multiple of the vector width
EXTRA_SHAPES = [
    ("f32_4096", "c1", dict(M=4096, N=4096, K=4096), "alu"),
    ("f32_1024x8192x1024", "c1", dict(M=1024, N=8192, K=1024), "alu"),
    ("bf16_4096x4100x4096_unaligned_n", "c4", dict(M=4096, N=4100, K=4096), "tensor"),
    ("f32_1024x1026x1024_unaligned_n", "c1", dict(M=1024, N=1026, K=1024), "alu"),
]


def measure_extras(handle, args, sampler, device, peaks, peak_src):
    rows = []
    for name, base, kw, bound in EXTRA_SHAPES:
        case = synth.make_case(base, **kw)
        r = measure(handle, name, case, bound, args, sampler, device, peaks, peak_src, with_e2e=False, quick=True)
        rows.append(shape_entry(r))
    return rows


def measure_reductions(handle, device, sampler, peaks, peak_src, quick):
    """The stand-alone K reductions (sum, dot, MSE) over 2^26 fp32 elements: one pass over HBM."""
    n = 1 << 26
    nsets = 3                                        # 3 x 512 MiB: every call finds L2 cold
    xs = [torch.from_numpy(synth.uniform(0, 0, n, -1.0, 1.0, synth.F32)).to(device)]
    ys = [torch.from_numpy(synth.uniform(0, 1, n, -1.0, 1.0, synth.F32)).to(device)]
    for _ in range(nsets - 1):
        xs.append(xs[0].clone())
        ys.append(ys[0].clone())
    out = torch.empty(1, dtype=torch.float32, device=device)
    stream = torch.cuda.current_stream(device)
    rows = []
    for kind, name, nvec in ((0, "sum", 1), (1, "dot", 2), (2, "mse", 2)):
        def step(i, kind=kind):
            handle.reduce_f32(kind, xs[i % nsets], ys[i % nsets], out=out, stream=stream)
        timer = Timer(step, stream, device, sampler)
        nbytes = 4 * n * nvec + 4
        stats, _, _ = protocol(timer, 20 if quick else 200, nbytes / (peaks["hbm_gbs"] * 1e6))
        gbs = nbytes / 1e3 / stats["mean"]
        row = {"kind": name, "n": n, "dtype": "f32", "us_per_step": stats["mean"], "per_call_us": stats, "gbs": gbs,
               "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": gbs / peaks["hbm_gbs"], "traffic": TRAFFIC.get(name), "algorithmic_bytes": nbytes,
                            "peak_source": f"of {peak_src}: copy bandwidth"}}
        if not quick:
            iso = timer.isolated(SINGLE_CALLS, gate=make_gate(device))
            row["single_call_us"] = {"median": statistics.median(iso), "min": min(iso), "calls": len(iso),
                                     "gbs": nbytes / 1e3 / statistics.median(iso),
                                     "frac": nbytes / 1e3 / statistics.median(iso) / peaks["hbm_gbs"]}
        rows.append(row)
    return rows


def measure_attention(handle, device, sampler, peaks, peak_src, quick):
    """Multi-head self-attention (bf16, tensor-core kernel) on the two large synthetic workloads:
    d_k = 128 and d_k = 64, 16384 rows, 16 heads.  Flops = 4 N^2 d_model (the two products)."""
    from paper_2602_12305_b200 import binding
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

        def step(i, sets=sets, heads=heads):
            Q, K, V, Y = sets[i % len(sets)]
            handle.mhsa(Q, K, V, heads, Y=Y, stream=stream)

        timer = Timer(step, stream, device, sampler)
        flops = 4.0 * n * n * d_model
        stats, t0, t1 = protocol(timer, 20, flops / (peaks["bf16_tflops"] * 1e9))
        clk = timer.clocks(t0, t1)
        tf = flops / 1e6 / stats["mean"]
        rl = {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
              "frac": tf / peaks["bf16_tflops"], "traffic": TRAFFIC.get(name), "algorithmic_flops": flops,
              "algorithmic_bytes": 8 * n * d_model, "peak_source": f"of {peak_src}: bf16 GEMM burst (regions of a few milliseconds)",
              "burst": {"us_per_call": stats["min"], "frac": flops / 1e6 / stats["min"] / peaks["bf16_tflops"],
                        "sm_mhz": clk["sm_mhz"], "us_x_mhz": stats["min"] * clk["sm_mhz"] if clk["sm_mhz"] else None}}
        if not quick:
            s = sustained(timer, stats["median"])
            stf = flops / 1e6 / s["us_per_call"]
            mhz = s["clocks"]["sm_mhz"]
            rl["sustained"] = {"us_per_call": s["us_per_call"], "achieved": stf, "peak": peaks["bf16_tflops_sustained"],
                               "frac": stf / peaks["bf16_tflops_sustained"], "launches": s["launches"],
                               "region_s": s["region_s"], "sm_mhz": mhz, "us_x_mhz": s["us_per_call"] * mhz if mhz else None,
                               "reasons": s["clocks"]["reasons"], "peak_source": f"of {peak_src}: bf16 GEMM sustained"}
        if handle.get_last_status() != binding.OK:
            raise RuntimeError(f"attention {name}: device-side time-out reported")
        rows.append({"workload": f"{name}: bf16 self-attention N={n} d_model={d_model} heads={heads} (d_k={d_model // heads})",
                     "name": name, "us_per_step": stats["mean"], "per_call_us": stats, "tflops": tf, "clocks": clk,
                     "roofline": rl})
        del sets, timer
        torch.cuda.empty_cache()
    return rows


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
                       f"bias + {['none', 'ReLU', 'GELU(tanh)', 'sigmoid'][case.act]}",
           "arithmetic": "fp32 products and sums on the FMA pipes" if case.dtype == synth.F32
                         else "exact bf16 products, fp32 accumulation, one rounding to bf16 at the store",
           "M": case.M, "N": case.N, "K": case.K,
           "l2": "consecutive steps use different buffer sets; one round over the sets moves >= 4 x L2"}
    if variant is not None:
        cfg["variant"] = variant
    return cfg


# ---------------------------------------------------------------- the dispatcher's crossover table

CROSSOVER_VARIANTS = ["gemv_splitk_stream", "skinny_streamk_tcgen05", "persistent_tcgen05", "persistent_tcgen05_cta_pair",
                      "cluster_splitk_tcgen05_cta_pair"]


def run_crossover(args):
    """Time every variant that can run a shape over a sweep of M at two (N, K): markdown tables with
    the dispatcher's pick and its fraction of the bounding roofline, max(bytes / HBM peak, flops /
    bf16 burst peak)."""
    from paper_2602_12305_b200 import binding, build
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    build.build_library()
    peaks, peak_src = load_peaks()
    h = binding.Handle(0)
    ids = {binding.variant_name(v): v for v in range(binding.VARIANT_COUNT)}
    act = synth.ACT_RELU
    print(f"Peaks ({peak_src}): HBM {peaks['hbm_gbs']:.0f} GB/s, bf16 burst {peaks['bf16_tflops']:.0f} TFLOP/s.  "
          f"Median of {REGIONS} regions of back-to-back launches between two CUDA events, buffer sets rotating (> 4 x L2).\n")
    for N, K in ((8192, 8192), (14336, 4096)):
        print(f"N = {N}, K = {K}, bf16, bias + ReLU; microseconds per launch\n")
        print("| M | " + " | ".join(CROSSOVER_VARIANTS) + " | dispatcher picks | us | roofline floor us (HBM / tensor) | fraction of the bounding roofline |")
        print("|---|" + "---|" * (len(CROSSOVER_VARIANTS) + 4))
        for M in [int(x) for x in args.crossover_ms.split(",")]:
            c = synth.make_case("c3", M=M, N=N, K=K, act=act)
            sets = make_sets(c, device, cap=8)
            timer = gemm_timer(h, c, sets, device, None)
            h.force_variant(binding.VARIANT_AUTO)
            pick = binding.variant_name(h.select_variant(M, N, K, binding.BF16))
            cells, t_pick = [], float("nan")
            est = estimate_ms(c, "tensor", peaks)
            for vn in CROSSOVER_VARIANTS:
                if vn == "gemv_splitk_stream" and M > 4:
                    cells.append("—")
                    continue
                h.force_variant(ids[vn])
                try:
                    timer.warm(5)
                except RuntimeError:          # the variant cannot run this shape
                    cells.append("—")
                    continue
                per = max(20, math.ceil(2.0 / est))
                t = statistics.median(timer.region(per)[0] * 1e3 / per for _ in range(REGIONS))
                if h.get_last_status() != binding.OK:
                    cells.append("TIMEOUT")
                    continue
                cells.append(f"{t:.1f}")
                if vn == pick:
                    t_pick = t
            t_hbm = c.algorithmic_bytes / (peaks["hbm_gbs"] * 1e3)
            t_tc = c.flops / (peaks["bf16_tflops"] * 1e6)
            print(f"| {M} | " + " | ".join(cells) + f" | {pick} | {t_pick:.1f} | {t_hbm:.1f} / {t_tc:.1f} | "
                  f"{max(t_hbm, t_tc) / t_pick:.2f} |", flush=True)
            del sets, timer
            torch.cuda.empty_cache()
        print()
    h.destroy()
    return 0


# ---------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c2", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-per-shape", action="store_true", help="headline workload only")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true",
                    help="few launches per workload and no sustained / isolated legs (for a profiler's launch list)")
    ap.add_argument("--crossover", action="store_true", help="print the dispatcher's M-sweep tables and exit")
    ap.add_argument("--crossover-ms", default="1,2,4,8,16,32,64,96,128,192,256,384,512,1024")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if args.crossover:
        return run_crossover(args)
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
    others = world == 1 and not args.no_per_shape     # the further rows are single-GPU information

    name = args.workload
    main_res = measure(handle, name, get_case(name), BOUND[name], args, sampler, device, peaks, peak_src,
                       contract_steps=args.steps, quick=args.quick)
    case, unit = main_res["case"], headline_unit(name)
    region_ms, units = replicas.aggregate(main_res["contract_ms"], throughput(case, 1.0, unit) * 1e-3 * args.steps, device)
    value = units / (region_ms / 1e3)          # units are GB or TFLOP done by all ranks
    e2e_ms, e2e_units = replicas.aggregate(main_res["e2e_ms"] * main_res["e2e_steps"],
                                           throughput(case, 1.0, unit) * 1e-3 * main_res["e2e_steps"], device)
    e2e_value = e2e_units / (e2e_ms / 1e3)
    # the headline roofline object is that of the contract region (K steps)
    head_rl = roofline(case, name, BOUND[name], main_res["contract_ms"] * 1e3 / args.steps, peaks, peak_src)
    head_rl["launches_timed"] = args.steps

    per_shape, reductions, attention, extras = [], [], [], []
    if others:
        for other in sorted(synth.WORKLOADS):
            r = main_res if other == name else measure(handle, other, get_case(other), BOUND[other], args, sampler,
                                                       device, peaks, peak_src, quick=args.quick)
            per_shape.append(shape_entry(r))
        reductions = measure_reductions(handle, device, sampler, peaks, peak_src, args.quick)
        attention = measure_attention(handle, device, sampler, peaks, peak_src, args.quick)
        extras = measure_extras(handle, args, sampler, device, peaks, peak_src)
    else:
        per_shape.append(shape_entry(main_res))

    line = {"metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": region_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if case.dtype == synth.F32 else "bf16", "data": "synthetic",
            "config": workload_config(case, name, None), "variant": main_res["variant"],
            "tflops": case.flops / 1e12 * world / (region_ms / args.steps / 1e3),
            "gbs": case.algorithmic_bytes / 1e9 * world / (region_ms / args.steps / 1e3),
            "roofline": head_rl, "clocks": main_res["contract_clocks"],
            "per_call_us": main_res["per_call_us"],
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": main_res["h2d"],
                    "d2h_bytes_per_step": main_res["d2h"], "ms_per_step": e2e_ms / main_res["e2e_steps"],
                    "steps": main_res["e2e_steps"]},
            "gpu_launches": args.steps, "gpu_launches_all_legs": main_res["launches"],
            "replicas": "independent replicas, no data-path collective",
            "per_shape": per_shape, "reductions": reductions, "attention": attention, "extra_shapes": extras}
    line["timed_region"] = {
        "how": "W warm-up steps, barrier + synchronize, a busy kernel of about 60 us, start event, exactly K steps, end "
               "event, synchronize + barrier: the K launches are queued behind the busy kernel when the start event "
               "completes, so the region holds the K steps and none of the host's start-up",
        "ms_per_step_host_started": main_res["contract_ms_host_started"] / args.steps,
        "host_started": "the same K steps with the start event recorded on an idle GPU, i.e. including the time the "
                        "host needs to get the first launch there (this rank's figure)"}
    if "single_call_us" in main_res:
        line["single_call_us"] = main_res["single_call_us"]
        line["single_call_floor_us"] = isolated_floor_us(handle, device, sampler)
    sampler.stop()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(case, unit)
        for entry in per_shape:
            if entry["workload"] != name:
                entry["cpu_baseline"] = cpu_baseline(get_case(entry["workload"]), headline_unit(entry["workload"]))
            else:
                entry["cpu_baseline"] = line["cpu_baseline"]
    # last key: every row in a few numbers -- [name, microseconds per call (mean of the protocol's
    # regions), fraction of its roofline, launches timed]; tensor-bound rows add the sustained figure
    summary = []
    for e in per_shape + extras:
        row = [e["workload"], round(e["us_per_step"], 2), round(e["roofline"]["frac"], 3), e["per_call_us"]["launches"]]
        if "sustained" in e["roofline"]:
            s = e["roofline"]["sustained"]
            row += ["sustained", round(s["us_per_call"], 1), round(s["frac"], 3), s["launches"]]
        if "single_call_us" in e and "frac" in e["single_call_us"]:
            row += ["isolated", round(e["single_call_us"]["median"], 2), round(e["single_call_us"]["frac"], 3)]
        summary.append(row)
    for e in reductions:
        summary.append([e["kind"], round(e["us_per_step"], 2), round(e["roofline"]["frac"], 3), e["per_call_us"]["launches"]])
    for e in attention:
        row = [e["name"], round(e["us_per_step"], 1), round(e["roofline"]["frac"], 3), e["per_call_us"]["launches"]]
        if "sustained" in e["roofline"]:
            s = e["roofline"]["sustained"]
            row += ["sustained", round(s["us_per_call"], 1), round(s["frac"], 3), s["launches"]]
        summary.append(row)
    line["summary"] = summary
    close_gates()
    handle.destroy()
    replicas.barrier()
    if rank == 0:
        print(json.dumps(line), flush=True)
    replicas.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())

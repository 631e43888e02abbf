"""Run one named workload a few times through the C ABI -- the command line used for
profiling (ncu) and for quick timing of a forced variant.

    python -m paper_2602_12305_b200.run_case --workload c3 [--variant auto|0..5] [--iters 3]
        [--M m --N n --K k] [--sets 2] [--time]
    python -m paper_2602_12305_b200.run_case --reduce sum|dot|mse [--n 67108864] [--iters 3]
    python -m paper_2602_12305_b200.run_case --mhsa a1|a2|a3 [--N n --K d_model --heads h] [--iters 3]

Each iteration uses the next of `--sets` distinct buffer sets.  With --time, CUDA-event
times per launch are printed (median / min) with the implied TFLOP/s and GB/s.
"""
from __future__ import annotations

import argparse
import statistics

import numpy as np
import torch

from . import binding, synth


def _dev(arr, dtype, shape):
    if dtype == synth.F32:
        return torch.from_numpy(arr).view(*shape).cuda()
    return torch.from_numpy(arr.view(np.int16)).view(torch.bfloat16).view(*shape).cuda()


def run_reduce(a):
    kind = {"sum": binding.REDUCE_SUM, "dot": binding.REDUCE_DOT, "mse": binding.REDUCE_MSE}[a.reduce]
    h = binding.Handle(0)
    x = torch.from_numpy(synth.uniform(0, 0, a.n, -1.0, 1.0, synth.F32)).cuda()
    y = torch.from_numpy(synth.uniform(0, 1, a.n, -1.0, 1.0, synth.F32)).cuda()
    out = torch.empty(1, dtype=torch.float32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(a.warmup):
        h.reduce_f32(kind, x, y, out=out)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(a.iters):
        h.reduce_f32(kind, x, y, out=out)
    e1.record()
    torch.cuda.synchronize()
    status = h.get_last_status()
    us = e0.elapsed_time(e1) * 1e3 / a.iters
    nbytes = 4 * a.n * (1 if a.reduce == "sum" else 2) + 4
    print(f"reduce {a.reduce} n={a.n}: {a.iters} launches, result {out.item():.9g}, status {binding.status_string(status)}, "
          f"{us:.2f} us per launch, {nbytes / 1e3 / us:.0f} GB/s")
    h.destroy()
    return 0 if status == binding.OK else 1


def run_mhsa(a):
    n, d_model, heads = synth.MHSA_WORKLOADS[a.mhsa]
    n, d_model, heads = a.N or n, a.K or d_model, a.heads or heads
    h = binding.Handle(0)
    if a.variant != "auto":
        h.force_variant(int(a.variant))
    q, k, v = synth.mhsa_inputs(n, d_model, synth.BF16)
    sets = []
    for _ in range(a.sets):
        Q, K, V = (_dev(x, synth.BF16, (n, d_model)) for x in (q, k, v))
        sets.append((Q, K, V, torch.empty_like(Q)))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(a.warmup):
        Q, K, V, Y = sets[i % len(sets)]
        h.mhsa(Q, K, V, heads, Y=Y)
    torch.cuda.synchronize()
    e0.record()
    for i in range(a.iters):
        Q, K, V, Y = sets[(a.warmup + i) % len(sets)]
        h.mhsa(Q, K, V, heads, Y=Y)
    e1.record()
    torch.cuda.synchronize()
    status = h.get_last_status()
    us = e0.elapsed_time(e1) * 1e3 / a.iters
    flops = 4 * n * n * d_model
    print(f"mhsa {a.mhsa} N={n} d_model={d_model} heads={heads}: {a.iters} launches, status {binding.status_string(status)}, "
          f"{us:.1f} us per launch, {flops / 1e6 / us:.1f} TFLOP/s")
    h.destroy()
    return 0 if status == binding.OK else 1


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--variant", default="auto")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--sets", type=int, default=2)
    ap.add_argument("--M", type=int)
    ap.add_argument("--N", type=int)
    ap.add_argument("--K", type=int)
    ap.add_argument("--time", action="store_true")
    ap.add_argument("--no-step-events", action="store_true", help="one event pair around all launches only")
    ap.add_argument("--reduce", choices=["sum", "dot", "mse"], help="run the stand-alone reduction instead")
    ap.add_argument("--n", type=int, default=1 << 26, help="vector length for --reduce")
    ap.add_argument("--mhsa", choices=sorted(synth.MHSA_WORKLOADS), help="run multi-head self-attention instead")
    ap.add_argument("--heads", type=int, help="with --mhsa: override the head count (and --N, --K = d_model)")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="optiml_set_option before the run, e.g. gemv_prefetch_rows=48, skinny_stage_rows=128, "
                         "skinny_ring_stages=3, skinny_prefetch_early=2, skinny_late_trigger=0, pair_split_max=1")
    a = ap.parse_args()
    if a.reduce:
        return run_reduce(a)
    if a.mhsa:
        return run_mhsa(a)

    c = synth.make_case(a.workload, M=a.M, N=a.N, K=a.K)
    h = binding.Handle(0)
    if a.variant != "auto":
        h.force_variant(int(a.variant))
    for item in a.option:
        name, value = item.split("=")
        h.set_option(getattr(binding, "OPT_" + name.upper()), int(value))
    tdt = torch.float32 if c.dtype == synth.F32 else torch.bfloat16
    A0, B0, b0 = _dev(c.A, c.dtype, (c.M, c.K)), _dev(c.B, c.dtype, (c.K, c.N)), _dev(c.bias, c.dtype, (c.N,))
    sets = [(A0, B0, b0, torch.empty((c.M, c.N), dtype=tdt, device="cuda"))]
    for _ in range(a.sets - 1):
        sets.append((A0.clone(), B0.clone(), b0.clone(), torch.empty((c.M, c.N), dtype=tdt, device="cuda")))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(a.iters + 1)]
    for i in range(a.warmup):
        A, B, b, Y = sets[i % len(sets)]
        h.gemm_epilogue(A, B, b, c.act, Y=Y)
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(a.iters):
        A, B, b, Y = sets[(a.warmup + i) % len(sets)]
        h.gemm_epilogue(A, B, b, c.act, Y=Y)
        if not a.no_step_events or i == a.iters - 1:
            ev[i + 1].record()
    torch.cuda.synchronize()
    status = h.get_last_status()
    name = binding.variant_name(h.select_variant(c.M, c.N, c.K, c.dtype))
    print(f"{a.workload} {c.M}x{c.N}x{c.K} via {name}: {a.iters} launches, status {binding.status_string(status)}")
    if a.time and a.no_step_events:
        mean = ev[0].elapsed_time(ev[a.iters]) / a.iters
        print(f"  us per launch: mean {mean * 1e3:.2f} (no per-step events)   "
              f"TFLOP/s {c.flops / 1e12 / (mean / 1e3):.1f}   GB/s {c.algorithmic_bytes / 1e9 / (mean / 1e3):.0f}")
    elif a.time:
        ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(a.iters)]
        # single event intervals are quantised by the timer; the mean over the region is not
        med, mn, mean = statistics.median(ms), min(ms), ev[0].elapsed_time(ev[a.iters]) / a.iters
        print(f"  us per launch: mean {mean * 1e3:.2f}  median {med * 1e3:.2f}  min {mn * 1e3:.2f}   "
              f"TFLOP/s {c.flops / 1e12 / (mean / 1e3):.1f}   GB/s {c.algorithmic_bytes / 1e9 / (mean / 1e3):.0f}")
    h.destroy()
    return 0 if status == binding.OK else 1


if __name__ == "__main__":
    raise SystemExit(main())

"""Time every kernel variant that can run a shape, over a sweep of M at fixed (N, K): the
evidence behind the dispatcher's thresholds.

    python -m paper_2602_12305_b200.sweep [--N 8192 --K 8192] [--Ms 1,2,4,...] [--iters 100]

Prints one markdown table row per M: microseconds per launch of each variant (mean over
`--iters` back-to-back launches between two CUDA events, rotating over buffer sets larger
than L2 together) and the variant the dispatcher picks.
"""
from __future__ import annotations

import argparse
import math

import numpy as np
import torch

from . import binding, synth

VARIANTS = [(binding.VARIANT_GEMV_SPLITK, "gemv"), (binding.VARIANT_SKINNY_UMMA, "skinny"),
            (binding.VARIANT_UMMA, "umma"), (binding.VARIANT_UMMA_2CTA, "umma_pair")]


def _dev(bits, shape):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).view(*shape).cuda()


def time_variant(h, variant, sets, M, N, K, act, iters):
    h.force_variant(variant)
    st = torch.cuda.current_stream().cuda_stream
    raw = [(A.data_ptr(), B.data_ptr(), b.data_ptr(), Y.data_ptr()) for A, B, b, Y in sets]

    def call(i):
        pa, pb, pbias, py = raw[i % len(raw)]
        return h.gemm_epilogue_raw(pa, pb, pbias, py, M, N, K, binding.BF16, act, st)

    if call(0) != binding.OK:          # variant cannot run this shape
        return None
    for i in range(1, 4):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        call(i)
    e1.record()
    torch.cuda.synchronize()
    if h.get_last_status() != binding.OK:
        return float("nan")            # a bounded on-device wait gave up (OPTIML_LOG=1 says where)
    return e0.elapsed_time(e1) * 1e3 / iters


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--N", type=int, default=8192)
    ap.add_argument("--K", type=int, default=8192)
    ap.add_argument("--Ms", default="1,2,4,8,16,32,64,96,128,192,256,512,1024")
    ap.add_argument("--iters", type=int, default=100)
    a = ap.parse_args()
    h = binding.Handle(0)
    act = synth.ACT_RELU
    print(f"N = {a.N}, K = {a.K}, bf16, bias + ReLU; microseconds per launch\n")
    print("| M | " + " | ".join(n for _, n in VARIANTS) + " | dispatcher picks | GB/s of the pick | TFLOP/s of the pick |")
    print("|---|" + "---|" * (len(VARIANTS) + 3))
    for M in [int(x) for x in a.Ms.split(",")]:
        c = synth.make_case("c3", M=M, N=a.N, K=a.K, act=act)
        nsets = max(2, min(8, math.ceil(4 * 126 * 2**20 / c.algorithmic_bytes)))
        A0, B0, b0 = _dev(c.A, (M, a.K)), _dev(c.B, (a.K, a.N)), _dev(c.bias, (a.N,))
        sets = [(A0, B0, b0, torch.empty((M, a.N), dtype=torch.bfloat16, device="cuda"))]
        for _ in range(nsets - 1):
            sets.append((A0.clone(), B0.clone(), b0.clone(), torch.empty((M, a.N), dtype=torch.bfloat16, device="cuda")))
        h.force_variant(binding.VARIANT_AUTO)
        pick = h.select_variant(M, a.N, a.K, binding.BF16)
        cells, t_pick = [], None
        for v, _ in VARIANTS:
            too_slow = v == binding.VARIANT_GEMV_SPLITK and M > 4
            t = None if too_slow else time_variant(h, v, sets, M, a.N, a.K, act, a.iters)
            cells.append("—" if t is None else ("TIMEOUT" if t != t else f"{t:.1f}"))
            if v == pick:
                t_pick = t
        t_pick = t_pick if t_pick and t_pick == t_pick else float("inf")
        gbs = c.algorithmic_bytes / 1e9 / (t_pick * 1e-6)
        tf = c.flops / 1e12 / (t_pick * 1e-6)
        print(f"| {M} | " + " | ".join(cells) + f" | {binding.variant_name(pick)} | {gbs:.0f} | {tf:.1f} |", flush=True)
        del sets
        torch.cuda.empty_cache()
    h.destroy()


if __name__ == "__main__":
    main()

"""Time every kernel variant that can run a shape, over a sweep of M at fixed (N, K): the
evidence behind the dispatcher's thresholds.

    python -m paper_2602_12305_b200.sweep [--N 8192 --K 8192] [--Ms 1,2,4,...] [--iters 100]

Prints one markdown table row per M: microseconds per launch of each variant (mean over
`--iters` back-to-back launches between two CUDA events, rotating over buffer sets larger
than L2 together) and the variant the dispatcher picks.

    python -m paper_2602_12305_b200.sweep --options [--iters 1000]

Times the two streaming workloads (c2: 1 x 8192 x 8192, c3: 16 x 14336 x 4096) over a grid of
the tuning options of optiml_set_option (L2 prefetch ahead of the dependency wait, stage height,
ring depth, trigger point): the evidence behind their defaults.  Also checks that the scheduling
options leave the output bits alone.
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


def sweep_options(iters):
    h = binding.Handle(0)
    opts = [binding.OPT_GEMV_PREFETCH_ROWS, binding.OPT_SKINNY_STAGE_ROWS, binding.OPT_SKINNY_RING_STAGES,
            binding.OPT_SKINNY_PREFETCH_EARLY, binding.OPT_SKINNY_LATE_TRIGGER]
    defaults = [h.get_option(o) for o in opts]

    def make_sets(c):
        n = max(2, math.ceil(4 * 126 * 2**20 / c.algorithmic_bytes))
        A0, B0, b0 = _dev(c.A, (c.M, c.K)), _dev(c.B, (c.K, c.N)), _dev(c.bias, (c.N,))
        return [(A0.clone(), B0.clone(), b0.clone(), torch.empty((c.M, c.N), dtype=torch.bfloat16, device="cuda"))
                for _ in range(n)]

    def run(c, sets, variant, values):
        for o, v in zip(opts, values):
            h.set_option(o, v)
        t = min(time_variant(h, variant, sets, c.M, c.N, c.K, c.act, iters) for _ in range(2))
        return t, sets[0][3].clone()

    print(f"defaults: gemv_prefetch_rows={defaults[0]} stage_rows={defaults[1]} ring_stages={defaults[2]} "
          f"prefetch_early={defaults[3]} late_trigger={defaults[4]}; best of two runs of {iters} back-to-back launches\n")
    c = synth.make_case("c2")
    sets = make_sets(c)
    print("c2: bf16 1 x 8192 x 8192, GEMV kernel\n\n| rows prefetched before the wait | us per launch | GB/s | same bits |\n|---|---|---|---|")
    ref = None
    for rows in (0, 16, 32, 48, 64, 96, 128, 192, 256):
        t, y = run(c, sets, binding.VARIANT_GEMV_SPLITK, [rows] + defaults[1:])
        ref = y if ref is None else ref
        print(f"| {rows} | {t:.2f} | {c.algorithmic_bytes / t / 1e3:.0f} | {bool(torch.equal(ref, y))} |", flush=True)
    del sets
    torch.cuda.empty_cache()
    c = synth.make_case("c3")
    sets = make_sets(c)
    print("\nc3: bf16 16 x 14336 x 4096, skinny kernel\n\n| stage rows | ring stages | stages prefetched before the wait | late trigger | us per launch | GB/s | same bits |\n|---|---|---|---|---|---|---|")
    ref = {}
    for rows, stage_list in ((192, (2, 3, 4)), (128, (2, 3, 6))):
        for stages in stage_list:
            for early, late in ((0, 0), (0, 1), (2, 0), (2, 1), (4, 1), (8, 1)):
                t, y = run(c, sets, binding.VARIANT_SKINNY_UMMA, [defaults[0], rows, stages, early, late])
                same = bool(torch.equal(ref.setdefault(rows, y), y))
                print(f"| {rows} | {stages} | {early} | {late} | {t:.2f} | {c.algorithmic_bytes / t / 1e3:.0f} | {same} |", flush=True)
    h.destroy()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--options", action="store_true", help="sweep the streaming kernels' tuning options instead")
    ap.add_argument("--N", type=int, default=8192)
    ap.add_argument("--K", type=int, default=8192)
    ap.add_argument("--Ms", default="1,2,4,8,16,32,64,96,128,192,256,512,1024")
    ap.add_argument("--iters", type=int, default=100)
    a = ap.parse_args()
    if a.options:
        return sweep_options(max(a.iters, 1000))
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

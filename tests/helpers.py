"""Shared pieces of the GPU parity tests: moving a synthetic case to the device, running
it through the C ABI, and the three acceptance checks against the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle
from paper_2602_12305_b200 import binding, synth

F32, BF16 = synth.F32, synth.BF16

# Acceptance bounds.
#   fp32: relative Frobenius error of the whole output.
#   bf16: elementwise |y - y_ref| <= BF16_TOL * (1 + |y_ref|) against the UNROUNDED fp64
#         reference (bf16 rounding itself costs 2^-9 relative; fp32 accumulation over
#         K <= 16384 terms and the hardware tanh stay far below the rest of the budget).
#   integer-valued inputs: bit-exact against the oracle's own rounding.
F32_REL_FROBENIUS = 1e-5
BF16_TOL = 1e-2


def to_device(arr: np.ndarray, dtype: int, shape, device="cuda:0") -> torch.Tensor:
    if dtype == F32:
        return torch.from_numpy(np.ascontiguousarray(arr)).view(*shape).to(device)
    return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).view(torch.bfloat16).view(*shape).to(device)


def to_host_bits(t: torch.Tensor, dtype: int) -> np.ndarray:
    """float32 values, or bf16 bit patterns as uint16."""
    t = t.detach().cpu().contiguous()
    if dtype == F32:
        return t.numpy()
    return t.view(torch.int16).numpy().view(np.uint16)


def run_case(handle: binding.Handle, case: synth.Case, poison: bool = True):
    """Run one case on the GPU through the C ABI; returns (Y as host bits, Y widened to fp64)."""
    A = to_device(case.A, case.dtype, (case.M, case.K))
    B = to_device(case.B, case.dtype, (case.K, case.N))
    bias = None if case.bias is None else to_device(case.bias, case.dtype, (case.N,))
    tdt = torch.float32 if case.dtype == F32 else torch.bfloat16
    # Y sits inside a larger buffer whose margins hold a sentinel, and starts as NaN:
    # out-of-bounds writes and unwritten elements both show up.
    guard = 256
    buf = torch.full((case.M * case.N + 2 * guard,), 777.0, dtype=tdt, device="cuda:0")
    Y = buf[guard:guard + case.M * case.N].view(case.M, case.N)
    if poison:
        Y.fill_(float("nan"))
    handle.gemm_epilogue(A, B, bias, case.act, Y=Y)
    torch.cuda.synchronize()
    assert handle.get_last_status() == binding.OK
    margins = torch.cat([buf[:guard], buf[guard + case.M * case.N:]])
    assert bool((margins == 777.0).all()), "kernel wrote outside Y"
    bits = to_host_bits(Y, case.dtype)
    return bits, oracle.widen(bits, case.dtype)


def oracle_full(case: synth.Case) -> np.ndarray:
    return oracle.gemm_epilogue(case.A, case.B, case.bias, case.M, case.N, case.K, case.dtype, case.act)


def check_tolerance(y: np.ndarray, y_ref: np.ndarray, dtype: int, what: str = ""):
    assert y.shape == y_ref.shape
    assert np.isfinite(y).all(), f"{what}: non-finite output (unwritten element?)"
    if dtype == F32:
        err = np.linalg.norm(y - y_ref) / max(np.linalg.norm(y_ref), 1e-300)
        assert err <= F32_REL_FROBENIUS, f"{what}: relative Frobenius error {err:.3e}"
    else:
        excess = np.abs(y - y_ref) - BF16_TOL * (1.0 + np.abs(y_ref))
        worst = np.unravel_index(np.argmax(excess), excess.shape)
        assert excess.max() <= 0.0, (f"{what}: |y - y_ref| = {abs(y[worst] - y_ref[worst]):.4g} at {worst}, "
                                     f"y_ref = {y_ref[worst]:.6g}")


def check_bit_exact(bits: np.ndarray, y_ref: np.ndarray, dtype: int, what: str = ""):
    want = oracle.round_to_dtype(y_ref, dtype)
    if dtype == F32:
        got = bits.astype(np.float32) + np.float32(0.0)     # -0 -> +0
        same = got.view(np.uint32) == want.view(np.uint32)
    else:
        got = np.where(bits == 0x8000, 0, bits).astype(np.uint16)
        same = got == want
    assert same.all(), f"{what}: {np.count_nonzero(~same)} of {same.size} elements differ in bits"

"""The stand-alone reductions (sum, dot, MSE): pins of their oracle on CPU, and GPU parity
through the C ABI."""
import math

import numpy as np
import pytest
import torch

from oracle import reduce_oracle as R
from paper_2602_12305_b200 import binding, synth


def vec(seed, tensor, n, lo=-1.0, hi=1.0):
    return synth.uniform(seed, tensor, n, lo, hi, synth.F32)


# ---------------------------------------------------------------- oracle pins (CPU)

def test_sum_of_integers_closed_form():
    n = 100000
    v, mag = R.reduce_f32(R.SUM, np.arange(1, n + 1, dtype=np.float32))
    assert v == n * (n + 1) / 2 and mag == v
    v, mag = R.reduce_f32(R.SUM, np.array([3.0, -3.0, 5.0, -5.0], np.float32))
    assert v == 0.0 and mag == 16.0


def test_dot_closed_forms():
    n = 1000
    x = np.arange(n, dtype=np.float32)
    e = np.zeros(n, np.float32)
    e[137] = 1.0
    assert R.reduce_f32(R.DOT, x, e)[0] == 137.0                       # selector picks one element
    assert R.reduce_f32(R.DOT, x, np.ones(n, np.float32))[0] == n * (n - 1) / 2
    assert R.reduce_f32(R.DOT, x, x)[0] == (n - 1) * n * (2 * n - 1) / 6   # sum of squares
    a, b = vec(1, 0, 5000), vec(1, 1, 5000)
    assert R.reduce_f32(R.DOT, a, b)[0] == R.reduce_f32(R.DOT, b, a)[0]    # symmetric


def test_mse_closed_forms():
    a = vec(2, 0, 4096)
    assert R.reduce_f32(R.MSE, a, a)[0] == 0.0
    ones = np.ones(4096, np.float32)
    assert R.reduce_f32(R.MSE, ones * 3, ones)[0] == 4.0               # constant offset c: c^2
    x = np.array([1.0, 2.0, 3.0, 4.0], np.float32)
    y = np.array([0.0, 0.0, 0.0, 0.0], np.float32)
    assert R.reduce_f32(R.MSE, x, y)[0] == 7.5                         # (1 + 4 + 9 + 16) / 4


@pytest.mark.parametrize("n", [1, 7, 1000, 250001])
def test_against_exactly_rounded_summation(n):
    a, b = vec(3, 0, n, -10, 10), vec(3, 1, n, -10, 10)
    exact_sum = math.fsum(float(v) for v in a)
    exact_dot = math.fsum(float(p) * float(q) for p, q in zip(a, b))
    exact_mse = math.fsum((float(p) - float(q)) ** 2 for p, q in zip(a, b)) / n
    for kind, exact, args in ((R.SUM, exact_sum, (a,)), (R.DOT, exact_dot, (a, b)), (R.MSE, exact_mse, (a, b))):
        v, mag = R.reduce_f32(kind, *args)
        scale = mag / n if kind == R.MSE else mag
        assert abs(v - exact) <= n * 2.3e-16 * scale + 1e-300           # plain recursive summation bound
    lib = torch.dot(torch.from_numpy(a).double(), torch.from_numpy(b).double()).item()
    assert abs(R.reduce_f32(R.DOT, a, b)[0] - lib) <= 1e-12 * R.reduce_f32(R.DOT, a, b)[1]


# ---------------------------------------------------------------- GPU parity

# fp32 accumulation chains are at most n / (threads * 16) + 16 terms long, then fp64: the
# error is bounded by a small multiple of 2^-24 times the sum of |terms|, plus the final
# rounding of the result to fp32.
GPU_TOL = 1e-5


@pytest.mark.gpu
@pytest.mark.parametrize("n", [1, 3, 4, 1023, 1024, 65537, 1 << 20, (1 << 24) + 5, 1 << 27])
@pytest.mark.parametrize("kind", [R.SUM, R.DOT, R.MSE])
def test_gpu_reduction_matches_oracle(kind, n):
    a, b = vec(5, 0, n, -2, 2), vec(5, 1, n, -2, 2)
    with binding.Handle(0) as h:
        x, y = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
        out = h.reduce_f32(kind, x, None if kind == R.SUM else y)
        out2 = h.reduce_f32(kind, x, None if kind == R.SUM else y)
        torch.cuda.synchronize()
        assert h.get_last_status() == binding.OK
    want, mag = R.reduce_f32(kind, a, None if kind == R.SUM else b)
    scale = mag / n if kind == R.MSE else mag
    got = float(out.item())
    assert abs(got - want) <= GPU_TOL * scale + 1.2e-7 * abs(want) + 1e-30, (got, want, scale)
    assert out.item() == out2.item(), "same call, different bits"


@pytest.mark.gpu
def test_gpu_reduction_integers_exact_and_errors():
    n = 1 << 16
    ones = torch.ones(n, dtype=torch.float32, device="cuda")
    idx = torch.arange(n, dtype=torch.float32, device="cuda") % 8
    with binding.Handle(0) as h:
        assert h.reduce_f32(binding.REDUCE_SUM, idx).item() == float((n // 8) * 28)
        assert h.reduce_f32(binding.REDUCE_DOT, idx, ones).item() == float((n // 8) * 28)
        assert h.reduce_f32(binding.REDUCE_MSE, idx + 2, idx).item() == 4.0
        lib = h._lib
        p = ones.data_ptr()
        assert lib.optiml_reduce_f32(h._h, 0, None, None, 4, p, None) == binding.ERR_INVALID_ARG
        assert lib.optiml_reduce_f32(h._h, 1, p, None, 4, p, None) == binding.ERR_INVALID_ARG
        assert lib.optiml_reduce_f32(h._h, 7, p, p, 4, p, None) == binding.ERR_INVALID_ARG
        assert lib.optiml_reduce_f32(h._h, 0, p, None, 0, p, None) == binding.ERR_INVALID_ARG
        assert lib.optiml_reduce_f32(h._h, 0, p + 4, None, 4, p, None) == binding.ERR_ALIGNMENT
        torch.cuda.synchronize()

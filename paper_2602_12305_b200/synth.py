"""Seeded synthetic inputs for Y = act(A.B + bias).

This module only draws numbers.  It holds none of the method's arithmetic (no
product, no bias add, no activation, no output rounding) and imports neither the
CUDA binding nor the CPU oracle; tests and the benchmark hand the same arrays to
both sides.

Generator.  Every element is a pure function of (seed, tensor id, draw id,
element index): a 64-bit counter is pushed through the SplitMix64 output mix
(Steele, Lea & Flood, "Fast splittable pseudorandom number generators", 2014),
so the value of element i never depends on chunking or on the thread count.

    uniform   u = (h >> 11) * 2^-53                      in [0, 1)
    fp32 U[lo,hi): 24 random bits, lo + (hi-lo) * (h >> 40) * 2^-24
    normal    Box-Muller in fp64: sqrt(-2 ln u1) * cos(2 pi u2), u1 in (0, 1]

bf16 tensors are returned as uint16 bit patterns (numpy has no bf16): the fp64
sample rounded once to 8 significant bits, round-to-nearest-even.

The five named workloads (matrix product as in the paper's Prompts appendix,
task 2, row-major as in its matmul case study; sizes and laws are this
project's) are built by `make_case`.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np

F32 = 0
BF16 = 1
ACT_NONE = 0
ACT_RELU = 1
ACT_GELU_TANH = 2
ACT_SIGMOID = 3

TENSOR_A = 0
TENSOR_B = 1
TENSOR_BIAS = 2

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on a uint64 array (wraps mod 2^64)."""
    x = x.copy()
    x ^= x >> np.uint64(30)
    x *= _M1
    x ^= x >> np.uint64(27)
    x *= _M2
    x ^= x >> np.uint64(31)
    return x


def _stream_key(seed: int, tensor: int, draw: int) -> np.uint64:
    k = (seed * 0x9E3779B97F4A7C15 + tensor * 0xD1B54A32D192ED03 + draw * 0x8CB92BA72F3D8DD7 + 1) & (2**64 - 1)
    return _mix64(np.array([k], dtype=np.uint64))[0]


def raw_bits(seed: int, tensor: int, draw: int, start: int, count: int) -> np.ndarray:
    """64 random bits for elements start .. start+count-1 of one stream."""
    key = _stream_key(seed, tensor, draw)
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix64(key + idx * _GOLDEN)


def _uniform01(seed, tensor, draw, start, count):
    return (raw_bits(seed, tensor, draw, start, count) >> np.uint64(11)).astype(np.float64) * 2.0**-53


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp64 -> bf16 bit patterns, one round-to-nearest-even (input side only)."""
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)
    # quantum of the bf16 grid at this magnitude: 8 significant bits, floor at the subnormal step
    q = np.ldexp(1.0, np.maximum(e - 8, -133))
    y = np.rint(x / q) * q
    return (y.astype(np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (for inspection in tests)."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _chunks(n):
    return [(s, min(_CHUNK, n - s)) for s in range(0, n, _CHUNK)]


def _run_chunks(n, fn, out):
    def work(sc):
        s, c = sc
        out[s:s + c] = fn(s, c)
    parts = _chunks(n)
    if len(parts) <= 1:
        for p in parts:
            work(p)
    else:
        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(work, parts))
    return out


def uniform(seed: int, tensor: int, n: int, lo: float, hi: float, dtype: int) -> np.ndarray:
    """n samples of U[lo, hi) as float32 (dtype F32) or bf16 bits (dtype BF16)."""
    if dtype == F32:
        def f(s, c):
            u24 = (raw_bits(seed, tensor, 0, s, c) >> np.uint64(40)).astype(np.float64)
            return (lo + (hi - lo) * u24 * 2.0**-24).astype(np.float32)
        return _run_chunks(n, f, np.empty(n, dtype=np.float32))

    def g(s, c):
        return round_to_bf16_bits(lo + (hi - lo) * _uniform01(seed, tensor, 0, s, c))
    return _run_chunks(n, g, np.empty(n, dtype=np.uint16))


def normal(seed: int, tensor: int, n: int, sigma: float, dtype: int,
           outlier_prob: float = 0.0, outlier_mag: float = 8.0) -> np.ndarray:
    """n samples of N(0, sigma^2); optionally a Bernoulli(outlier_prob) subset is
    overwritten with +-outlier_mag (sign from an independent bit)."""
    def f(s, c):
        u1 = ((raw_bits(seed, tensor, 0, s, c) >> np.uint64(11)).astype(np.float64) + 1.0) * 2.0**-53
        u2 = _uniform01(seed, tensor, 1, s, c)
        z = sigma * np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        if outlier_prob > 0.0:
            hit = _uniform01(seed, tensor, 2, s, c) < outlier_prob
            sign = np.where(raw_bits(seed, tensor, 3, s, c) >> np.uint64(63), -1.0, 1.0)
            z = np.where(hit, sign * outlier_mag, z)
        return z.astype(np.float32) if dtype == F32 else round_to_bf16_bits(z)
    return _run_chunks(n, f, np.empty(n, dtype=np.float32 if dtype == F32 else np.uint16))


def small_integers(seed: int, tensor: int, n: int, lo: int, hi: int, dtype: int) -> np.ndarray:
    """n integers uniform on lo..hi inclusive, stored exactly in dtype."""
    span = hi - lo + 1
    v = (raw_bits(seed, tensor, 0, 0, n) >> np.uint64(33)).astype(np.int64) % span + lo
    v = v.astype(np.float64)
    return v.astype(np.float32) if dtype == F32 else round_to_bf16_bits(v)


@dataclasses.dataclass
class Case:
    """One problem instance: host arrays plus its shape and epilogue."""
    name: str
    M: int
    N: int
    K: int
    dtype: int
    act: int
    A: np.ndarray      # M*K, row-major, float32 or bf16 bits (uint16)
    B: np.ndarray      # K*N, row-major
    bias: np.ndarray   # N

    @property
    def flops(self) -> int:
        return 2 * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> int:
        """A, B, bias read once and Y written once."""
        es = 4 if self.dtype == F32 else 2
        return es * (self.M * self.K + self.K * self.N + self.N + self.M * self.N)


# name -> (M, N, K, dtype, act, bias law, outlier probability in A)
WORKLOADS = {
    "c1": (256, 256, 256, F32, ACT_RELU, "u1", 0.0),
    "c2": (1, 8192, 8192, BF16, ACT_GELU_TANH, "u0.1", 0.0),
    "c3": (16, 14336, 4096, BF16, ACT_RELU, "zero", 0.0),
    "c4": (4096, 4096, 4096, BF16, ACT_GELU_TANH, "u0.1", 0.0),
    "c5": (8192, 8192, 16384, BF16, ACT_RELU, "u0.1", 0.01),
}


def make_case(name: str, M: int | None = None, N: int | None = None, K: int | None = None,
              seed: int = 0, sigma: float | None = None, act: int | None = None) -> Case:
    """Build workload `name` ("c1".."c5"), optionally at other sizes (same laws).

    bf16 workloads draw A and B from N(0, sigma^2) with sigma = K^(-1/4), i.e.
    variance 1/sqrt(K), so that A.B has unit variance; pass sigma = K^(-1/2) for
    the other reading of "N(0, 1/sqrt(K))".  c1 draws A, B, bias from U[-1, 1).
    """
    m0, n0, k0, dtype, act0, bias_law, p_out = WORKLOADS[name]
    M, N, K = M or m0, N or n0, K or k0
    act = act0 if act is None else act
    if dtype == F32:
        A = uniform(seed, TENSOR_A, M * K, -1.0, 1.0, F32)
        B = uniform(seed, TENSOR_B, K * N, -1.0, 1.0, F32)
    else:
        s = float(K) ** -0.25 if sigma is None else sigma
        A = normal(seed, TENSOR_A, M * K, s, BF16, outlier_prob=p_out)
        B = normal(seed, TENSOR_B, K * N, s, BF16)
    if bias_law == "zero":
        bias = np.zeros(N, dtype=np.float32 if dtype == F32 else np.uint16)
    elif bias_law == "u1":
        bias = uniform(seed, TENSOR_BIAS, N, -1.0, 1.0, dtype)
    else:
        bias = uniform(seed, TENSOR_BIAS, N, -0.1, 0.1, dtype)
    return Case(name, M, N, K, dtype, act, A, B, bias)


def integer_case(M: int, N: int, K: int, dtype: int, act: int, seed: int = 0, amax: int = 4) -> Case:
    """Integer-valued inputs in -amax..amax: every partial sum is an exact
    integer below 2^24 when K*amax^2 + amax < 2^24, so any summation order
    gives the same fp32 accumulator."""
    assert K * amax * amax + amax < 2**24
    A = small_integers(seed, TENSOR_A, M * K, -amax, amax, dtype)
    B = small_integers(seed, TENSOR_B, K * N, -amax, amax, dtype)
    bias = small_integers(seed, TENSOR_BIAS, N, -amax, amax, dtype)
    return Case(f"int{M}x{N}x{K}", M, N, K, dtype, act, A, B, bias)


# ---------------------------------------------------------------- attention inputs

# name -> (N, d_model, heads): the benchmark shapes of the attention row
MHSA_WORKLOADS = {
    "a1": (2048, 1024, 16),      # d_k = 64, small enough for the full oracle
    "a2": (16384, 2048, 16),     # d_k = 128
    "a3": (16384, 1024, 16),     # d_k = 64
}


def mhsa_inputs(n: int, d_model: int, dtype: int = BF16, seed: int = 0, q_gain: float = 1.0, key_growth: float = 0.0):
    """Q, K, V of shape (n, d_model) as flat arrays, N(0, 1) entries (tensor ids 10, 11, 12).
    q_gain scales Q (sharper softmax); key_growth > 0 scales key row j by 1 + key_growth * j / n,
    so that the largest score of a row tends to arrive late in the sweep over the keys."""
    def draw(tensor, gain_rows=None, gain=1.0):
        x = normal(seed, tensor, n * d_model, 1.0, F32).astype(np.float64) * gain
        if gain_rows is not None:
            x = (x.reshape(n, d_model) * gain_rows[:, None]).reshape(-1)
        return x.astype(np.float32) if dtype == F32 else round_to_bf16_bits(x)
    rows = None if key_growth == 0.0 else 1.0 + key_growth * np.arange(n, dtype=np.float64) / n
    return draw(10, gain=q_gain), draw(11, gain_rows=rows), draw(12)

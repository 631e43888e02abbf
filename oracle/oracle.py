"""ctypes front end of the CPU oracle (gemm_epilogue_oracle.c).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline call this; the product path never does.  It imports nothing from the
CUDA package.  Arrays are numpy: float32 for fp32 tensors, uint16 bit patterns
for bf16 tensors; results are float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

F32 = 0
BF16 = 1
ACT_NONE = 0
ACT_RELU = 1
ACT_GELU_TANH = 2
ACT_SIGMOID = 3

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gemm_epilogue_oracle.c")
_LIB = os.path.join(_HERE, "libgemm_epilogue_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (strict IEEE: no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
                        "-o", tmp, _SRC, "-lm", "-lpthread"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.oracle_gemm_epilogue.argtypes = [vp, vp, vp, vp, i64, i64, i64, ci, ci, ci]
        lib.oracle_gemm_epilogue.restype = ci
        lib.oracle_gemm_epilogue_sampled.argtypes = [vp, vp, vp, vp, i64, i64, i64, ci, ci, vp, i64, vp, i64, ci]
        lib.oracle_gemm_epilogue_sampled.restype = ci
        lib.oracle_round_to_dtype.argtypes = [vp, vp, i64, ci]
        lib.oracle_round_to_dtype.restype = None
        lib.oracle_act.argtypes = [ctypes.c_double, ci]
        lib.oracle_act.restype = ctypes.c_double
        lib.oracle_bf16_from_double.argtypes = [ctypes.c_double]
        lib.oracle_bf16_from_double.restype = ctypes.c_uint16
        lib.oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
        lib.oracle_bf16_to_double.restype = ctypes.c_double
        _lib = lib
    return _lib


def _check(arr, dtype, n, what):
    want = np.float32 if dtype == F32 else np.uint16
    a = np.ascontiguousarray(arr).reshape(-1)
    if a.dtype != want or a.size != n:
        raise ValueError(f"{what}: expected {n} elements of {want}, got {a.size} of {a.dtype}")
    return a


def default_threads() -> int:
    return os.cpu_count() or 1


def gemm_epilogue(A, B, bias, M, N, K, dtype, act, nthreads=None) -> np.ndarray:
    """Unrounded fp64 y_ref, shape (M, N)."""
    A = _check(A, dtype, M * K, "A")
    B = _check(B, dtype, K * N, "B")
    b = None if bias is None else _check(bias, dtype, N, "bias")
    y = np.empty(M * N, dtype=np.float64)
    used = _load().oracle_gemm_epilogue(A.ctypes.data, B.ctypes.data, None if b is None else b.ctypes.data,
                                        y.ctypes.data, M, N, K, dtype, act, nthreads or default_threads())
    if used < 0:
        raise RuntimeError("oracle_gemm_epilogue failed")
    gemm_epilogue.threads_used = used
    return y.reshape(M, N)


def gemm_epilogue_sampled(A, B, bias, M, N, K, dtype, act, rows, cols, nthreads=None) -> np.ndarray:
    """Unrounded fp64 y_ref restricted to rows x cols, shape (len(rows), len(cols))."""
    A = _check(A, dtype, M * K, "A")
    B = _check(B, dtype, K * N, "B")
    b = None if bias is None else _check(bias, dtype, N, "bias")
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    y = np.empty(rows.size * cols.size, dtype=np.float64)
    used = _load().oracle_gemm_epilogue_sampled(A.ctypes.data, B.ctypes.data, None if b is None else b.ctypes.data,
                                                y.ctypes.data, M, N, K, dtype, act, rows.ctypes.data, rows.size,
                                                cols.ctypes.data, cols.size, nthreads or default_threads())
    if used < 0:
        raise RuntimeError("oracle_gemm_epilogue_sampled failed (index out of range?)")
    gemm_epilogue_sampled.threads_used = used
    return y.reshape(rows.size, cols.size)


def round_to_dtype(y, dtype) -> np.ndarray:
    """fp64 -> float32 array or bf16 bit patterns (uint16), nearest-even, -0 mapped to +0."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    out = np.empty(y.size, dtype=np.float32 if dtype == F32 else np.uint16)
    _load().oracle_round_to_dtype(y.ctypes.data, out.ctypes.data, y.size, dtype)
    return out.reshape(y.shape)


def act(x: float, kind: int) -> float:
    return _load().oracle_act(float(x), kind)


def bf16_from_double(x: float) -> int:
    return int(_load().oracle_bf16_from_double(float(x)))


def bf16_to_double(bits: int) -> float:
    return float(_load().oracle_bf16_to_double(int(bits)))


def widen(arr, dtype) -> np.ndarray:
    """Exact fp64 view of an input or output array of `dtype` (bf16 given as uint16 bits)."""
    a = np.asarray(arr)
    if dtype == F32:
        return a.astype(np.float64)
    return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)

"""ctypes front end of the reduction oracle (reduce_oracle.c).  TEST INFRASTRUCTURE ONLY."""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

SUM, DOT, MSE = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "reduce_oracle.c")
_LIB = os.path.join(_HERE, "libreduce_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
                        "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_reduce_f32.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
        lib.oracle_reduce_f32.restype = ctypes.c_int
        _lib = lib
    return _lib


def reduce_f32(kind: int, x, y=None):
    """(value, sum of |terms|) in fp64 for float32 arrays x (and y)."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    yy = None if y is None else np.ascontiguousarray(y, dtype=np.float32).reshape(-1)
    if yy is not None and yy.size != x.size:
        raise ValueError("x and y differ in length")
    res = np.zeros(2, dtype=np.float64)
    rc = _load().oracle_reduce_f32(kind, x.ctypes.data, None if yy is None else yy.ctypes.data, x.size, res.ctypes.data)
    if rc != 0:
        raise RuntimeError("oracle_reduce_f32 failed")
    return float(res[0]), float(res[1])

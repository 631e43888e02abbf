"""Build the C-ABI CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2602_12305_b200.build [--force] [--verbose]

Produces paper_2602_12305_b200/liboptiml_gemm.so (cudart linked statically, the driver
API reached through cudaGetDriverEntryPoint, so the file loads on a machine without a GPU).
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "liboptiml_gemm.so")
SOURCES = [os.path.join(CSRC, "optiml_api.cu")]


def _inputs():
    out = [os.path.join(os.path.dirname(_HERE), "include", "optiml.h")]
    for f in sorted(os.listdir(CSRC)):
        if f.endswith((".cu", ".cuh", ".h")):
            out.append(os.path.join(CSRC, f))
    return out


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(p) > t for p in _inputs())


def nvcc_command(out: str, verbose: bool = False) -> list[str]:
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "static", "-o", out] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return cmd


def build_library(force: bool = False, verbose: bool = False) -> str:
    if force or is_stale():
        tmp = LIB_PATH + f".{os.getpid()}.tmp"
        subprocess.run(nvcc_command(tmp, verbose), check=True)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))

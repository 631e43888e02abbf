"""B200-native fused GEMM + bias + activation, Y = act(A.B + bias).

`binding` wraps the C-ABI library (CUDA, sm_100a); `synth` draws the seeded
synthetic inputs.  Importing the package loads neither: the library is opened on
first use and a missing build raises instead of falling back to anything.
"""
__all__ = ["binding", "synth", "build"]

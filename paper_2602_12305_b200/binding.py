"""Python binding of the C-ABI library (include/optiml.h): argument marshalling only.

Every function has the name of the C entry point it calls, minus the `optiml_`
prefix; every step of Y = act(A.B + bias) runs in the CUDA kernels behind it.
PyTorch is used for device memory and streams.  There is no fallback: if the
library has not been built, or there is no B200, calls raise.
"""
from __future__ import annotations

import ctypes
import os

import torch

F32, BF16 = 0, 1
ACT_NONE, ACT_RELU, ACT_GELU_TANH, ACT_SIGMOID = 0, 1, 2, 3
VARIANT_AUTO, VARIANT_GENERIC, VARIANT_F32_TILED, VARIANT_GEMV_SPLITK, VARIANT_SKINNY_UMMA, VARIANT_UMMA = -1, 0, 1, 2, 3, 4
VARIANT_UMMA_2CTA = 5
VARIANT_UMMA_2CTA_STREAM = 6
VARIANT_COUNT = 7

REDUCE_SUM, REDUCE_DOT, REDUCE_MSE = 0, 1, 2

(OPT_GEMV_PREFETCH_ROWS, OPT_SKINNY_STAGE_ROWS, OPT_SKINNY_RING_STAGES, OPT_SKINNY_PREFETCH_EARLY,
 OPT_SKINNY_LATE_TRIGGER, OPT_PAIR_SPLIT_MAX, OPT_PAIR_HALF_HEIGHT, OPT_PAIR_TILE_WIDTH) = range(8)
OPT_COUNT = 8

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_ARCH, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT = range(8)

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liboptiml_gemm.so")

# name -> (restype, argtypes); the same list the header declares
_vp, _i64, _ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
EXPORTS = {
    "optiml_create": (_ci, [ctypes.POINTER(_vp), _ci]),
    "optiml_destroy": (_ci, [_vp]),
    "optiml_gemm_epilogue": (_ci, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _ci, _ci, _vp]),
    "optiml_gemm_epilogue_host": (_ci, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _ci, _ci, _vp]),
    "optiml_gemv_noalloc": (_ci, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _ci, _ci, _vp]),
    "optiml_get_last_status": (_ci, [_vp]),
    "optiml_selftest_timeout": (_ci, [_vp, _i64, _vp]),
    "optiml_set_alloc_hook": (_ci, [_vp, _vp]),
    "optiml_reduce_f32": (_ci, [_vp, _ci, _vp, _vp, _i64, _vp, _vp]),
    "optiml_mhsa": (_ci, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _ci, _vp]),
    "optiml_force_variant": (_ci, [_vp, _ci]),
    "optiml_select_variant": (_ci, [_vp, _i64, _i64, _i64, _ci]),
    "optiml_launch_count": (_i64, [_vp]),
    "optiml_set_option": (_ci, [_vp, _ci, _i64]),
    "optiml_get_option": (_i64, [_vp, _ci]),
    "optiml_status_string": (ctypes.c_char_p, [_ci]),
    "optiml_variant_name": (ctypes.c_char_p, [_ci]),
    "optiml_version": (_ci, []),
}

_lib = None


class OptimlError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


def load_library() -> ctypes.CDLL:
    """Open the in-tree shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2602_12305_b200.build` "
                               "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load_library().optiml_status_string(int(code)).decode()


def variant_name(variant: int) -> str:
    return load_library().optiml_variant_name(int(variant)).decode()


def version() -> int:
    return load_library().optiml_version()


def _check(code: int, where: str):
    if code != OK:
        raise OptimlError(code, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}: float32 or bfloat16 only")


def gemv_noalloc_raw(A: int, B: int, bias: int | None, Y: int, M: int, N: int, K: int, act: int, device: int = 0,
                     stream: int | None = None) -> int:
    """optiml_gemv_noalloc with raw device addresses; returns the status code."""
    return load_library().optiml_gemv_noalloc(A, B, bias, Y, M, N, K, act, device, stream)


def gemv_noalloc(A: torch.Tensor, B: torch.Tensor, bias: torch.Tensor | None, Y: torch.Tensor, act: int,
                 stream: torch.cuda.Stream | None = None) -> torch.Tensor:
    """Y = act(A @ B + bias) for bf16, M <= 4, N <= 65536, without a handle and without any
    allocation inside the library (its scratch is a fixed array in the library image).
    For callers whose device memory is owned by another allocator or who cannot afford an
    allocation's synchronisation.  The caller provides Y.  Calls on one device share the
    scratch: keep them in one stream order."""
    M, K = A.shape
    N = B.shape[1]
    dev = A.device.index
    st = (stream or torch.cuda.current_stream(dev)).cuda_stream
    _check(gemv_noalloc_raw(A.data_ptr(), B.data_ptr(), None if bias is None else bias.data_ptr(), Y.data_ptr(),
                            M, N, K, act, dev, st), "optiml_gemv_noalloc")
    return Y


ALLOC_HOOK = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p)


def set_alloc_hook(hook) -> None:
    """optiml_set_alloc_hook: `hook` is an ALLOC_HOOK instance (keep a reference to it while it is
    set) or None to remove it."""
    lib = load_library()
    _check(lib.optiml_set_alloc_hook(None if hook is None else ctypes.cast(hook, _vp), None), "optiml_set_alloc_hook")


class Handle:
    """Owns one optiml_handle_t (device scratch + tensor-map cache).  One per stream."""

    def __init__(self, device: int = 0):
        self._h = _vp()
        self._lib = load_library()
        _check(self._lib.optiml_create(ctypes.byref(self._h), int(device)), "optiml_create")
        self.device = int(device)

    def destroy(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.optiml_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.destroy()
        except Exception:      # interpreter shutdown: the library object may already be gone
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()

    # -- same names as the C entry points ------------------------------------------------

    def gemm_epilogue_raw(self, A: int, B: int, bias: int | None, Y: int, M: int, N: int, K: int, dtype: int,
                          act: int, stream: int | None = None) -> int:
        """Direct call with raw device addresses; returns the status code."""
        return self._lib.optiml_gemm_epilogue(self._h, A, B, bias, Y, M, N, K, dtype, act, stream)

    def gemm_epilogue(self, A: torch.Tensor, B: torch.Tensor, bias: torch.Tensor | None, act: int,
                      Y: torch.Tensor | None = None, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Y = act(A @ B + bias) on CUDA tensors (A: M x K, B: K x N, bias: N; contiguous)."""
        if A.dim() != 2 or B.dim() != 2 or A.shape[1] != B.shape[0]:
            raise ValueError("A must be M x K and B K x N")
        M, K = A.shape
        N = B.shape[1]
        dt = _dtype_code(A)
        for t, name in ((A, "A"), (B, "B"), (bias, "bias"), (Y, "Y")):
            if t is None:
                continue
            if not t.is_cuda or t.device.index != self.device or t.dtype != A.dtype or not t.is_contiguous():
                raise ValueError(f"{name}: need a contiguous {A.dtype} tensor on cuda:{self.device}")
        if bias is not None and bias.numel() != N:
            raise ValueError("bias must have N elements")
        if Y is None:
            Y = torch.empty((M, N), dtype=A.dtype, device=A.device)
        elif tuple(Y.shape) != (M, N):
            raise ValueError("Y must be M x N")
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        _check(self.gemm_epilogue_raw(A.data_ptr(), B.data_ptr(), None if bias is None else bias.data_ptr(),
                                      Y.data_ptr(), M, N, K, dt, act, st), "optiml_gemm_epilogue")
        return Y

    def gemm_epilogue_host(self, A: torch.Tensor, B: torch.Tensor, bias: torch.Tensor | None, Y: torch.Tensor,
                           act: int, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Same with HOST tensors (pinned for asynchronous copies); returns after Y is filled."""
        M, K = A.shape
        N = B.shape[1]
        dt = _dtype_code(A)
        for t in (A, B, bias, Y):
            if t is not None and (t.is_cuda or not t.is_contiguous() or t.dtype != A.dtype):
                raise ValueError("host entry point needs contiguous CPU tensors of one dtype")
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        _check(self._lib.optiml_gemm_epilogue_host(self._h, A.data_ptr(), B.data_ptr(),
                                                   None if bias is None else bias.data_ptr(), Y.data_ptr(), M, N, K,
                                                   dt, act, st), "optiml_gemm_epilogue_host")
        return Y

    def reduce_f32(self, kind: int, x: torch.Tensor, y: torch.Tensor | None = None, out: torch.Tensor | None = None,
                   stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """sum(x), dot(x, y) or mean((x - y)^2) of fp32 CUDA vectors into a one-element fp32 tensor."""
        for t in (x, y):
            if t is not None and (not t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous()):
                raise ValueError("reduce_f32 needs contiguous float32 CUDA tensors")
        if y is not None and y.numel() != x.numel():
            raise ValueError("x and y must have the same length")
        if out is None:
            out = torch.empty(1, dtype=torch.float32, device=x.device)
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        _check(self._lib.optiml_reduce_f32(self._h, int(kind), x.data_ptr(), None if y is None else y.data_ptr(),
                                           x.numel(), out.data_ptr(), st), "optiml_reduce_f32")
        return out

    def mhsa(self, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, heads: int, Y: torch.Tensor | None = None,
             stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Multi-head self-attention of (N, d_model) CUDA tensors (float32 or bfloat16), heads in column blocks."""
        n, d_model = Q.shape
        for t in (Q, K, V):
            if not t.is_cuda or t.dtype != Q.dtype or tuple(t.shape) != (n, d_model) or not t.is_contiguous():
                raise ValueError("mhsa needs contiguous CUDA tensors of one dtype and shape (N, d_model)")
        if Q.dtype not in (torch.float32, torch.bfloat16):
            raise ValueError("mhsa supports float32 and bfloat16")
        if Y is None:
            Y = torch.empty_like(Q)
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        _check(self._lib.optiml_mhsa(self._h, Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(), n, d_model, int(heads),
                                     F32 if Q.dtype == torch.float32 else BF16, st), "optiml_mhsa")
        return Y

    def get_last_status(self) -> int:
        return self._lib.optiml_get_last_status(self._h)

    def selftest_timeout(self, limit_cycles: int, stream: torch.cuda.Stream | None = None) -> int:
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        return self._lib.optiml_selftest_timeout(self._h, int(limit_cycles), st)

    def force_variant(self, variant: int):
        _check(self._lib.optiml_force_variant(self._h, int(variant)), "optiml_force_variant")

    def select_variant(self, M: int, N: int, K: int, dtype: int) -> int:
        return self._lib.optiml_select_variant(self._h, M, N, K, dtype)

    def launch_count(self) -> int:
        return self._lib.optiml_launch_count(self._h)

    def set_option(self, opt: int, value: int):
        _check(self._lib.optiml_set_option(self._h, int(opt), int(value)), "optiml_set_option")

    def get_option(self, opt: int) -> int:
        return self._lib.optiml_get_option(self._h, int(opt))

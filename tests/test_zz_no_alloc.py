"""The entry point that allocates nothing (optiml_gemv_noalloc), checked against the
regular entry point.  It exists for callers that cannot call cudaMalloc -- their device
memory belongs to another allocator, or they cannot take an allocation's synchronisation
-- and therefore cannot create a handle either.  Collected last on purpose: a run that
stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2602_12305_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _device_case(M, N, K, act):
    c = synth.make_case("c2", M=M, N=N, K=K, act=act)
    A = H.to_device(c.A, c.dtype, (M, K))
    B = H.to_device(c.B, c.dtype, (K, N))
    bias = H.to_device(c.bias, c.dtype, (N,))
    return c, A, B, bias


@pytest.mark.parametrize("M,N,K,act", [(1, 8192, 8192, synth.ACT_GELU_TANH), (3, 1032, 777, synth.ACT_RELU),
                                       (4, 65536, 256, synth.ACT_NONE)])
def test_noalloc_matches_the_regular_entry_point_twice_in_a_row(M, N, K, act):
    c, A, B, bias = _device_case(M, N, K, act)
    with binding.Handle(0) as h:
        h.force_variant(binding.VARIANT_GEMV_SPLITK)
        want = h.gemm_epilogue(A, B, bias, act)
        torch.cuda.synchronize()
    want64 = oracle.widen(H.to_host_bits(want, c.dtype), c.dtype)
    ref = H.oracle_full(c) if M * N * K <= 2 ** 28 else None
    Ys = [torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda:0") for _ in range(2)]
    torch.cuda.synchronize()
    for call in range(2):                       # the second call finds the first call's leftovers in the scratch
        Y = Ys[call]
        # free device memory as the driver counts it (cudaMemGetInfo): unlike the framework's own
        # allocator statistics it would move if the library called cudaMalloc.  The first call on a
        # device may load the kernel's module, so equality is demanded of the second call only.
        before = torch.cuda.mem_get_info(0)[0]
        binding.gemv_noalloc(A, B, bias, Y, act)
        torch.cuda.synchronize()
        if call == 1:
            assert torch.cuda.mem_get_info(0)[0] == before, "the call changed the device's free memory"
        got64 = oracle.widen(H.to_host_bits(Y, c.dtype), c.dtype)
        # same tolerance as every bf16 parity test, against the regular entry point's output
        H.check_tolerance(got64, want64, c.dtype, f"noalloc call {call} vs regular entry point")
        if ref is not None:
            H.check_tolerance(got64, ref, c.dtype, f"noalloc call {call} vs CPU reference")


def test_noalloc_rejects_what_the_fixed_scratch_cannot_hold():
    x = torch.zeros(1024, dtype=torch.bfloat16, device="cuda:0")
    p = x.data_ptr()
    call = binding.gemv_noalloc_raw
    assert call(p, p, None, p, 1, 65536 + 8, 8, synth.ACT_NONE) == binding.ERR_UNSUPPORTED     # N beyond the maximum
    assert call(p, p, None, p, 5, 64, 8, synth.ACT_NONE) == binding.ERR_UNSUPPORTED            # M beyond the maximum
    assert call(p, p, None, p, 1, 60, 8, synth.ACT_NONE) == binding.ERR_UNSUPPORTED            # N % 8 != 0
    assert call(p + 2, p, None, p, 1, 64, 8, synth.ACT_NONE) == binding.ERR_ALIGNMENT
    assert call(None, p, None, p, 1, 64, 8, synth.ACT_NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, p, 1, 64, 0, synth.ACT_NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, p, 1, 64, 8, synth.ACT_NONE, device=torch.cuda.device_count()) == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()

"""Failure paths, exercised without faulting, trapping or hanging the GPU:

* a bounded on-device wait that runs out (optiml_selftest_timeout: a barrier nobody signals,
  a short limit) must surface as OPTIML_ERR_TIMEOUT exactly once, leave the context usable
  and the handle's arrival counters re-armed;
* a device allocation that fails (injected on the host through optiml_set_alloc_hook) must
  surface as OPTIML_ERR_ALLOC, leak nothing and leave the handle usable where it survives;
* the tensor-map cache must hand out the right map when more distinct output buffers pass
  through one handle than it has slots.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2602_12305_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_a_bounded_wait_that_runs_out_is_reported_once_and_the_handle_stays_usable():
    with binding.Handle(0) as h:
        assert h.get_last_status() == binding.OK
        n0 = h.launch_count()
        assert h.selftest_timeout(100_000) == binding.OK          # about 50 microseconds
        assert h.launch_count() == n0 + 1
        torch.cuda.synchronize()                                    # returns: nothing trapped, nothing hangs
        assert h.get_last_status() == binding.ERR_TIMEOUT
        assert h.get_last_status() == binding.OK                    # the word was cleared by the first read
        # split-K / stream-K shapes right after: their arrival counters were re-armed by the read above
        for name, kw in (("c3", dict(N=1160, K=1096)), ("c2", dict(N=2048, K=2048)), ("c4", dict(M=520, N=776, K=512))):
            c = synth.make_case(name, **kw)
            _, y = H.run_case(h, c)
            H.check_tolerance(y, H.oracle_full(c), c.dtype, f"{name} after a reported time-out")
        # bad arguments never launch
        assert h.selftest_timeout(0) == binding.ERR_INVALID_ARG
        assert h.selftest_timeout(10 ** 10) == binding.ERR_INVALID_ARG
        assert h.get_last_status() == binding.OK


def test_a_time_out_between_two_calls_does_not_disturb_their_results():
    c = synth.make_case("c3", N=1160, K=1096)
    with binding.Handle(0) as h:
        bits0, _ = H.run_case(h, c)
        assert h.selftest_timeout(50_000) == binding.OK
        assert h.get_last_status() == binding.ERR_TIMEOUT
        bits1, _ = H.run_case(h, c)
        assert np.array_equal(bits0, bits1)


class _FailNth:
    """Allocation hook that refuses the n-th request it sees (1-based) and records all sizes."""

    def __init__(self, n):
        self.n, self.seen = n, []
        self.cb = binding.ALLOC_HOOK(self._call)

    def _call(self, nbytes, _user):
        self.seen.append(int(nbytes))
        return 1 if len(self.seen) == self.n else 0


@pytest.fixture
def no_hook_afterwards():
    yield
    binding.set_alloc_hook(None)


def test_create_reports_a_failed_allocation_and_leaks_nothing(no_hook_afterwards):
    with binding.Handle(0):
        pass                                        # context and library set-up are done before the measurement
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info(0)[0]
    for n in (1, 2, 3):                             # partial sums, counters, status word
        hook = _FailNth(n)
        binding.set_alloc_hook(hook.cb)
        with pytest.raises(binding.OptimlError) as e:
            binding.Handle(0)
        assert e.value.code == binding.ERR_ALLOC
        assert len(hook.seen) == n
        binding.set_alloc_hook(None)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(0)[0] == free0, "a failed optiml_create kept device memory"
    hook = _FailNth(0)                              # a hook that never refuses: create succeeds, three requests
    binding.set_alloc_hook(hook.cb)
    with binding.Handle(0) as h:
        assert len(hook.seen) == 3 and hook.seen[0] == 32 << 20
        assert h.get_last_status() == binding.OK


def test_host_entry_point_survives_a_failed_staging_allocation(no_hook_afterwards):
    c = synth.make_case("c4", M=96, N=264, K=136)
    A = torch.from_numpy(c.A.view(np.int16)).view(torch.bfloat16).view(c.M, c.K)
    B = torch.from_numpy(c.B.view(np.int16)).view(torch.bfloat16).view(c.K, c.N)
    bias = torch.from_numpy(c.bias.view(np.int16)).view(torch.bfloat16)
    Y = torch.zeros((c.M, c.N), dtype=torch.bfloat16)
    with binding.Handle(0) as h:
        for n in (1, 2, 4):                         # A, B and Y staging buffers in turn
            hook = _FailNth(n)
            binding.set_alloc_hook(hook.cb)
            with pytest.raises(binding.OptimlError) as e:
                h.gemm_epilogue_host(A, B, bias, Y, c.act)
            assert e.value.code == binding.ERR_ALLOC
            binding.set_alloc_hook(None)
            # fresh handle state is not needed: the same handle completes the same call now
            h.gemm_epilogue_host(A, B, bias, Y, c.act)
            assert h.get_last_status() == binding.OK
            from oracle import oracle
            y = oracle.widen(Y.view(torch.int16).numpy().view(np.uint16), c.dtype)
            H.check_tolerance(y, H.oracle_full(c), c.dtype, f"host call after failed allocation {n}")
            # make the next round allocate again: a larger problem needs larger buffers
            c = synth.make_case("c4", M=c.M + 8, N=c.N + 8, K=c.K + 8)
            A = torch.from_numpy(c.A.view(np.int16)).view(torch.bfloat16).view(c.M, c.K)
            B = torch.from_numpy(c.B.view(np.int16)).view(torch.bfloat16).view(c.K, c.N)
            bias = torch.from_numpy(c.bias.view(np.int16)).view(torch.bfloat16)
            Y = torch.zeros((c.M, c.N), dtype=torch.bfloat16)


@pytest.mark.parametrize("variant,M,N,K", [(binding.VARIANT_UMMA_2CTA, 136, 264, 200), (binding.VARIANT_UMMA, 136, 264, 200),
                                           (binding.VARIANT_SKINNY_UMMA, 16, 264, 200)])
def test_more_output_buffers_than_tensor_map_cache_slots(variant, M, N, K):
    """Fixed A and B, a fresh Y address on every call (slices of one buffer): the misses on Y walk
    through every cache slot, including the ones that hold A's and B's maps."""
    c = synth.make_case("c4", M=M, N=N, K=K)
    want = H.oracle_full(c)
    A = H.to_device(c.A, c.dtype, (M, K))
    B = H.to_device(c.B, c.dtype, (K, N))
    bias = H.to_device(c.bias, c.dtype, (N,))
    n_calls = 80
    out = torch.full((n_calls, M, N), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    with binding.Handle(0) as h:
        h.force_variant(variant)
        for i in range(n_calls):
            h.gemm_epilogue(A, B, bias, c.act, Y=out[i])
            if variant == binding.VARIANT_SKINNY_UMMA and i % 3 == 0:
                # this variant has no map for Y: rotate A instead, B stays
                A = A.clone()
        torch.cuda.synchronize()
        assert h.get_last_status() == binding.OK
    from oracle import oracle
    for i in range(n_calls):
        y = oracle.widen(H.to_host_bits(out[i], c.dtype), c.dtype)
        H.check_tolerance(y, want, c.dtype, f"call {i}")

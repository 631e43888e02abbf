"""GPU parity of multi-head self-attention (paper: Prompts appendix, task 6) against the fp64
oracle, through the C ABI: the tcgen05 kernel (bf16, d_k = 64 / 128) and the FMA kernel."""
import numpy as np
import pytest
import torch

from oracle import mhsa_oracle
from paper_2602_12305_b200 import binding, synth
from tests.helpers import to_device, to_host_bits

pytestmark = pytest.mark.gpu

F32, BF16 = synth.F32, synth.BF16


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(0)
    yield h
    h.destroy()


def run(handle, q, k, v, n, d_model, heads, dtype):
    """Y on the host (fp64) from one call; Y sits between sentinel margins and starts as NaN."""
    Q, K, V = (to_device(x, dtype, (n, d_model)) for x in (q, k, v))
    tdt = torch.float32 if dtype == F32 else torch.bfloat16
    guard = 512
    buf = torch.full((n * d_model + 2 * guard,), 777.0, dtype=tdt, device="cuda:0")
    Y = buf[guard:guard + n * d_model].view(n, d_model)
    Y.fill_(float("nan"))
    handle.mhsa(Q, K, V, heads, Y=Y)
    torch.cuda.synchronize()
    assert handle.get_last_status() == binding.OK
    margins = torch.cat([buf[:guard], buf[guard + n * d_model:]])
    assert bool((margins == 777.0).all()), "kernel wrote outside Y"
    return mhsa_oracle.widen(to_host_bits(Y, dtype)).reshape(n, d_model)


def check_bf16(y, ref, v):
    """Probabilities are rounded to bf16 (unit roundoff u = 2^-9) before they multiply V, while
    their sum is kept unrounded: the quotient is off by at most u * max|V|; the store adds
    u * |y|.  fp32 accumulation and the hardware exp2 are orders of magnitude below.  Twice that."""
    vmax = np.abs(mhsa_oracle.widen(v)).max()
    assert np.isfinite(y).all()
    err = np.abs(y - ref)
    bound = 2.0 ** -8 * (vmax + np.abs(ref))
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), f"worst at {worst}: got {y[worst]}, want {ref[worst]}"


TENSOR_CORE_CASES = [
    # n, d_model, heads
    (256, 128, 2), (256, 256, 2), (128, 64, 1), (512, 128, 1),
    (1, 64, 1), (100, 128, 2), (129, 256, 2), (257, 192, 3), (1000, 256, 4), (383, 128, 1),
    (2048, 1024, 16), (2048, 1024, 8), (4096, 256, 2),
]


@pytest.mark.parametrize("n,d_model,heads", TENSOR_CORE_CASES)
def test_tensor_core_kernel_matches_oracle(handle, n, d_model, heads):
    q, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=n + heads)
    y = run(handle, q, k, v, n, d_model, heads, BF16)
    check_bf16(y, mhsa_oracle.mhsa(q, k, v, n, d_model, heads), v)


# d_k = 128 also has a CTA-pair kernel (each CTA stages half of every K and V block), a forced variant only
PAIR_CASES = [(257, 128, 1), (512, 128, 1), (513, 256, 2), (640, 384, 3), (1000, 256, 2), (1537, 128, 1), (4096, 256, 2),
              (2048, 2048, 16)]


@pytest.mark.parametrize("n,d_model,heads", PAIR_CASES + [(100, 128, 1), (256, 256, 2)])
def test_cta_pair_kernel_matches_oracle(handle, n, d_model, heads):
    q, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=n + heads)
    handle.force_variant(binding.VARIANT_UMMA_2CTA)
    try:
        y = run(handle, q, k, v, n, d_model, heads, BF16)
    finally:
        handle.force_variant(binding.VARIANT_AUTO)
    check_bf16(y, mhsa_oracle.mhsa(q, k, v, n, d_model, heads), v)


def test_cta_pair_kernel_with_late_maxima(handle):
    n, d_model, heads = 1500, 256, 2
    q, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=7, q_gain=3.0, key_growth=3.0)
    handle.force_variant(binding.VARIANT_UMMA_2CTA)
    try:
        y = run(handle, q, k, v, n, d_model, heads, BF16)
    finally:
        handle.force_variant(binding.VARIANT_AUTO)
    check_bf16(y, mhsa_oracle.mhsa(q, k, v, n, d_model, heads), v)


@pytest.mark.parametrize("d_model,heads", [(128, 2), (256, 2)])
@pytest.mark.parametrize("q_gain,key_growth", [(4.0, 0.0), (1.0, 6.0), (3.0, 3.0), (16.0, 0.0)])
def test_sharp_and_late_maxima(handle, d_model, heads, q_gain, key_growth):
    """Scores whose row maximum keeps rising along the keys exercise the rescaling of the
    accumulator; a large query gain makes the softmax nearly one-hot."""
    n = 1500
    q, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=7, q_gain=q_gain, key_growth=key_growth)
    y = run(handle, q, k, v, n, d_model, heads, BF16)
    check_bf16(y, mhsa_oracle.mhsa(q, k, v, n, d_model, heads), v)


def test_zero_queries_average_the_values(handle):
    n, d_model, heads = 640, 128, 2
    _, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=3)
    q = np.zeros(n * d_model, dtype=np.uint16)
    y = run(handle, q, k, v, n, d_model, heads, BF16)
    mean = mhsa_oracle.widen(v).reshape(n, d_model).mean(axis=0)
    assert np.abs(y - mean).max() <= 2.0 ** -8 * (np.abs(mean).max() + 1e-3) + 1e-6


def test_same_bits_every_time(handle):
    n, d_model, heads = 900, 256, 2
    q, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=5)
    Q, K, V = (to_device(x, BF16, (n, d_model)) for x in (q, k, v))
    first = handle.mhsa(Q, K, V, heads).clone()
    for _ in range(3):
        assert torch.equal(handle.mhsa(Q, K, V, heads).view(torch.int16), first.view(torch.int16))
    assert handle.get_last_status() == binding.OK


@pytest.mark.parametrize("name", ["a2", "a3"])
def test_benchmark_shapes_on_sampled_rows(handle, name):
    n, d_model, heads = synth.MHSA_WORKLOADS[name]
    q, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=0)
    y = run(handle, q, k, v, n, d_model, heads, BF16)
    # every residue of the row index modulo the 256-row CTA tile, spread over the matrix
    rows = sorted({(i * 8209 + (i % 256)) % n for i in range(256)} | {0, 127, 128, 255, 256, n - 1})
    ref = mhsa_oracle.mhsa(q, k, v, n, d_model, heads, rows=rows)
    check_bf16(y[rows], ref, v)


GENERIC_CASES = [
    # n, d_model, heads, dtype
    (200, 96, 3, F32), (77, 64, 8, F32), (33, 256, 1, F32), (300, 60, 3, F32), (1, 8, 2, F32),
    (200, 96, 3, BF16), (150, 80, 1, BF16), (260, 128, 2, BF16),
]


@pytest.mark.parametrize("n,d_model,heads,dtype", GENERIC_CASES)
def test_fma_kernel_matches_oracle(handle, n, d_model, heads, dtype):
    q, k, v = synth.mhsa_inputs(n, d_model, dtype, seed=n)
    handle.force_variant(binding.VARIANT_GENERIC)
    try:
        y = run(handle, q, k, v, n, d_model, heads, dtype)
    finally:
        handle.force_variant(binding.VARIANT_AUTO)
    ref = mhsa_oracle.mhsa(q, k, v, n, d_model, heads)
    if dtype == F32:
        # fp32 throughout: a few hundred roundings of relative size 2^-24 per output
        assert np.abs(y - ref).max() <= 1e-5 * (1.0 + np.abs(ref).max())
    else:
        assert (np.abs(y - ref) <= 2.0 ** -8 * (1e-2 + np.abs(ref)) + 1e-5).all()


def test_the_two_kernels_agree(handle):
    n, d_model, heads = 700, 256, 4
    q, k, v = synth.mhsa_inputs(n, d_model, BF16, seed=11)
    fast = run(handle, q, k, v, n, d_model, heads, BF16)
    handle.force_variant(binding.VARIANT_GENERIC)
    try:
        slow = run(handle, q, k, v, n, d_model, heads, BF16)
    finally:
        handle.force_variant(binding.VARIANT_AUTO)
    vmax = np.abs(mhsa_oracle.widen(v)).max()
    assert (np.abs(fast - slow) <= 2.0 ** -7 * (vmax + np.abs(slow))).all()


def test_argument_errors(handle):
    x = torch.zeros((64, 96), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(binding.OptimlError) as e:
        handle.mhsa(x, x, x, 5)                                  # 96 is not a multiple of 5
    assert e.value.code == binding.ERR_INVALID_ARG
    wide = torch.zeros((8, 1024), dtype=torch.float32, device="cuda:0")
    with pytest.raises(binding.OptimlError) as e:
        handle.mhsa(wide, wide, wide, 2)                         # d_k = 512
    assert e.value.code == binding.ERR_UNSUPPORTED
    f = torch.zeros((64, 128), dtype=torch.float32, device="cuda:0")
    handle.force_variant(binding.VARIANT_UMMA)
    try:
        with pytest.raises(binding.OptimlError) as e:
            handle.mhsa(f, f, f, 2)                              # fp32 has no tensor-core path
        assert e.value.code == binding.ERR_UNSUPPORTED
    finally:
        handle.force_variant(binding.VARIANT_AUTO)

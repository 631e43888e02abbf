"""Pins for the CPU oracle: every check here compares it with something that does
not go through oracle/ -- closed forms, exact integer arithmetic, invariants, or
an independent library routine in fp64.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2602_12305_b200 import synth

F32, BF16 = oracle.F32, oracle.BF16
NONE, RELU, GELU = oracle.ACT_NONE, oracle.ACT_RELU, oracle.ACT_GELU_TANH


def enc(x, dtype):
    """Exact encoding of values known to be representable in dtype."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == F32:
        out = x.astype(np.float32)
        assert np.array_equal(out.astype(np.float64), x)
        return out.reshape(-1)
    out = synth.round_to_bf16_bits(x)
    assert np.array_equal(synth.bf16_bits_to_f64(out), x)
    return out.reshape(-1)


def run(A, B, bias, M, N, K, dtype, act, **kw):
    return oracle.gemm_epilogue(A, B, bias, M, N, K, dtype, act, **kw)


# ---------------------------------------------------------------- layout / indexing

@pytest.mark.parametrize("dtype", [F32, BF16])
def test_identity_B_returns_A_plus_bias(dtype):
    M, K = 5, 7
    A = np.arange(M * K, dtype=np.float64).reshape(M, K) - 17.0
    bias = np.arange(K, dtype=np.float64) * 2.0 - 3.0
    y = run(enc(A, dtype), enc(np.eye(K), dtype), enc(bias, dtype), M, K, K, dtype, NONE)
    assert np.array_equal(y, A + bias)
    y = run(enc(A, dtype), enc(np.eye(K), dtype), enc(bias, dtype), M, K, K, dtype, RELU)
    assert np.array_equal(y, np.maximum(A + bias, 0.0))


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_permutation_B_permutes_columns(dtype):
    # B[k, n] = 1 iff k == perm[n]  =>  Y[:, n] = A[:, perm[n]]; non-square A so a
    # transposed read of either operand cannot pass.
    M, K = 3, 6
    perm = np.array([4, 0, 5, 2, 1, 3])
    A = (np.arange(M * K, dtype=np.float64).reshape(M, K) * 3.0) % 11.0 - 5.0
    B = np.zeros((K, K))
    B[perm, np.arange(K)] = 1.0
    y = run(enc(A, dtype), enc(B, dtype), None, M, K, K, dtype, NONE)
    assert np.array_equal(y, A[:, perm])


def test_selector_B_rectangular():
    # K != N: B picks column 2 of A into output column 0 and column 0 into column 3.
    M, K, N = 4, 3, 5
    A = np.array([[1, 2, 3], [4, 5, 6], [7, 8, 9], [10, 11, 12]], dtype=np.float64)
    B = np.zeros((K, N))
    B[2, 0] = 1.0
    B[0, 3] = 1.0
    y = run(enc(A, F32), enc(B, F32), None, M, N, K, F32, NONE)
    want = np.zeros((M, N))
    want[:, 0] = A[:, 2]
    want[:, 3] = A[:, 0]
    assert np.array_equal(y, want)


# ---------------------------------------------------------------- contraction

@pytest.mark.parametrize("dtype", [F32, BF16])
def test_rank_one_closed_form(dtype):
    # A[m,k] = u[m], B[k,n] = v[n]  =>  Y[m,n] = K u[m] v[n], exact for small integers.
    M, N, K = 6, 9, 37
    u = np.array([1, -2, 3, 0, 4, -1], dtype=np.float64)
    v = np.array([2, 1, -1, 0, 3, -3, 4, 1, -2], dtype=np.float64)
    A = np.repeat(u[:, None], K, axis=1)
    B = np.repeat(v[None, :], K, axis=0)
    y = run(enc(A, dtype), enc(B, dtype), None, M, N, K, dtype, NONE)
    assert np.array_equal(y, K * np.outer(u, v))


@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("act", [NONE, RELU])
def test_integer_inputs_match_exact_integer_arithmetic(dtype, act):
    c = synth.integer_case(13, 21, 300, dtype, act, seed=3)
    Ai = oracle.widen(c.A, dtype).astype(np.int64).reshape(c.M, c.K)
    Bi = oracle.widen(c.B, dtype).astype(np.int64).reshape(c.K, c.N)
    bi = oracle.widen(c.bias, dtype).astype(np.int64)
    want = Ai @ Bi + bi                      # int64: exact
    if act == RELU:
        want = np.maximum(want, 0)
    y = run(c.A, c.B, c.bias, c.M, c.N, c.K, dtype, act)
    assert np.array_equal(y, want.astype(np.float64))
    assert np.abs(want).max() > 50          # the case is not trivially zero


def test_zero_A_gives_activated_bias_on_every_row():
    M, N, K = 4, 6, 10
    bias = np.array([-3.0, -0.5, 0.0, 0.25, 1.0, 2.5])
    B = np.arange(K * N, dtype=np.float64).reshape(K, N) - 20.0
    for act, f in ((NONE, lambda x: x), (RELU, lambda x: np.maximum(x, 0.0))):
        y = run(enc(np.zeros((M, K)), F32), enc(B, F32), enc(bias, F32), M, N, K, F32, act)
        assert np.array_equal(y, np.tile(f(bias), (M, 1)))


def test_null_bias_is_zero_bias():
    c = synth.make_case("c1", M=7, N=12, K=9)
    y0 = run(c.A, c.B, None, c.M, c.N, c.K, c.dtype, NONE)
    y1 = run(c.A, c.B, np.zeros(c.N, np.float32), c.M, c.N, c.K, c.dtype, NONE)
    assert np.array_equal(y0, y1)


# ---------------------------------------------------------------- activations

def test_relu_fixed_points():
    # K = 1, B = [1]: y = act(a)
    for a, want in ((-3.0, 0.0), (0.0, 0.0), (2.5, 2.5), (-0.0, 0.0)):
        y = run(enc([a], F32), enc([1.0], F32), None, 1, 1, 1, F32, RELU)
        assert y[0, 0] == want and not math.copysign(1.0, y[0, 0]) < 0
    assert oracle.act(-1e-300, RELU) == 0.0 and oracle.act(1e-300, RELU) == 1e-300


def test_gelu_tanh_invariants():
    assert oracle.act(0.0, GELU) == 0.0
    xs = np.linspace(-9.0, 9.0, 721)
    g = np.array([oracle.act(x, GELU) for x in xs])
    gm = np.array([oracle.act(-x, GELU) for x in xs])
    # tanh is odd, so G(x) - G(-x) = x exactly in real arithmetic
    assert np.allclose(g - gm, xs, rtol=0, atol=4e-16 * 9)
    # saturation: G(x) -> x and G(-x) -> 0 for large x
    assert abs(oracle.act(9.0, GELU) - 9.0) < 1e-14 and abs(oracle.act(-9.0, GELU)) < 1e-14
    # one global minimum near x = -0.75 with value about -0.17; monotone to the right of it
    i = int(np.argmin(g))
    assert -0.80 < xs[i] < -0.70 and -0.1705 < g[i] < -0.1695
    assert np.all(np.diff(g[i:]) > 0)


def test_gelu_tanh_is_the_tanh_form_not_erf():
    xs = np.linspace(-6.0, 6.0, 4801)
    g = np.array([oracle.act(x, GELU) for x in xs])
    t = torch.from_numpy(xs)
    lib_tanh = torch.nn.functional.gelu(t, approximate="tanh").numpy()
    lib_erf = torch.nn.functional.gelu(t).numpy()
    assert np.abs(g - lib_tanh).max() < 1e-14
    d = np.abs(g - lib_erf).max()
    assert 1e-4 < d < 1e-3        # the tanh form differs from the erf form by a few 1e-4


def test_gelu_tanh_stored_values():
    """Golden values written with 50-digit decimal arithmetic (tests/golden/make_gelu_tanh_values.py):
    G(0), G(+-0.5), G(+-1), G(+-2), G(+-3), G(+-6) and three more, to a few ulp of fp64."""
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "gelu_tanh_values.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 11
    for xs, gs in rows:
        x, want = float(xs), float(gs)
        got = oracle.act(x, GELU)
        # the cancellation in 1 + tanh(u) for negative x costs absolute, not relative, accuracy
        assert abs(got - want) <= 4e-16 * max(abs(x), 1e-3), (x, got, want)
        # and through the whole function: K = 1, B = [1], no bias
        y = run(enc([x], F32), enc([1.0], F32), None, 1, 1, 1, F32, GELU)
        assert abs(y[0, 0] - want) <= 4e-16 * max(abs(x), 1e-3)


def test_gelu_through_the_gemm():
    xs = np.array([-2.0, -1.0, -0.5, 0.5, 1.0, 2.0, 3.0])
    y = run(enc(xs[:, None], F32), enc([[1.0]], F32), None, len(xs), 1, 1, F32, GELU)
    lib = torch.nn.functional.gelu(torch.from_numpy(xs), approximate="tanh").numpy()
    assert np.abs(y[:, 0] - lib).max() < 1e-15


def test_sigmoid_closed_forms_and_library():
    SIG = oracle.ACT_SIGMOID
    assert oracle.act(0.0, SIG) == 0.5
    xs = np.linspace(-12.0, 12.0, 481)
    s = np.array([oracle.act(x, SIG) for x in xs])
    sm = np.array([oracle.act(-x, SIG) for x in xs])
    assert np.allclose(s + sm, 1.0, rtol=0, atol=5e-16)          # sigmoid(x) + sigmoid(-x) = 1
    assert np.all(np.diff(s) > 0) and 0.0 < s[0] < 1e-5 and 1 - 1e-5 < s[-1] < 1.0
    assert abs(oracle.act(math.log(3.0), SIG) - 0.75) < 1e-15    # e^x / (1 + e^x) at x = ln 3
    lib = torch.sigmoid(torch.from_numpy(xs)).numpy()
    assert np.abs(s - lib).max() < 1e-15
    # through the GEMM: K = 1, B = [1]
    y = run(enc(np.array([[-2.0], [0.0], [2.0]]), F32), enc([[1.0]], F32), None, 3, 1, 1, F32, SIG)
    assert np.abs(y[:, 0] - torch.sigmoid(torch.tensor([-2.0, 0.0, 2.0], dtype=torch.float64)).numpy()).max() < 1e-15


# ---------------------------------------------------------------- rounding helpers

def test_bf16_round_ties_to_even():
    assert oracle.bf16_from_double(1.0 + 2.0**-8) == 0x3F80          # tie -> even (1.0)
    assert oracle.bf16_from_double(1.0 + 3 * 2.0**-8) == 0x3F82      # tie -> even (1.015625)
    assert oracle.bf16_to_double(0x3F82) == 1.015625
    assert oracle.bf16_from_double(1.0 + 2.0**-8 + 2.0**-40) == 0x3F81   # just above a tie
    assert oracle.bf16_from_double(-(1.0 + 2.0**-8)) == 0xBF80
    assert oracle.bf16_from_double(255.5) == 0x4380                  # mantissa carry: 256
    assert oracle.bf16_from_double(3.0e38 * 2) == 0x7F80             # overflow -> inf
    assert oracle.bf16_from_double(2.0**-133) == 0x0001              # smallest subnormal
    assert oracle.bf16_from_double(2.0**-134) == 0x0000              # tie -> even (0)
    assert oracle.bf16_from_double(3 * 2.0**-134) == 0x0002          # tie -> even (2)


def test_bf16_all_patterns_round_trip():
    for bits in range(0x10000):
        if (bits & 0x7F80) == 0x7F80 and (bits & 0x7F):
            continue  # NaN payloads
        assert oracle.bf16_from_double(oracle.bf16_to_double(bits)) == bits


def test_bf16_rounding_matches_library_conversion():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-30, 30, 20000),
                        rng.standard_normal(2000) * 1e-39]).astype(np.float32)
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    mine = oracle.round_to_dtype(x.astype(np.float64), BF16)
    neg_zero = mine != lib
    assert np.all(lib[neg_zero] == 0x8000) and np.all(mine[neg_zero] == 0)   # -0 is mapped to +0
    # and the input generator's own rounding agrees with both
    gen = synth.round_to_bf16_bits(x.astype(np.float64))
    assert np.array_equal(gen, lib)


def test_f32_rounding_matches_numpy():
    rng = np.random.default_rng(6)
    x = rng.standard_normal(10000) * 10.0 ** rng.integers(-20, 20, 10000)
    assert np.array_equal(oracle.round_to_dtype(x, F32), x.astype(np.float32))


# ---------------------------------------------------------------- whole function vs an fp64 library routine

def lib_reference(c):
    A = torch.from_numpy(oracle.widen(c.A, c.dtype)).view(c.M, c.K)
    B = torch.from_numpy(oracle.widen(c.B, c.dtype)).view(c.K, c.N)
    b = torch.from_numpy(oracle.widen(c.bias, c.dtype))
    z = A @ B + b
    if c.act == RELU:
        z = torch.relu(z)
    elif c.act == GELU:
        z = torch.nn.functional.gelu(z, approximate="tanh")
    return z.numpy()


@pytest.mark.parametrize("name,M,N,K", [("c1", 256, 256, 256), ("c1", 33, 70, 129), ("c2", 1, 512, 1024),
                                         ("c3", 16, 640, 768), ("c4", 96, 160, 320), ("c5", 64, 128, 2048)])
def test_oracle_agrees_with_fp64_library_gemm(name, M, N, K):
    c = synth.make_case(name, M=M, N=N, K=K)
    y = run(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act)
    ref = lib_reference(c)
    assert np.abs(y - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())
    assert np.abs(ref).max() > 0.5


def test_thread_count_does_not_change_the_result():
    c = synth.make_case("c4", M=37, N=64, K=256)
    y1 = run(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act, nthreads=1)
    y5 = run(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act, nthreads=5)
    assert np.array_equal(y1, y5)


def test_sampled_oracle_matches_library_on_the_sampled_entries():
    c = synth.make_case("c5", M=48, N=96, K=512)
    rows = np.array([0, 5, 17, 47])
    cols = np.array([95, 0, 33, 64, 7])
    ys = oracle.gemm_epilogue_sampled(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act, rows, cols)
    ref = lib_reference(c)[np.ix_(rows, cols)]
    assert np.abs(ys - ref).max() <= 1e-12 * np.abs(ref).max()
    with pytest.raises(RuntimeError):
        oracle.gemm_epilogue_sampled(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act, [48], [0])


# ---------------------------------------------------------------- metamorphic relations

@pytest.mark.parametrize("act", [NONE, RELU])
def test_power_of_two_scaling_is_exact(act):
    c = synth.make_case("c1", M=9, N=14, K=40)
    y = run(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, act)
    y8 = run(c.A * np.float32(8.0), c.B, c.bias * np.float32(8.0), c.M, c.N, c.K, c.dtype, act)
    assert np.array_equal(y8, 8.0 * y)


def test_row_and_column_permutation_equivariance():
    c = synth.make_case("c4", M=10, N=16, K=64)
    y = run(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act)
    rp = np.random.default_rng(1).permutation(c.M)
    cp = np.random.default_rng(2).permutation(c.N)
    Ap = c.A.reshape(c.M, c.K)[rp]
    yr = run(Ap, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act)
    assert np.array_equal(yr, y[rp])
    Bp = c.B.reshape(c.K, c.N)[:, cp]
    yc = run(c.A, Bp, c.bias[cp], c.M, c.N, c.K, c.dtype, c.act)
    assert np.array_equal(yc, y[:, cp])


def test_empty_reduction_gives_activated_bias():
    y = run(np.zeros(0, np.float32), np.zeros(0, np.float32), enc([1.0, -1.0], F32), 3, 2, 0, F32, RELU)
    assert np.array_equal(y, np.tile([1.0, 0.0], (3, 1)))


# ---------------------------------------------------------------- the input generator (no method arithmetic)

def test_generator_is_reproducible_and_chunk_independent():
    a = synth.normal(0, 1, 1000, 0.1, BF16)
    b = synth.normal(0, 1, 5_000_000, 0.1, BF16)    # spans several chunks and threads
    assert np.array_equal(a, b[:1000])
    assert not np.array_equal(synth.normal(1, 1, 1000, 0.1, BF16), a)
    assert not np.array_equal(synth.normal(0, 0, 1000, 0.1, BF16), a)


def test_generator_distributions():
    n = 2_000_000
    z = synth.bf16_bits_to_f64(synth.normal(0, 0, n, 0.125, BF16))
    assert abs(z.mean()) < 5e-4 and abs(z.std() - 0.125) < 5e-4
    u = synth.uniform(0, 2, n, -1.0, 1.0, F32).astype(np.float64)
    assert u.min() >= -1.0 and u.max() < 1.0 and abs(u.mean()) < 3e-3 and abs(u.std() - 1 / math.sqrt(3)) < 1e-3
    ub = synth.bf16_bits_to_f64(synth.uniform(0, 2, n, -0.1, 0.1, BF16))
    assert ub.min() >= -0.1 - 1e-3 and ub.max() <= 0.1 + 1e-3 and abs(ub.mean()) < 3e-4
    o = synth.bf16_bits_to_f64(synth.normal(0, 0, n, 0.1, BF16, outlier_prob=0.01))
    frac = np.mean(np.abs(o) == 8.0)
    assert 0.009 < frac < 0.011 and abs(np.mean(o[np.abs(o) == 8.0] > 0) - 0.5) < 0.02


def test_named_workloads_have_the_stated_shapes():
    want = {"c1": (256, 256, 256), "c2": (1, 8192, 8192), "c3": (16, 14336, 4096),
            "c4": (4096, 4096, 4096), "c5": (8192, 8192, 16384)}
    for k, v in want.items():
        assert synth.WORKLOADS[k][:3] == v
    c = synth.make_case("c3", N=64, K=128)
    assert c.M == 16 and not c.bias.any() and c.act == RELU
    assert c.algorithmic_bytes == 2 * (16 * 128 + 128 * 64 + 64 + 16 * 64) and c.flops == 2 * 16 * 64 * 128

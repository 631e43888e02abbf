"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs -- element by element at sizes the oracle finishes in seconds (several
tiles plus ragged tails, every variant forced in turn), bit-exact on integer-valued
inputs, and on sampled outputs at the five full-size workloads."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2602_12305_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

F32, BF16 = synth.F32, synth.BF16
NONE, RELU, GELU = synth.ACT_NONE, synth.ACT_RELU, synth.ACT_GELU_TANH
V = binding


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(0)
    yield h
    h.destroy()


@pytest.fixture(autouse=True)
def _auto_variant(handle):
    handle.force_variant(V.VARIANT_AUTO)
    yield
    handle.force_variant(V.VARIANT_AUTO)


def parity(handle, case, variant=None, what=""):
    if variant is not None:
        handle.force_variant(variant)
    bits, y = H.run_case(handle, case)
    H.check_tolerance(y, H.oracle_full(case), case.dtype, what or f"{case.name} {case.M}x{case.N}x{case.K}")
    return bits


# ---------------------------------------------------------------- every variant, small and ragged shapes

@pytest.mark.parametrize("name,M,N,K", [("c1", 1, 1, 1), ("c1", 3, 5, 7), ("c1", 65, 130, 33), ("c1", 200, 300, 150),
                                         ("c4", 1, 1, 1), ("c4", 3, 5, 7), ("c4", 65, 130, 33), ("c2", 1, 257, 1000)])
@pytest.mark.parametrize("act", [NONE, RELU, GELU])
def test_generic_variant(handle, name, M, N, K, act):
    parity(handle, synth.make_case(name, M=M, N=N, K=K, act=act), V.VARIANT_GENERIC)


@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (8, 12, 20), (260, 132, 516), (37, 64, 4), (130, 260, 1028),
                                   (1000, 1280, 96),      # >= 148 tiles of 64x64
                                   (1664, 1536, 72)])     # >= 148 tiles of 128x128
@pytest.mark.parametrize("act", [RELU, GELU])
def test_f32_tiled_variant(handle, M, N, K, act):
    parity(handle, synth.make_case("c1", M=M, N=N, K=K, act=act), V.VARIANT_F32_TILED)


@pytest.mark.parametrize("M,N,K", [(1, 512, 1024), (1, 264, 100), (2, 1032, 333), (3, 520, 777), (4, 8192, 300),
                                   (1, 8, 1), (4, 40000, 64)])
@pytest.mark.parametrize("act", [NONE, GELU])
def test_gemv_variant(handle, M, N, K, act):
    parity(handle, synth.make_case("c2", M=M, N=N, K=K, act=act), V.VARIANT_GEMV_SPLITK)


@pytest.mark.parametrize("M,N,K", [(1, 512, 1024), (1, 132, 100), (2, 1028, 333), (3, 516, 777), (4, 4096, 300),
                                   (1, 4, 1), (1, 8192, 8192)])
@pytest.mark.parametrize("act", [RELU, GELU])
def test_gemv_variant_fp32(handle, M, N, K, act):
    c = synth.make_case("c1", M=M, N=N, K=K, act=act)
    assert handle.select_variant(M, N, K, F32) == V.VARIANT_GEMV_SPLITK
    parity(handle, c, V.VARIANT_GEMV_SPLITK)


@pytest.mark.parametrize("M,N,K", [(16, 1160, 1096),     # 180 units over 148 CTAs: tiles split mid-K
                                   (16, 20480, 64),      # one K block per tile: every segment whole
                                   (1, 1024, 2048), (5, 136, 8), (17, 392, 520), (33, 1288, 264), (64, 2056, 712),
                                   (100, 520, 1096), (128, 1160, 328)])
@pytest.mark.parametrize("act", [RELU, GELU])
def test_skinny_variant(handle, M, N, K, act):
    parity(handle, synth.make_case("c3", M=M, N=N, K=K, act=act), V.VARIANT_SKINNY_UMMA)


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 256, 512), (300, 520, 200), (130, 264, 72), (1, 8, 8),
                                   (1024, 1024, 512),     # 32 tiles: each cut into 2 K slices
                                   (256, 520, 4096),      # 6 tiles, 8 K slices each
                                   (2432, 4096, 256),     # 304 tiles = 2 rounds + 8 tiles cut into 4 K slices
                                   (512, 14336, 520),     # 112 tiles on 74 CTA pairs: two rounds of whole tiles
                                   (2048, 4096, 128)])   # 256 tiles: more than one tile per CTA
@pytest.mark.parametrize("act", [RELU, GELU])
@pytest.mark.parametrize("variant", [V.VARIANT_UMMA, V.VARIANT_UMMA_2CTA])
def test_umma_variant(handle, M, N, K, act, variant):
    parity(handle, synth.make_case("c4", M=M, N=N, K=K, act=act), variant)


@pytest.mark.parametrize("M,N,K", [(256, 256, 64),        # one tile, one K block: no split possible
                                   (200, 520, 1096),      # 3 tiles, ragged everywhere; up to 4 K slices
                                   (100, 264, 2048),      # M <= 128: the second CTA of every pair has no rows
                                   (130, 1288, 520),      # two rows in the second CTA
                                   (512, 776, 1032),      # two tile rows
                                   (65, 4096, 4096),      # 16 tiles: clusters of 8 where the device holds 16 of them
                                   (256, 8192, 1024)])    # 32 tiles
@pytest.mark.parametrize("act", [RELU, GELU])
@pytest.mark.parametrize("split_max", [1, 2, 4])
def test_streaming_pair_variant(handle, M, N, K, act, split_max):
    handle.set_option(V.OPT_PAIR_SPLIT_MAX, split_max)
    try:
        parity(handle, synth.make_case("c4", M=M, N=N, K=K, act=act), V.VARIANT_UMMA_2CTA_STREAM)
    finally:
        handle.set_option(V.OPT_PAIR_SPLIT_MAX, 8)


@pytest.mark.parametrize("M,N,K", [(128, 256, 64),        # one tile, one K block
                                   (128, 520, 1096),      # ragged columns and K, every lane of both halves live
                                   (100, 264, 2048),      # rows 64..99 in the second CTA
                                   (64, 1288, 520),       # the second CTA of every pair has no rows
                                   (33, 776, 4096),
                                   (5, 8, 8),
                                   (96, 8192, 1024)])     # 32 tiles
@pytest.mark.parametrize("act", [RELU, GELU])
@pytest.mark.parametrize("split_max", [1, 2, 4])
def test_streaming_pair_variant_half_height_tiles(handle, M, N, K, act, split_max):
    """M <= 128: 64 rows per CTA (tcgen05.mma.cta_group::2 with M = 128), on by default; the 256-row
    form on the same shapes is the comparison."""
    assert handle.get_option(V.OPT_PAIR_HALF_HEIGHT) == 1
    handle.set_option(V.OPT_PAIR_SPLIT_MAX, split_max)
    try:
        c = synth.make_case("c4", M=M, N=N, K=K, act=act)
        parity(handle, c, V.VARIANT_UMMA_2CTA_STREAM, "64 rows per CTA")
        handle.set_option(V.OPT_PAIR_HALF_HEIGHT, 0)
        parity(handle, c, V.VARIANT_UMMA_2CTA_STREAM, "128 rows per CTA")
    finally:
        handle.set_option(V.OPT_PAIR_SPLIT_MAX, 8)
        handle.set_option(V.OPT_PAIR_HALF_HEIGHT, 1)


@pytest.mark.parametrize("M,N,K", [(256, 128, 64),         # one narrow tile, one K block
                                   (200, 520, 1096),       # 256-row tiles, ragged everywhere
                                   (512, 392, 1032),       # two tile rows
                                   (128, 264, 2048),       # 128-row tiles: 32 columns per lane half and CTA
                                   (100, 776, 1096),
                                   (64, 4096, 1024),       # 32 narrow tiles
                                   (33, 136, 4096)])
@pytest.mark.parametrize("act", [RELU, GELU])
@pytest.mark.parametrize("split_max", [1, 2, 4])
def test_streaming_pair_variant_narrow_tiles(handle, M, N, K, act, split_max):
    """128-column tiles (64 columns of B per CTA), forced through the tile-width option, with one, two
    and four CTA pairs per tile where the shape allows them."""
    handle.set_option(V.OPT_PAIR_SPLIT_MAX, split_max)
    handle.set_option(V.OPT_PAIR_TILE_WIDTH, 128)
    try:
        parity(handle, synth.make_case("c4", M=M, N=N, K=K, act=act), V.VARIANT_UMMA_2CTA_STREAM, "128-column tiles")
    finally:
        handle.set_option(V.OPT_PAIR_SPLIT_MAX, 8)
        handle.set_option(V.OPT_PAIR_TILE_WIDTH, 0)


@pytest.mark.parametrize("M,N,K", [(128, 776, 1024), (384, 520, 2048), (100, 2056, 4096)])
@pytest.mark.parametrize("width", [128, 256])
def test_streaming_pair_variant_integer_inputs_either_width(handle, M, N, K, width):
    handle.set_option(V.OPT_PAIR_TILE_WIDTH, width)
    try:
        c = synth.integer_case(M, N, K, BF16, RELU, seed=13)
        handle.force_variant(V.VARIANT_UMMA_2CTA_STREAM)
        bits, _ = H.run_case(handle, c)
        H.check_bit_exact(bits, H.oracle_full(c), BF16, f"cluster kernel, {width}-column tiles, {M}x{N}x{K}")
    finally:
        handle.set_option(V.OPT_PAIR_TILE_WIDTH, 0)


def test_streaming_pair_variant_refuses_more_tiles_than_clusters(handle):
    handle.force_variant(V.VARIANT_UMMA_2CTA_STREAM)
    c = synth.make_case("c4", M=2048, N=4096, K=64)          # 128 tiles
    A, B = H.to_device(c.A, c.dtype, (c.M, c.K)), H.to_device(c.B, c.dtype, (c.K, c.N))
    with pytest.raises(binding.OptimlError) as e:
        handle.gemm_epilogue(A, B, None, c.act)
    assert e.value.code == binding.ERR_UNSUPPORTED


def test_null_bias_and_act_none(handle):
    for variant, name, shape in ((V.VARIANT_F32_TILED, "c1", (64, 64, 64)), (V.VARIANT_GEMV_SPLITK, "c2", (1, 512, 512)),
                                 (V.VARIANT_SKINNY_UMMA, "c3", (16, 512, 512)), (V.VARIANT_UMMA, "c4", (256, 512, 256)),
                                 (V.VARIANT_UMMA_2CTA, "c4", (256, 512, 256)),
                                 (V.VARIANT_UMMA_2CTA_STREAM, "c4", (256, 512, 1024)),
                                 (V.VARIANT_GENERIC, "c4", (50, 60, 70))):
        c = synth.make_case(name, M=shape[0], N=shape[1], K=shape[2], act=NONE)
        c.bias = None
        parity(handle, c, variant)


@pytest.mark.parametrize("variant,name,M,N,K", [(V.VARIANT_GENERIC, "c1", 70, 90, 65), (V.VARIANT_GENERIC, "c4", 70, 90, 65),
                                                (V.VARIANT_F32_TILED, "c1", 260, 132, 516),
                                                (V.VARIANT_GEMV_SPLITK, "c2", 1, 1032, 2048),
                                                (V.VARIANT_SKINNY_UMMA, "c3", 16, 1160, 1096),
                                                (V.VARIANT_UMMA, "c4", 300, 520, 200),
                                                (V.VARIANT_UMMA_2CTA, "c4", 300, 520, 1096),
                                                (V.VARIANT_UMMA_2CTA_STREAM, "c4", 300, 520, 1096)])
def test_sigmoid_epilogue(handle, variant, name, M, N, K):
    parity(handle, synth.make_case(name, M=M, N=N, K=K, act=synth.ACT_SIGMOID), variant)


# ---------------------------------------------------------------- integer-valued inputs: bit-exact

@pytest.mark.parametrize("variant,dtype,M,N,K", [
    (V.VARIANT_GENERIC, F32, 70, 90, 300), (V.VARIANT_GENERIC, BF16, 70, 90, 300),
    (V.VARIANT_F32_TILED, F32, 96, 160, 512), (V.VARIANT_GEMV_SPLITK, BF16, 1, 1024, 4096),
    (V.VARIANT_GEMV_SPLITK, F32, 1, 1028, 4096), (V.VARIANT_GEMV_SPLITK, F32, 3, 260, 1000),
    (V.VARIANT_GEMV_SPLITK, BF16, 4, 520, 1000), (V.VARIANT_SKINNY_UMMA, BF16, 16, 1160, 1096),
    (V.VARIANT_SKINNY_UMMA, BF16, 48, 648, 2048), (V.VARIANT_UMMA, BF16, 384, 776, 1024),
    (V.VARIANT_UMMA_2CTA, BF16, 384, 776, 1024), (V.VARIANT_UMMA_2CTA, BF16, 1000, 520, 320),
    (V.VARIANT_UMMA_2CTA_STREAM, BF16, 384, 776, 1024), (V.VARIANT_UMMA_2CTA_STREAM, BF16, 100, 2056, 4096),
    (V.VARIANT_UMMA_2CTA_STREAM, BF16, 128, 776, 1024)])
@pytest.mark.parametrize("act", [NONE, RELU])
def test_integer_inputs_are_bit_exact(handle, variant, dtype, M, N, K, act):
    c = synth.integer_case(M, N, K, dtype, act, seed=11)
    handle.force_variant(variant)
    bits, _ = H.run_case(handle, c)
    H.check_bit_exact(bits, H.oracle_full(c), dtype, f"{binding.variant_name(variant)} {M}x{N}x{K}")


def test_permutation_B_on_the_tensor_core_path(handle):
    # B = permutation matrix: Y's columns are A's columns permuted, exactly (catches a
    # transposed or mis-swizzled operand on the MMA paths).
    M, K = 256, 512
    c = synth.integer_case(M, K, K, BF16, NONE, seed=2)
    perm = np.random.default_rng(0).permutation(K)
    Bm = np.zeros((K, K))
    Bm[perm, np.arange(K)] = 1.0
    c.B = synth.round_to_bf16_bits(Bm).reshape(-1)
    c.bias = None
    for variant in (V.VARIANT_UMMA, V.VARIANT_UMMA_2CTA, V.VARIANT_SKINNY_UMMA, V.VARIANT_GENERIC):
        if variant == V.VARIANT_SKINNY_UMMA:
            c2 = synth.Case("perm", 64, K, K, BF16, NONE, c.A[:64 * K], c.B, None)
        else:
            c2 = c
        handle.force_variant(variant)
        _, y = H.run_case(handle, c2)
        A = oracle.widen(c2.A, BF16).reshape(c2.M, K)
        assert np.array_equal(y, A[:, perm])


# ---------------------------------------------------------------- the five full-size workloads

def sample_indices(n, tile, count, seed):
    """Indices covering every residue modulo `tile`, the first and last tile, plus random ones."""
    rng = np.random.default_rng(seed)
    base = (np.arange(tile) + tile * rng.integers(0, max(1, n // tile), tile)) % n
    extra = rng.integers(0, n, max(0, count - tile))
    edge = np.array([0, 1, n - 2, n - 1, min(n - 1, tile - 1), min(n - 1, tile)])
    return np.unique(np.concatenate([base, extra, edge]))


def test_c1_full(handle):
    c = synth.make_case("c1")
    assert handle.select_variant(c.M, c.N, c.K, c.dtype) == V.VARIANT_F32_TILED
    parity(handle, c)


@pytest.mark.parametrize("sigma", [None, 8192 ** -0.5])
def test_c2_full(handle, sigma):
    c = synth.make_case("c2", sigma=sigma)
    assert handle.select_variant(c.M, c.N, c.K, c.dtype) in (V.VARIANT_GEMV_SPLITK, V.VARIANT_SKINNY_UMMA)
    parity(handle, c)
    parity(handle, c, V.VARIANT_GEMV_SPLITK)
    parity(handle, c, V.VARIANT_SKINNY_UMMA)


def test_c3_full(handle):
    c = synth.make_case("c3")
    assert handle.select_variant(c.M, c.N, c.K, c.dtype) == V.VARIANT_SKINNY_UMMA
    bits = parity(handle, c)
    bits2, _ = H.run_case(handle, c)
    assert np.array_equal(bits, bits2), "stream-K reduction is not reproducible"


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_c4_c5_sampled(handle, name):
    c = synth.make_case(name)
    assert handle.select_variant(c.M, c.N, c.K, c.dtype) == V.VARIANT_UMMA_2CTA
    bits, y = H.run_case(handle, c)
    rows = sample_indices(c.M, 128, 160, 1)
    cols = sample_indices(c.N, 256, 288, 2)
    ref = oracle.gemm_epilogue_sampled(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act, rows, cols)
    H.check_tolerance(y[np.ix_(rows, cols)], ref, c.dtype, f"{name} sampled {len(rows)}x{len(cols)}")
    # a few complete rows and columns as well
    frows = np.array([0, c.M // 2 + 3, c.M - 1])
    ref_r = oracle.gemm_epilogue_sampled(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act, frows, np.arange(c.N))
    H.check_tolerance(y[frows], ref_r, c.dtype, f"{name} full rows")
    fcols = np.array([0, c.N // 2 + 5, c.N - 1])
    ref_c = oracle.gemm_epilogue_sampled(c.A, c.B, c.bias, c.M, c.N, c.K, c.dtype, c.act, np.arange(c.M), fcols)
    H.check_tolerance(y[:, fcols], ref_c, c.dtype, f"{name} full columns")
    assert np.isfinite(y).all()
    # properties that hold at any size: ReLU output is non-negative; results are reproducible
    if c.act == RELU:
        assert (y >= 0).all()
    bits2, _ = H.run_case(handle, c)
    assert np.array_equal(bits, bits2)


@pytest.mark.parametrize("M,N,K,variant", [
    (256, 8192, 8192, V.VARIANT_UMMA_2CTA_STREAM),      # 32 tiles, two CTA pairs per tile: the exchange between the pairs
    (128, 8192, 8192, V.VARIANT_UMMA_2CTA_STREAM),      # the same with 128-row tiles, 64 rows per CTA
    (96, 14336, 4096, V.VARIANT_UMMA_2CTA_STREAM),      # 128-row tiles, one pair per tile, rows 64..95 in the second CTA
    (256, 14336, 4096, V.VARIANT_UMMA_2CTA_STREAM),     # 56 tiles, one pair per tile
    (512, 8192, 8192, V.VARIANT_UMMA_2CTA_STREAM),      # two rows of tiles
    (512, 14336, 4096, V.VARIANT_UMMA_2CTA)])           # persistent pairs: two rounds of whole tiles, the second half empty
def test_crossover_shapes_on_sampled_outputs(handle, M, N, K, variant):
    """The shapes of the dispatcher's crossover table at full size, as the benchmark launches them."""
    c = synth.make_case("c4", M=M, N=N, K=K)
    assert handle.select_variant(M, N, K, c.dtype) == variant
    bits, y = H.run_case(handle, c)
    rows = sample_indices(M, 128, 96, 1)
    cols = sample_indices(N, 256, 320, 2)
    ref = oracle.gemm_epilogue_sampled(c.A, c.B, c.bias, M, N, K, c.dtype, c.act, rows, cols)
    H.check_tolerance(y[np.ix_(rows, cols)], ref, c.dtype, f"{M}x{N}x{K} sampled {len(rows)}x{len(cols)}")
    frows = np.array([0, M // 2 + 3, M - 1])
    ref_r = oracle.gemm_epilogue_sampled(c.A, c.B, c.bias, M, N, K, c.dtype, c.act, frows, np.arange(N))
    H.check_tolerance(y[frows], ref_r, c.dtype, "full rows")
    assert np.isfinite(y).all()
    bits2, _ = H.run_case(handle, c)
    assert np.array_equal(bits, bits2)


def _random_shapes(seed, count):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        dtype = BF16 if rng.random() < 0.7 else F32
        M = int(rng.choice([1, 2, 7, 16, 33, 64, 65, 100, 128, 129, 200, 256, 300, 513, 700]))
        N = int(rng.integers(1, 40)) * int(rng.choice([8, 8, 64, 72, 128])) + int(rng.choice([0, 0, 0, 1, 2, 4]))
        K = int(rng.integers(1, 40)) * int(rng.choice([8, 16, 64, 96])) + int(rng.choice([0, 0, 0, 1, 3, 4]))
        act = int(rng.choice([NONE, RELU, GELU, synth.ACT_SIGMOID]))
        out.append((dtype, M, N, K, act))
    return out


@pytest.mark.parametrize("dtype,M,N,K,act", _random_shapes(2024, 60))
def test_random_shapes_through_the_dispatcher(handle, dtype, M, N, K, act):
    """Whatever the dispatcher picks for a shape (aligned or not, any regime), the result matches the oracle."""
    c = synth.make_case("c1" if dtype == F32 else "c4", M=M, N=N, K=K, act=act)
    parity(handle, c)


# ---------------------------------------------------------------- dispatcher, metamorphic relations, edge cases

def test_dispatcher_choices(handle):
    sel = handle.select_variant
    assert sel(256, 256, 256, F32) == V.VARIANT_F32_TILED
    assert sel(255, 255, 255, F32) == V.VARIANT_GENERIC
    assert sel(1, 8192, 8192, BF16) in (V.VARIANT_GEMV_SPLITK, V.VARIANT_SKINNY_UMMA)
    assert sel(16, 14336, 4096, BF16) == V.VARIANT_SKINNY_UMMA
    assert sel(4096, 4096, 4096, BF16) == V.VARIANT_UMMA_2CTA
    assert sel(8192, 8192, 16384, BF16) == V.VARIANT_UMMA_2CTA
    assert sel(128, 4096, 4096, BF16) == V.VARIANT_UMMA_2CTA_STREAM     # 16 tiles for 74 CTA pairs
    assert sel(256, 8192, 8192, BF16) == V.VARIANT_UMMA_2CTA_STREAM
    assert sel(32, 4096, 4096, BF16) == V.VARIANT_SKINNY_UMMA and sel(2, 4096, 4096, BF16) == V.VARIANT_SKINNY_UMMA
    assert sel(64, 14336, 4096, BF16) == V.VARIANT_SKINNY_UMMA          # every column tile whole in one CTA
    assert sel(64, 8192, 8192, BF16) == V.VARIANT_UMMA_2CTA_STREAM      # the skinny schedule would cut tiles along K
    assert sel(96, 14336, 4096, BF16) == V.VARIANT_UMMA_2CTA_STREAM     # above 64 rows the cluster kernel (64 rows per CTA)
    assert sel(130, 262, 100, BF16) == V.VARIANT_GENERIC         # N % 8 != 0 (large ones are re-pitched, then dispatched again)
    assert sel(0, 1, 1, BF16) == -1


@pytest.mark.parametrize("M,N,K", [(520, 516, 520),        # N ragged
                                   (520, 520, 516),        # K ragged
                                   (300, 1030, 1001),      # both ragged, odd K
                                   (300, 1031, 1000),      # odd N: rows of B and Y start on 2-byte boundaries only
                                   (64, 2052, 1100),       # lands on the skinny kernel
                                   (1100, 1028, 260)])
@pytest.mark.parametrize("act", [RELU, GELU])
def test_large_unaligned_bf16_shapes_take_the_fast_variants_through_padded_copies(handle, M, N, K, act):
    c = synth.make_case("c4", M=M, N=N, K=K, act=act)
    before = handle.launch_count()
    bits = parity(handle, c)
    assert handle.launch_count() - before >= 3          # copies in, the GEMM itself, copy out
    # the same bits a second time (buffers reused, nothing left over from the first call)
    bits2, _ = H.run_case(handle, c)
    assert np.array_equal(bits, bits2)


@pytest.mark.parametrize("M,N,K", [(520, 518, 520), (520, 520, 517), (300, 1030, 1001), (300, 1031, 1003), (1100, 1026, 260)])
def test_large_unaligned_fp32_shapes_take_the_tile_kernel_through_padded_copies(handle, M, N, K):
    c = synth.make_case("c1", M=M, N=N, K=K, act=GELU)
    before = handle.launch_count()
    bits = parity(handle, c)
    assert handle.launch_count() - before >= 3
    bits2, _ = H.run_case(handle, c)
    assert np.array_equal(bits, bits2)
    ci = synth.integer_case(M, N, K, F32, RELU, seed=3)
    bi, _ = H.run_case(handle, ci)
    H.check_bit_exact(bi, H.oracle_full(ci), F32, f"unaligned fp32 {M}x{N}x{K} through padded copies")


def test_padded_copies_keep_integer_cases_exact(handle):
    c = synth.integer_case(300, 1030, 1001, BF16, RELU, seed=5)
    bits, _ = H.run_case(handle, c)
    H.check_bit_exact(bits, H.oracle_full(c), BF16, "unaligned 300x1030x1001 through padded copies")
    c.bias = None
    bits, _ = H.run_case(handle, c)
    H.check_bit_exact(bits, H.oracle_full(c), BF16, "the same without bias")


def test_unaligned_shapes_and_pointers_fall_back_to_the_generic_kernel(handle):
    before = handle.launch_count()
    parity(handle, synth.make_case("c4", M=130, N=262, K=100))       # N % 8 != 0
    parity(handle, synth.make_case("c1", M=30, N=31, K=33))          # fp32, N % 4 != 0
    assert handle.launch_count() == before + 2
    # a 2-byte aligned (not 16-byte aligned) bf16 B pointer
    c = synth.make_case("c4", M=128, N=256, K=64)
    A = H.to_device(c.A, BF16, (c.M, c.K))
    Bbuf = torch.zeros(c.K * c.N + 8, dtype=torch.bfloat16, device="cuda:0")
    Bv = Bbuf[1:1 + c.K * c.N].view(c.K, c.N)
    Bv.copy_(H.to_device(c.B, BF16, (c.K, c.N)))
    bias = H.to_device(c.bias, BF16, (c.N,))
    Y = torch.empty(c.M, c.N, dtype=torch.bfloat16, device="cuda:0")
    rc = handle.gemm_epilogue_raw(A.data_ptr(), Bv.data_ptr(), bias.data_ptr(), Y.data_ptr(), c.M, c.N, c.K, BF16,
                                  c.act, torch.cuda.current_stream().cuda_stream)
    assert rc == binding.OK
    torch.cuda.synchronize()
    H.check_tolerance(oracle.widen(H.to_host_bits(Y, BF16), BF16), H.oracle_full(c), BF16, "unaligned B")


def test_error_codes(handle):
    x = torch.zeros(64, dtype=torch.float32, device="cuda:0")
    p = x.data_ptr()
    call = handle.gemm_epilogue_raw
    assert call(None, p, None, p, 1, 1, 1, F32, NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, None, 1, 1, 1, F32, NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, p, 0, 1, 1, F32, NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, p, 1, -3, 1, F32, NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, p, 1, 1, 2 ** 31, F32, NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, p, 1, 1, 1, 7, NONE) == binding.ERR_INVALID_ARG
    assert call(p, p, None, p, 1, 1, 1, F32, 9) == binding.ERR_INVALID_ARG
    assert call(p + 2, p, None, p + 32, 1, 1, 1, F32, NONE) == binding.ERR_ALIGNMENT
    assert call(p + 1, p, None, p + 32, 1, 1, 1, BF16, NONE) == binding.ERR_ALIGNMENT
    handle.force_variant(V.VARIANT_UMMA)
    assert call(p, p, None, p + 128, 2, 2, 2, F32, NONE) == binding.ERR_UNSUPPORTED
    handle.force_variant(V.VARIANT_GEMV_SPLITK)
    assert call(p, p, None, p + 128, 8, 8, 8, BF16, NONE) == binding.ERR_UNSUPPORTED     # M > 4
    handle.force_variant(V.VARIANT_AUTO)
    assert handle.get_last_status() == binding.OK
    with pytest.raises(binding.OptimlError):
        handle.force_variant(17)


@pytest.mark.parametrize("variant,name,M,N,K", [(V.VARIANT_F32_TILED, "c1", 96, 128, 256),
                                                (V.VARIANT_GEMV_SPLITK, "c2", 2, 1024, 2048),
                                                (V.VARIANT_SKINNY_UMMA, "c3", 16, 1160, 1096),
                                                (V.VARIANT_UMMA, "c4", 384, 512, 512),
                                                (V.VARIANT_UMMA_2CTA, "c4", 384, 512, 512)])
def test_metamorphic_relations(handle, variant, name, M, N, K):
    c = synth.make_case(name, M=M, N=N, K=K, act=RELU)
    handle.force_variant(variant)
    bits, y = H.run_case(handle, c)
    bits_again, _ = H.run_case(handle, c)
    assert np.array_equal(bits, bits_again), "same call, different bits"
    # permuting the rows of A permutes the rows of Y, bit for bit
    rp = np.random.default_rng(3).permutation(M)
    cp = synth.Case(c.name, M, N, K, c.dtype, c.act, c.A.reshape(M, K)[rp].reshape(-1), c.B, c.bias)
    bits_p, _ = H.run_case(handle, cp)
    assert np.array_equal(bits_p.reshape(M, N), bits.reshape(M, N)[rp])
    # scaling A and bias by 4 scales Y by 4 exactly (ReLU is positively homogeneous)
    if c.dtype == F32:
        c4 = synth.Case(c.name, M, N, K, c.dtype, c.act, c.A * np.float32(4), c.B, c.bias * np.float32(4))
    else:
        up = lambda b: np.where((b & 0x7FFF) == 0, b, b + np.uint16(2 << 7)).astype(np.uint16)   # exponent + 2
        c4 = synth.Case(c.name, M, N, K, c.dtype, c.act, up(c.A), c.B, up(c.bias))
    _, y4 = H.run_case(handle, c4)
    assert np.array_equal(y4, 4.0 * y)


def test_host_entry_point(handle):
    c = synth.make_case("c4", M=256, N=512, K=320)
    A = H.to_device(c.A, BF16, (c.M, c.K), "cpu").pin_memory()
    B = H.to_device(c.B, BF16, (c.K, c.N), "cpu").pin_memory()
    bias = H.to_device(c.bias, BF16, (c.N,), "cpu").pin_memory()
    Y = torch.full((c.M, c.N), float("nan"), dtype=torch.bfloat16).pin_memory()
    for _ in range(2):      # second call reuses the staging buffers
        handle.gemm_epilogue_host(A, B, bias, Y, c.act)
        H.check_tolerance(oracle.widen(H.to_host_bits(Y, BF16), BF16), H.oracle_full(c), BF16, "host entry point")


def test_many_shapes_back_to_back_leave_the_scratch_clean(handle):
    # split-K and stream-K kernels share arrival counters; interleave shapes and check all
    cases = [synth.make_case("c3", M=16, N=1160, K=1096), synth.make_case("c2", M=1, N=2048, K=4096),
             synth.make_case("c3", M=8, N=392, K=2056), synth.make_case("c2", M=3, N=520, K=1500)]
    refs = [H.oracle_full(c) for c in cases]
    for _ in range(3):
        for c, r in zip(cases, refs):
            _, y = H.run_case(handle, c)
            H.check_tolerance(y, r, c.dtype, "interleaved")


# ---------------------------------------------------------------- tuning options of the streaming kernels

def test_option_arguments(handle):
    for opt in range(V.OPT_COUNT):
        assert handle.get_option(opt) >= 0
    with pytest.raises(binding.OptimlError):
        handle.set_option(V.OPT_COUNT, 1)
    with pytest.raises(binding.OptimlError):
        handle.set_option(V.OPT_GEMV_PREFETCH_ROWS, -1)
    assert handle.get_option(V.OPT_COUNT) == -1


@pytest.mark.parametrize("name,M,N,K,variant", [("c2", 1, 2056, 3000, V.VARIANT_GEMV_SPLITK),
                                                 ("c2", 3, 520, 777, V.VARIANT_GEMV_SPLITK),
                                                 ("c3", 16, 1160, 1096, V.VARIANT_SKINNY_UMMA),
                                                 ("c3", 40, 2312, 4104, V.VARIANT_SKINNY_UMMA)])
def test_scheduling_options_leave_the_bits_alone(handle, name, M, N, K, variant):
    """Prefetch depth, ring depth and trigger point only reschedule the stream over B: every
    setting must match the oracle and give the very same bits; the stage height may move the
    K cuts of a split problem, so it is held to the tolerance only."""
    case = synth.make_case(name, M=M, N=N, K=K)
    saved = [handle.get_option(o) for o in range(V.OPT_COUNT)]
    try:
        ref_bits = {}
        for rows in (128, 192):
            for pf_rows, stages, early, late in ((0, 0, 0, 0), (1, 2, 1, 1), (64, 3, 5, 0), (100000, 9, 1000, 1)):
                handle.set_option(V.OPT_GEMV_PREFETCH_ROWS, pf_rows)
                handle.set_option(V.OPT_SKINNY_STAGE_ROWS, rows)
                handle.set_option(V.OPT_SKINNY_RING_STAGES, stages)
                handle.set_option(V.OPT_SKINNY_PREFETCH_EARLY, early)
                handle.set_option(V.OPT_SKINNY_LATE_TRIGGER, late)
                bits = parity(handle, case, variant, what=f"{name} {M}x{N}x{K} options {(rows, pf_rows, stages, early, late)}")
                assert np.array_equal(ref_bits.setdefault(rows, bits), bits)
    finally:
        for o, v in enumerate(saved):
            handle.set_option(o, v)


# ---------------------------------------------------------------- stream order across the dependency wait

@pytest.mark.parametrize("name,M,N,K,variant", [("c2", 1, 2056, 3000, V.VARIANT_GEMV_SPLITK),
                                                 ("c3", 16, 1160, 1096, V.VARIANT_SKINNY_UMMA),
                                                 ("c1", 64, 96, 256, V.VARIANT_F32_TILED),
                                                 ("c4", 300, 520, 264, V.VARIANT_UMMA_2CTA)])
def test_operands_written_just_before_the_call_are_seen(handle, name, M, N, K, variant):
    """The streaming kernels ask L2 for lines of B before they wait for the previous kernel in the
    stream.  That must never show stale data: B (and A, bias) are overwritten on the same stream
    immediately before each call, alternating between two contents, with no synchronisation in
    between, and every output must be the one of the contents written last."""
    cases = [synth.make_case(name, M=M, N=N, K=K, seed=s) for s in (0, 1)]
    refs = [H.oracle_full(c) for c in cases]
    dt = cases[0].dtype
    src = [(H.to_device(c.A, dt, (M, K)), H.to_device(c.B, dt, (K, N)), H.to_device(c.bias, dt, (N,))) for c in cases]
    A, B, bias = (torch.empty_like(x) for x in src[0])
    handle.force_variant(variant)
    outs = []
    for i in range(12):
        a, b, bb = src[i & 1]
        A.copy_(a)
        B.copy_(b)
        bias.copy_(bb)
        outs.append((i & 1, handle.gemm_epilogue(A, B, bias, cases[0].act)))
    torch.cuda.synchronize()
    assert handle.get_last_status() == binding.OK
    for which, Y in outs:
        y = oracle.widen(H.to_host_bits(Y, dt), dt)
        H.check_tolerance(y, refs[which], dt, f"{name} {M}x{N}x{K}, contents {which}")


def test_chained_calls_consume_the_previous_output(handle):
    """Y1 = act(A B1) feeds the next call as its A operand with nothing in between: the second
    kernel is resident while the first still runs and must wait for its output."""
    M, K1, N1, N2 = 16, 1096, 1160, 1288
    c1 = synth.make_case("c3", M=M, N=N1, K=K1, act=GELU)
    c2 = synth.make_case("c3", M=M, N=N2, K=N1, seed=3)
    A, B1, b1 = H.to_device(c1.A, BF16, (M, K1)), H.to_device(c1.B, BF16, (K1, N1)), H.to_device(c1.bias, BF16, (N1,))
    B2, b2 = H.to_device(c2.B, BF16, (N1, N2)), H.to_device(c2.bias, BF16, (N2,))
    results = []
    for _ in range(6):
        Y1 = handle.gemm_epilogue(A, B1, b1, GELU)
        Y2 = handle.gemm_epilogue(Y1, B2, b2, RELU)
        results.append((Y1, Y2))
    torch.cuda.synchronize()
    assert handle.get_last_status() == binding.OK
    for Y1, Y2 in results:
        y1_bits = H.to_host_bits(Y1, BF16)
        H.check_tolerance(oracle.widen(y1_bits, BF16), H.oracle_full(c1), BF16, "first call")
        ref2 = oracle.gemm_epilogue(y1_bits.reshape(-1), c2.B, c2.bias, M, N2, N1, BF16, RELU)
        H.check_tolerance(oracle.widen(H.to_host_bits(Y2, BF16), BF16), ref2, BF16, "second call on the first call's output")

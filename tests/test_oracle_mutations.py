"""Are the oracle's pins sharp?  Each case below plants one plausible mistake in a COPY of
the oracle's C source (a dropped term, a wrong index, a wrong sign or constant, a wrong
rounding rule), builds it, swaps it in for the real library and checks that at least one
of the pins in test_oracle_pins.py fails.  CPU only; the mistakes live in the oracle copy."""
import ctypes
import os
import subprocess

import pytest

from oracle import oracle
from tests import test_oracle_pins as P

SRC = os.path.join(os.path.dirname(os.path.abspath(oracle.__file__)), "gemm_epilogue_oracle.c")

F32, BF16 = oracle.F32, oracle.BF16
NONE, RELU = oracle.ACT_NONE, oracle.ACT_RELU

MUTATIONS = {
    "bias dropped": ("acc[c] = oracle_act(acc[c] + b, j->act);", "acc[c] = oracle_act(acc[c], j->act);"),
    "bias indexed by row": ("const double b = j->bias ? load_elem(j->bias, n, j->dtype) : 0.0;",
                            "const double b = j->bias ? load_elem(j->bias, m % j->N, j->dtype) : 0.0;"),
    "A read with reversed k": ("load_elem(j->A, m * j->K + k, j->dtype)", "load_elem(j->A, m * j->K + (j->K - 1 - k), j->dtype)"),
    "last k skipped": ("for (int64_t k = 0; k < j->K; ++k) {", "for (int64_t k = 0; k + 1 < j->K; ++k) {"),
    "fp32 accumulator": ("acc[c] += a * load_elem(j->B, k * j->N + n, j->dtype);",
                         "acc[c] = (double)(float)(acc[c] + a * load_elem(j->B, k * j->N + n, j->dtype));"),
    "ReLU keeps negatives": ("return x > 0.0 ? x : 0.0;", "return x < 0.0 ? x : 0.0;"),
    "GELU cubic coefficient": ("0.044715 * x * x * x", "0.0447 * x * x * x"),
    "GELU erf form": ("return 0.5 * x * (1.0 + tanh(c * (x + 0.044715 * x * x * x)));",
                      "(void)c; return 0.5 * x * (1.0 + erf(x / 1.4142135623730951));"),
    "GELU sqrt(2/pi) constant": ("const double c = 0.7978845608028654;", "const double c = 0.7978;"),
    "bf16 ties round up": ("if (rem > half || (rem == half && (kept & 1))) kept += 1;", "if (rem >= half) kept += 1;"),
    "bf16 truncates": ("if (rem > half || (rem == half && (kept & 1))) kept += 1;", "(void)half; (void)rem;"),
    "sampled columns ignored": ("const int64_t n = j->cols ? j->cols[c] : c;\n                acc[c] += a",
                                "const int64_t n = c;\n                acc[c] += a"),
}


def run_pins():
    """A representative subset of the pins, called directly (parametrised ones with their arguments)."""
    for dt in (F32, BF16):
        P.test_identity_B_returns_A_plus_bias(dt)
        P.test_permutation_B_permutes_columns(dt)
        P.test_rank_one_closed_form(dt)
        for act in (NONE, RELU):
            P.test_integer_inputs_match_exact_integer_arithmetic(dt, act)
    P.test_selector_B_rectangular()
    P.test_zero_A_gives_activated_bias_on_every_row()
    P.test_relu_fixed_points()
    P.test_gelu_tanh_invariants()
    P.test_gelu_tanh_is_the_tanh_form_not_erf()
    P.test_gelu_through_the_gemm()
    P.test_bf16_round_ties_to_even()
    P.test_bf16_rounding_matches_library_conversion()
    P.test_oracle_agrees_with_fp64_library_gemm("c1", 33, 70, 129)
    P.test_oracle_agrees_with_fp64_library_gemm("c4", 96, 160, 320)
    P.test_sampled_oracle_matches_library_on_the_sampled_entries()


@pytest.fixture
def swap_library(monkeypatch, tmp_path):
    def build_and_swap(source_text: str):
        c = tmp_path / "mutant.c"
        so = tmp_path / "libmutant.so"
        c.write_text(source_text)
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-o", str(so), str(c),
                        "-lm", "-lpthread"], check=True)
        real = oracle._load()
        lib = ctypes.CDLL(str(so))
        for name in ("oracle_gemm_epilogue", "oracle_gemm_epilogue_sampled", "oracle_round_to_dtype", "oracle_act",
                     "oracle_bf16_from_double", "oracle_bf16_to_double"):
            getattr(lib, name).argtypes = getattr(real, name).argtypes
            getattr(lib, name).restype = getattr(real, name).restype
        monkeypatch.setattr(oracle, "_lib", lib)
    return build_and_swap


def test_the_unmutated_copy_passes(swap_library):
    swap_library(open(SRC).read())
    run_pins()


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_a_planted_mistake_is_caught(name, swap_library):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation target for {name!r} not found in the oracle source"
    swap_library(text.replace(old, new))
    with pytest.raises((AssertionError, RuntimeError)):
        run_pins()

"""Pins for the attention oracle (paper: Prompts appendix, task 6).  None of the expected values
comes from the oracle itself: brute-force loops, closed forms, invariants and a library routine.
The same checks are then run against copies of the oracle with one mistake planted in each."""
import math
import os
import types

import numpy as np
import pytest
import torch

from oracle import mhsa_oracle

SRC = os.path.join(os.path.dirname(os.path.abspath(mhsa_oracle.__file__)), "mhsa_oracle.py")


def rnd(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


def brute_force(Q, K, V, n, d_model, h):
    """Element-by-element loops straight from the benchmark spec."""
    dk = d_model // h
    out = [[0.0] * d_model for _ in range(n)]
    for head in range(h):
        c0 = head * dk
        for i in range(n):
            s = [sum(Q[i][c0 + t] * K[j][c0 + t] for t in range(dk)) / math.sqrt(dk) for j in range(n)]
            e = [math.exp(x) for x in s]
            z = math.fsum(e)
            for t in range(dk):
                out[i][c0 + t] = math.fsum(e[j] * V[j][c0 + t] for j in range(n)) / z
    return np.array(out)


# ---------------------------------------------------------------- the pins, as functions of the module

def pin_brute_force(O):
    for (n, d_model, h, seed) in ((5, 6, 3, 1), (7, 8, 2, 2), (4, 4, 1, 3), (3, 6, 6, 4)):
        Q, K, V = rnd((n, d_model), seed), rnd((n, d_model), seed + 10), rnd((n, d_model), seed + 20)
        want = brute_force(Q.tolist(), K.tolist(), V.tolist(), n, d_model, h)
        np.testing.assert_allclose(O.mhsa(Q, K, V, n, d_model, h), want, rtol=1e-12, atol=1e-13)


def pin_zero_queries_average_the_values(O):
    n, d_model, h = 9, 12, 3
    K, V = rnd((n, d_model), 5), rnd((n, d_model), 6)
    got = O.mhsa(np.zeros((n, d_model)), K, V, n, d_model, h)
    np.testing.assert_allclose(got, np.tile(V.mean(axis=0), (n, 1)), rtol=1e-13, atol=1e-14)


def pin_single_key_returns_its_value(O):
    Q, K, V = rnd((1, 8), 7), rnd((1, 8), 8), rnd((1, 8), 9)
    np.testing.assert_allclose(O.mhsa(Q, K, V, 1, 8, 2), V, rtol=0, atol=1e-15)


def pin_two_keys_closed_form(O):
    # softmax over two scores is a logistic function of their difference; d_k = 4 with h = 2
    n, d_model, h = 2, 8, 2
    Q, K, V = rnd((n, d_model), 11), rnd((n, d_model), 12), rnd((n, d_model), 13)
    want = np.empty((n, d_model))
    for head in range(h):
        c = slice(4 * head, 4 * head + 4)
        for i in range(n):
            diff = (Q[i, c] @ K[1, c] - Q[i, c] @ K[0, c]) / 2.0            # sqrt(d_k) = 2
            w1 = 1.0 / (1.0 + math.exp(-diff))
            want[i, c] = V[0, c] + w1 * (V[1, c] - V[0, c])
    np.testing.assert_allclose(O.mhsa(Q, K, V, n, d_model, h), want, rtol=1e-12, atol=1e-14)


def pin_sharp_scores_select_one_row(O):
    # keys are the unit vectors; query r points at key perm[r] with a large gain
    dk, h = 8, 2
    n, d_model = dk, dk * h
    perm = np.array([3, 0, 7, 1, 6, 2, 5, 4])
    K = np.tile(np.eye(dk), (1, h))
    Q = 200.0 * K[perm]
    V = rnd((n, d_model), 14)
    np.testing.assert_allclose(O.mhsa(Q, K, V, n, d_model, h), V[perm], rtol=0, atol=1e-25)


def pin_library_attention(O):
    for (n, d_model, h, seed) in ((33, 64, 4, 21), (130, 96, 3, 22), (64, 128, 1, 23)):
        Q, K, V = rnd((n, d_model), seed), rnd((n, d_model), seed + 1), rnd((n, d_model), seed + 2, 3.0)
        dk = d_model // h
        t = [torch.from_numpy(x).reshape(n, h, dk).permute(1, 0, 2) for x in (Q, K, V)]
        want = torch.nn.functional.scaled_dot_product_attention(*t).permute(1, 0, 2).reshape(n, d_model).numpy()
        np.testing.assert_allclose(O.mhsa(Q, K, V, n, d_model, h), want, rtol=1e-11, atol=1e-12)


def pin_invariances(O):
    n, d_model, h = 17, 12, 3
    dk = d_model // h
    Q, K, V = rnd((n, d_model), 31), rnd((n, d_model), 32), rnd((n, d_model), 33)
    base = O.mhsa(Q, K, V, n, d_model, h)
    # the same vector added to every key shifts each row of scores by a constant
    np.testing.assert_allclose(O.mhsa(Q, K + rnd((1, d_model), 34), V, n, d_model, h), base, rtol=1e-11, atol=1e-12)
    # keys and values reordered together; queries reordered
    p = np.random.default_rng(35).permutation(n)
    np.testing.assert_allclose(O.mhsa(Q, K[p], V[p], n, d_model, h), base, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(O.mhsa(Q[p], K, V, n, d_model, h), base[p], rtol=1e-13, atol=1e-14)
    # outputs are convex combinations of the values, column by column
    assert (base <= V.max(axis=0) + 1e-12).all() and (base >= V.min(axis=0) - 1e-12).all()
    # a head sees only its own columns
    Q2, K2, V2 = Q.copy(), K.copy(), V.copy()
    for x in (Q2, K2, V2):
        x[:, dk:2 * dk] = rnd((n, dk), 36)
    other = O.mhsa(Q2, K2, V2, n, d_model, h)
    np.testing.assert_array_equal(other[:, :dk], base[:, :dk])
    np.testing.assert_array_equal(other[:, 2 * dk:], base[:, 2 * dk:])
    assert np.abs(other[:, dk:2 * dk] - base[:, dk:2 * dk]).max() > 1e-3
    # and equals single-head attention on those columns
    one = O.mhsa(Q[:, dk:2 * dk].copy(), K[:, dk:2 * dk].copy(), V[:, dk:2 * dk].copy(), n, dk, 1)
    np.testing.assert_allclose(base[:, dk:2 * dk], one, rtol=1e-13, atol=1e-14)


def pin_large_scores_stay_finite(O):
    n, d_model, h = 6, 8, 2
    Q, K, V = rnd((n, d_model), 41, 40.0), rnd((n, d_model), 42, 40.0), rnd((n, d_model), 43)
    got = O.mhsa(Q, K, V, n, d_model, h)            # scores of order 1e3: exp would overflow unshifted
    assert np.isfinite(got).all()
    assert (got <= V.max(axis=0) + 1e-12).all() and (got >= V.min(axis=0) - 1e-12).all()


def pin_row_subset_and_bf16_input(O):
    n, d_model, h = 40, 16, 2
    Q, K, V = rnd((n, d_model), 51), rnd((n, d_model), 52), rnd((n, d_model), 53)
    full = brute_force(Q.tolist(), K.tolist(), V.tolist(), n, d_model, h)
    rows = [39, 0, 17]
    np.testing.assert_allclose(O.mhsa(Q, K, V, n, d_model, h, rows=rows), full[rows], rtol=1e-12, atol=1e-13)
    # bf16 bit patterns: 1.0, -2.0, 0.099609375, 2^-126 * 1.5
    bits = np.array([0x3F80, 0xC000, 0x3DCC, 0x00C0], dtype=np.uint16)
    np.testing.assert_array_equal(O.widen(bits), np.array([1.0, -2.0, 0.099609375, 1.5 * 2.0 ** -126]))


PINS = [pin_brute_force, pin_zero_queries_average_the_values, pin_single_key_returns_its_value, pin_two_keys_closed_form,
        pin_sharp_scores_select_one_row, pin_library_attention, pin_invariances, pin_large_scores_stay_finite,
        pin_row_subset_and_bf16_input]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(mhsa_oracle)


# ---------------------------------------------------------------- planted mistakes

MUTATIONS = {
    "scale by sqrt(d_model)": ("/ np.sqrt(float(dk))", "/ np.sqrt(float(d_model))"),
    "no scale": ("/ np.sqrt(float(dk))", "/ 1.0"),
    "scale by d_k": ("/ np.sqrt(float(dk))", "/ float(dk)"),
    "softmax over queries": ("E / E.sum(axis=1, keepdims=True)", "E / E.sum(axis=0, keepdims=True)"),
    "no max subtraction": ("np.exp(S - S.max(axis=1, keepdims=True))", "np.exp(S)"),
    "interleaved heads": ("cols = slice(i * dk, (i + 1) * dk)", "cols = slice(i, d_model, h)"),
    "heads concatenated in the wrong order": ("out[:, cols] = ", "out[:, slice((h - 1 - i) * dk, (h - i) * dk)] = "),
    "keys and queries swapped": ("Qf[:, cols] @ Kf[:, cols].T", "Kf[:Qf.shape[0], cols] @ Qf[:, cols].T if Qf.shape[0] == Kf.shape[0] else Qf[:, cols] @ Kf[:, cols].T"),
    "values from the keys": ("softmax_rows(S) @ Vf[:, cols]", "softmax_rows(S) @ Kf[:, cols]"),
    "unnormalised": ("return E / E.sum(axis=1, keepdims=True)", "return E"),
    "rows ignored": ("Qf = Qf[np.asarray(rows, dtype=np.int64)]", "Qf = Qf[:len(rows)]"),
    "bf16 shifted wrongly": ("<< np.uint32(16)", "<< np.uint32(15)"),
    "last key dropped": ("softmax_rows(S) @ Vf[:, cols]", "softmax_rows(S[:, :max(1, n - 1)]) @ Vf[:max(1, n - 1), cols]"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch_planted_mistake(name):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, f"mutation site for {name!r} not found exactly once"
    mod = types.ModuleType("mhsa_oracle_mutant")
    exec(compile(src.replace(old, new), "mhsa_oracle_mutant", "exec"), mod.__dict__)
    caught = []
    for pin in PINS:
        try:
            with np.errstate(all="ignore"):
                pin(mod)
        except Exception:                       # an assertion, or the mutant breaking outright
            caught.append(pin.__name__)
    assert caught, f"no pin notices: {name}"

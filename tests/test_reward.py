"""The paper's reward (time term, proxy term with bottleneck-aware weights, guardrails, total)
pinned by hand arithmetic: closed forms, the weights table, and a worked example on the
numbers the paper prints for its own matrix-multiplication task.  CPU only."""
import math
import os

import pytest

from paper_2602_12305_b200 import reward as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_table1_matmul.txt")


def st(time=1.0, sm=50.0, dram=50.0, tex=50.0, db=100.0, l1=100.0, inst=100.0, regs=32.0, lmem=0.0):
    return W.State(time, sm, dram, tex, db, l1, inst, regs, lmem)


def test_time_reward_closed_forms():
    assert W.time_reward(5.0, 5.0) == 0.0
    assert W.time_reward(4.0, 0.0) == pytest.approx(math.tanh(0.40))          # all the time removed
    assert W.time_reward(4.0, 2.0) == pytest.approx(math.tanh(0.20))          # 2x faster
    assert W.time_reward(4.0, 8.0) == pytest.approx(-math.tanh(0.40))         # 2x slower
    assert -1.0 <= W.time_reward(1.0, 1e9) < -0.999999                         # bounded below by -1


def test_regime_uses_the_margin_of_7_5():
    assert W.regime(st(sm=50.0, dram=57.5)) == "mixed" and W.regime(st(sm=50.0, dram=57.6)) == "memory"
    assert W.regime(st(sm=57.5, dram=50.0)) == "mixed" and W.regime(st(sm=57.6, dram=50.0)) == "compute"


def test_weights_are_the_papers_table():
    assert W.WEIGHTS["mixed"] == (0.20, 0.30, 0.10, 0.15, 0.15, 0.10)
    assert W.WEIGHTS["memory"] == (0.20, 0.90, 0.10, 0.15, 0.45, 0.10)      # 3 x dram, 3 x dram bytes
    assert W.WEIGHTS["compute"] == (0.60, 0.30, 0.10, 0.15, 0.15, 0.30)     # 3 x sm, 3 x instructions
    assert W.PENALTIES == (0.05, 0.05, 0.03, 0.04, 0.04, 0.03)
    for regime_name, scaled in (("memory", (1, 4)), ("compute", (0, 5))):
        for i in range(6):
            factor = W.WEIGHTS[regime_name][i] / W.WEIGHTS["mixed"][i]
            assert factor == pytest.approx(3.0 if i in scaled else 1.0)


def test_proxy_reward_term_by_term():
    base = st()
    assert W.proxy_reward(base, base) == 0.0
    # one term at a time, mixed regime: +10 points of utilisation = 0.1 w; 25 % less work = 0.25 w
    assert W.proxy_reward(base, st(sm=60.0)) == pytest.approx(0.20 * 0.10)
    assert W.proxy_reward(base, st(dram=60.0)) == pytest.approx(0.30 * 0.10)
    assert W.proxy_reward(base, st(tex=60.0)) == pytest.approx(0.10 * 0.10)
    assert W.proxy_reward(base, st(l1=75.0)) == pytest.approx(0.15 * 0.25)
    assert W.proxy_reward(base, st(db=75.0)) == pytest.approx(0.15 * 0.25)
    assert W.proxy_reward(base, st(inst=75.0)) == pytest.approx(0.10 * 0.25)
    # regressions are weighted by the small penalties, and clipped at -1
    assert W.proxy_reward(base, st(sm=40.0)) == pytest.approx(-0.05 * 0.10)
    assert W.proxy_reward(base, st(db=1e9)) == pytest.approx(-0.04 * 1.0)
    # memory-bound baseline: dram terms count three times
    mem = st(sm=20.0, dram=60.0)
    assert W.proxy_reward(mem, st(sm=20.0, dram=70.0, db=50.0)) == pytest.approx(0.90 * 0.10 + 0.45 * 0.50)


def test_guardrails_and_total():
    base = st()
    assert W.guard_penalty(base, base) == 0.0
    assert W.guard_penalty(base, st(lmem=8.0)) == 1.0
    assert W.guard_penalty(base, st(regs=300.0)) == 0.5
    assert W.guard_penalty(base, st(db=150.0)) == 0.0 and W.guard_penalty(base, st(db=150.1)) == 0.5
    assert W.guard_penalty(base, st(inst=151.0, db=151.0)) == 0.5                # one "work" indicator
    r = W.total_reward(base, st(time=0.5, lmem=4.0))
    assert r["R"] == pytest.approx(math.tanh(0.20) - 1.0)
    assert W.total_reward(base, st(time=0.1), passed_tests=False)["R"] == -math.inf


def test_worked_example_on_the_papers_own_matmul_numbers():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    (_, t0, sm0, d0, x0, b0, l0, i0), (_, t1, sm1, d1, x1, b1, l1, i1) = rows
    base = W.State(float(t0), float(sm0), float(d0), float(x0), float(b0), float(l0), float(i0))
    cand = W.State(float(t1), float(sm1), float(d1), float(x1), float(b1), float(l1), float(i1))
    r = W.total_reward(base, cand)
    assert r["regime"] == "compute"                                   # 71.26 - 8.42 > 7.5
    # by hand: tanh(0.4 * 2.8 / 7.2); 0.6*0.0991 + 0.3*0.0261 + 0.1*0.0125 + 0.15*126/408
    #          - 0.04*7/63 (DRAM bytes went up: penalty weight) + 0.3*38/419
    assert r["r_time"] == pytest.approx(0.1543128951113633, abs=1e-12)
    assert r["r_proxy"] == pytest.approx(0.13762672219882383, abs=1e-12)
    assert r["p_guard"] == 0.0                                         # 70 / 63 < 1.5
    assert r["R"] == pytest.approx(0.1543128951113633 + 0.5 * 0.13762672219882383, abs=1e-12)


def test_reads_this_repositorys_profile_summaries():
    prof = os.path.join(os.path.dirname(GOLDEN), "..", "..", "profiles")
    s = W.state_from_summary(os.path.join(prof, "gemv_splitk_kernel_c2_1x8192x8192_bf16.md"))
    assert 10.0 < s.time < 60.0 and 1.3e8 < s.dram_bytes < 1.5e8 and s.lmem_bytes == 0.0
    assert W.regime(s) == "memory"
    c5 = W.state_from_summary(os.path.join(prof, "gemm_umma2_kernel_c5_8192x8192x16384_bf16.md"))
    assert W.regime(c5) == "compute" and 1000.0 < c5.time < 3000.0

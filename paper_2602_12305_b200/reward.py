"""The paper's reward for one kernel edit, evaluated on Nsight Compute summaries.

Host-side arithmetic only.  Given a baseline state (T0, m0) and a candidate state (T, m),
each a run time plus the profiler vector the paper lists under "Profiling Signals" (SM,
DRAM and L1/TEX throughput in % of peak, DRAM bytes, L1 sectors, instructions executed,
registers per thread, local-memory traffic), it computes

    r_time   -- Eq. "time_reward":  tanh(alpha_t (T0 - T) / max(T0, eps))
    r_proxy  -- Eq. "proxy_reward": sum_m w_m clip(dSOL_m / 100) + sum_x w_x clip(dX_x / (X_x0 + eps)),
                clip(z) = max(-1, min(1, z)), with the regime-specific weights of the table
                "Proxy-metric weighting" (Weights appendix) and its regression penalties
    p_guard  -- Eq. "guardrails_penalty": spills, register budget, inflated DRAM bytes / instructions
    R        -- Eq. "total_reward":  beta_t r_time + beta_p r_proxy + beta_l r_llm - p_guard

The regime is memory-bound if SOL_dram - SOL_sm > delta, compute-bound if SOL_sm - SOL_dram >
delta, mixed otherwise (delta = 7.5).  alpha_t = 0.40, the weights, the penalties, delta and
the 1.5x inflation threshold are the paper's.  What the paper leaves open is a parameter here
with a stated default: the beta weights (1.0 / 0.5 / 0: time dominant, no LLM judge), the
guardrail sizes (1.0 spill, 0.5 registers, 0.5 work), rho_max (255, the hardware limit),
which state fixes the regime (the baseline's) and how a regression penalty enters (a term
whose normalised change is negative is weighted by lambda instead of w).

    python -m paper_2602_12305_b200.reward BEFORE_SUMMARY.md AFTER_SUMMARY.md [T0_US T1_US]

reads two summaries in the format of this repository's profiles/ directory; the optional two
numbers replace the run times measured under the profiler by times measured elsewhere (CUDA
events over back-to-back launches), as the paper's search does.
"""
from __future__ import annotations

import dataclasses
import math
import re
import sys

ALPHA_T = 0.40
DELTA = 7.5
INFLATION = 1.5
EPS = 1e-9

# order: sm, dram, tex, l1_sectors, dram_bytes, inst_executed
TERMS = ("sm", "dram", "tex", "l1_sectors", "dram_bytes", "inst_executed")
WEIGHTS = {
    "mixed": (0.20, 0.30, 0.10, 0.15, 0.15, 0.10),
    "memory": (0.20, 0.90, 0.10, 0.15, 0.45, 0.10),
    "compute": (0.60, 0.30, 0.10, 0.15, 0.15, 0.30),
}
PENALTIES = (0.05, 0.05, 0.03, 0.04, 0.04, 0.03)


@dataclasses.dataclass
class State:
    """Run time (any unit, the same for both states) and the profiler vector."""
    time: float
    sol_sm: float
    sol_dram: float
    sol_tex: float
    dram_bytes: float
    l1_sectors: float
    inst_executed: float
    regs_per_thread: float = 0.0
    lmem_bytes: float = 0.0


def clip(z: float) -> float:
    return max(-1.0, min(1.0, z))


def regime(s: State, delta: float = DELTA) -> str:
    if s.sol_dram - s.sol_sm > delta:
        return "memory"
    if s.sol_sm - s.sol_dram > delta:
        return "compute"
    return "mixed"


def time_reward(t0: float, t: float, alpha_t: float = ALPHA_T) -> float:
    return math.tanh(alpha_t * (t0 - t) / max(t0, EPS))


def normalised_changes(base: State, cand: State) -> dict:
    """Positive = good: utilisation up (in units of 100 %), work counters down (relative)."""
    return {
        "sm": clip((cand.sol_sm - base.sol_sm) / 100.0),
        "dram": clip((cand.sol_dram - base.sol_dram) / 100.0),
        "tex": clip((cand.sol_tex - base.sol_tex) / 100.0),
        "l1_sectors": clip((base.l1_sectors - cand.l1_sectors) / (base.l1_sectors + EPS)),
        "dram_bytes": clip((base.dram_bytes - cand.dram_bytes) / (base.dram_bytes + EPS)),
        "inst_executed": clip((base.inst_executed - cand.inst_executed) / (base.inst_executed + EPS)),
    }


def proxy_reward(base: State, cand: State, which: str | None = None) -> float:
    which = which or regime(base)
    z = normalised_changes(base, cand)
    total = 0.0
    for name, w, lam in zip(TERMS, WEIGHTS[which], PENALTIES):
        total += (w if z[name] >= 0.0 else lam) * z[name]
    return total


def guard_penalty(base: State, cand: State, rho_max: float = 255.0, lam_spill: float = 1.0, lam_regs: float = 0.5,
                  lam_work: float = 0.5, inflation: float = INFLATION) -> float:
    p = 0.0
    if cand.lmem_bytes > 0:
        p += lam_spill
    if cand.regs_per_thread > rho_max:
        p += lam_regs
    if cand.dram_bytes > inflation * base.dram_bytes or cand.inst_executed > inflation * base.inst_executed:
        p += lam_work
    return p


def total_reward(base: State, cand: State, r_llm: float = 0.0, passed_tests: bool = True, beta_time: float = 1.0,
                 beta_proxy: float = 0.5, beta_llm: float = 0.0, **guard) -> dict:
    """All the pieces; R is -inf when the candidate failed its correctness tests."""
    which = regime(base)
    rt, rp, pg = time_reward(base.time, cand.time), proxy_reward(base, cand, which), guard_penalty(base, cand, **guard)
    R = beta_time * rt + beta_proxy * rp + beta_llm * r_llm - pg if passed_tests else -math.inf
    return {"regime": which, "r_time": rt, "r_proxy": rp, "p_guard": pg, "R": R,
            "changes": normalised_changes(base, cand)}


# ---------------------------------------------------------------- reading profiles/*.md

_UNITS = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "us": 1.0, "ms": 1e3, "ns": 1e-3, "s": 1e6}


def _metrics(text: str) -> dict:
    out = {}
    for line in text.splitlines():
        m = re.match(r"^\s*([a-z_0-9.]+)\s+([-0-9.eE+]+)\s*([A-Za-z/%]*)", line)
        if m and "__" in m.group(1):
            out[m.group(1)] = (float(m.group(2)), m.group(3))
    return out


def state_from_summary(path: str) -> State:
    """One State from a summary written in this repository's profiles/ format (microseconds)."""
    m = _metrics(open(path).read())

    def val(key, scale=False):
        v, u = m[key]
        return v * _UNITS.get(u, 1.0) if scale else v

    inst_key = "sm__inst_executed.sum" if "sm__inst_executed.sum" in m else "smsp__inst_executed.sum"
    local = m.get("smsp__sass_inst_executed_op_local_ld.sum", (0.0, ""))[0] + \
        m.get("smsp__sass_inst_executed_op_local_st.sum", (0.0, ""))[0]
    return State(time=val("gpu__time_duration.sum", True),
                 sol_sm=val("sm__throughput.avg.pct_of_peak_sustained_elapsed"),
                 sol_dram=val("gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed"),
                 sol_tex=val("l1tex__throughput.avg.pct_of_peak_sustained_elapsed"),
                 dram_bytes=val("dram__bytes_read.sum", True) + val("dram__bytes_write.sum", True),
                 l1_sectors=val("l1tex__t_sectors.sum"), inst_executed=val(inst_key),
                 regs_per_thread=val("launch__registers_per_thread"), lmem_bytes=local)


def main(argv):
    if len(argv) not in (3, 5):
        print(__doc__)
        return 2
    base, cand = state_from_summary(argv[1]), state_from_summary(argv[2])
    if len(argv) == 5:
        base.time, cand.time = float(argv[3]), float(argv[4])
    r = total_reward(base, cand)
    print(f"baseline  {argv[1]}: T = {base.time:.2f} us, regime {r['regime']}-bound "
          f"(SOL sm {base.sol_sm:.1f} %, dram {base.sol_dram:.1f} %)")
    print(f"candidate {argv[2]}: T = {cand.time:.2f} us")
    for k, v in r["changes"].items():
        print(f"  normalised change {k:14s} {v:+.4f}")
    print(f"r_time {r['r_time']:+.4f}   r_proxy {r['r_proxy']:+.4f}   p_guard {r['p_guard']:.2f}   R {r['R']:+.4f}")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))

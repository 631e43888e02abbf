"""Host logic of bench.py that needs no GPU: the timing protocol's launch counts, the roofline
arithmetic, the clock-rejection rule and the traffic table it reads from profiles/."""
import json
import math
import os

import bench
from paper_2602_12305_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class _FakeTimer:
    """Stands in for bench.Timer: records how many launches each region was asked for."""

    def __init__(self, us_per_call):
        self.us, self.regions, self.warmed = us_per_call, [], 0
        self.sampler = None

    def warm(self, n):
        self.warmed += n

    def region(self, launches, barrier=False):
        self.regions.append(launches)
        return launches * self.us / 1e3, 0.0, 1.0


def test_protocol_launch_counts_do_not_depend_on_steps():
    assert bench.PROTOCOL_MIN_LAUNCHES == {"c1": 200, "c2": 200, "c3": 200, "c4": 50, "c5": 20}
    assert bench.PROTOCOL_WARMUP >= 20 and bench.REGIONS >= 5
    peaks = dict(bench.FALLBACK_PEAKS)
    shapes = {"c1": (256, 256, 256, synth.F32), "c2": (1, 8192, 8192, synth.BF16), "c3": (16, 14336, 4096, synth.BF16),
              "c4": (4096, 4096, 4096, synth.BF16), "c5": (8192, 8192, 16384, synth.BF16)}
    for name, (M, N, K, dt) in shapes.items():
        case = synth.Case(name, M, N, K, dt, synth.ACT_RELU, None, None, None)
        est = bench.estimate_ms(case, bench.BOUND[name], peaks)
        assert 1e-4 < est < 10.0, (name, est)           # milliseconds, not bytes
        t = _FakeTimer(est * 1e3)
        stats, _, _ = bench.protocol(t, bench.PROTOCOL_MIN_LAUNCHES[name], est)
        assert t.warmed >= 20 and len(t.regions) == bench.REGIONS
        assert stats["launches"] == sum(t.regions) >= bench.PROTOCOL_MIN_LAUNCHES[name]
        assert stats["min"] <= stats["median"] <= stats["max"]
        assert math.isclose(stats["mean"], est * 1e3, rel_tol=1e-9)


def test_roofline_object():
    case = synth.Case("c2", 1, 8192, 8192, synth.BF16, synth.ACT_GELU_TANH, None, None, None)
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    r = bench.roofline(case, "c2", "hbm", 21.0, peaks, "measured")
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] == 6500.0
    assert math.isclose(r["achieved"], case.algorithmic_bytes / 1e9 / 21e-6) and math.isclose(r["frac"], r["achieved"] / 6500.0)
    assert case.algorithmic_bytes == 134266880
    big = synth.Case("c5", 8192, 8192, 16384, synth.BF16, synth.ACT_RELU, None, None, None)
    burst = bench.roofline(big, "c5", "tensor", 1400.0, peaks, "measured")
    sus = bench.roofline(big, "c5", "tensor", 1600.0, peaks, "measured", sustained_region=True)
    assert burst["peak"] == 1600.0 and sus["peak"] == 1400.0 and "sustained" in sus["peak_source"]
    f32 = synth.Case("c1", 256, 256, 256, synth.F32, synth.ACT_RELU, None, None, None)
    alu = bench.roofline(f32, "c1", "alu", 5.0, peaks, "measured", sm_mhz=1500.0)
    assert math.isclose(alu["peak"], 148 * 128 * 2 * 1.965e9 / 1e12) and alu["frac_at_sampled_clock"] > alu["frac"]


def test_clock_rejection_rule():
    ok = {"sm_mhz": 1400.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"]}
    assert not bench.clocks_rejected(ok)                                   # power cap is kept and noted
    assert bench.clocks_rejected({**ok, "reasons": ["hw_thermal_slowdown"]})
    assert bench.clocks_rejected({**ok, "reasons": ["sw_power_cap", "hw_slowdown"]})
    assert bench.clocks_rejected({"sm_mhz": 900.0, "sm_max_mhz": 1965.0, "reasons": []})     # stuck low, no reason
    assert not bench.clocks_rejected({"sm_mhz": None, "sm_max_mhz": None, "reasons": []})


def test_traffic_table_is_data_not_code():
    with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
        t = json.load(f)
    for name in ("c1", "c2", "c3", "c4", "c5"):
        assert name in t["dram_bytes_per_launch"]
        v = t["dram_bytes_per_launch"][name]
        assert v is None or (isinstance(v, int) and v > 100000)
        assert os.path.exists(os.path.join(ROOT, "profiles", t["source"][name]))
    assert bench.load_traffic()["c2"] == t["dram_bytes_per_launch"]["c2"]


def test_config_names_the_workload_only():
    case = synth.Case("c2", 1, 8192, 8192, synth.BF16, synth.ACT_GELU_TANH, None, None, None)
    cfg = bench.workload_config(case, "c2", None)
    assert set(cfg) == {"workload", "arithmetic", "M", "N", "K", "l2"} and "GELU" in cfg["workload"]

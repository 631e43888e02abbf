"""Host logic of the skinny kernel's schedule and of the persistent CTA-pair kernel's work split:
the self-test program enumerates the segments of every CTA (pair) for a sweep of shapes and checks
exact coverage, balance and scratch-slot bookkeeping.  nvcc builds it; nothing runs on a GPU."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_skinny_schedule_selftest(tmp_path):
    exe = tmp_path / "plan_selftest"
    src = os.path.join(ROOT, "tests", "plan_selftest.cu")
    inc = os.path.join(ROOT, "paper_2602_12305_b200", "csrc")
    subprocess.run(["nvcc", "-std=c++17", "-O1", "-gencode", "arch=compute_100a,code=sm_100a", "-I", inc, "-o", str(exe),
                    src], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout
    assert "0 failed" in out.stdout and "pair plans checked, 0 wrong" in out.stdout
    assert ("pair plan 512x14336x4096: full=112 rem=0 split=1 grid=74; 4096^3: full=222 rem=34 split=2 grid=74"
            in out.stdout)
    # the 16 x 14336 x 4096 workload: one full band of 112 CTAs over K blocks 0..51 and a wide
    # band of 36 CTAs (3 or 4 column tiles each) over the last 12 K blocks
    assert "c3 plan: S=1 k_split=52 G1=36 k_mid=64 G2=0 nbands=2 G=148" in out.stdout

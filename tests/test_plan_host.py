"""Runs the host-side plan checker (tests/plan_check.cpp): every output of every fast-path kernel
is owned by exactly one thread of one tile, every TMA box of the fill obeys the alignment rules and
stays inside its channel row and its shared-memory stage, and every word a consumer reads holds the
sample it expects."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_plan_covers_every_output_once_and_copies_stay_in_bounds(tmp_path):
    csrc = os.path.join(ROOT, "paper_2301_08527_b200", "csrc")
    exe = str(tmp_path / "plan_check")
    cmd = ["g++", "-O2", "-std=c++17", "-I", csrc, "-I", os.path.join(ROOT, "include"), "-I", "/usr/local/cuda/include",
           os.path.join(ROOT, "tests", "plan_check.cpp"), os.path.join(csrc, "rocket_plan.cpp"),
           os.path.join(csrc, "rocket_generate.cpp"), "-o", exe]
    subprocess.check_call(cmd)
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok seed") == 10

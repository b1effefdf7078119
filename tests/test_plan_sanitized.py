"""The planner's host code under AddressSanitizer and UBSan: a seeded sweep of plans (Strassen-Winograd with every
option, and the generic bilinear schemes) whose node tables must stay inside the allocations they name."""
import os
import shutil
import subprocess
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_1202_3173_b200", "csrc")


def test_planner_sweep_under_asan_and_ubsan():
    cuda_inc = "/usr/local/cuda/include"
    if not shutil.which("g++") or not os.path.isdir(cuda_inc):
        pytest.skip("needs g++ and the CUDA headers")
    with tempfile.TemporaryDirectory() as d:
        exe = os.path.join(d, "plan_bounds")
        cmd = ["g++", "-std=c++17", "-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all", "-include", "algorithm",
               "-I", CSRC, "-I", os.path.join(ROOT, "include"), "-I", cuda_inc,
               os.path.join(ROOT, "tests", "native", "plan_bounds.cpp"), os.path.join(CSRC, "plan.cpp"),
               os.path.join(CSRC, "bilinear_plan.cpp"), "-o", exe]
        subprocess.check_call(cmd)
        out = subprocess.run([exe], capture_output=True, text=True, timeout=600,
                             env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1", UBSAN_OPTIONS="halt_on_error=1"))
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    status, plans, nodes = out.stdout.split()[-3:]
    assert status == "ok" and int(plans) >= 500 and int(nodes) > 10000

"""strassen_dgemm_static: the entry point for callers that may not allocate device memory
(its temporaries sit in a static device array inside the library).  It must give the same
result as strassen_dgemm with one level, on consecutive calls that reuse the shared array."""
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest
import torch

import oracle
from paper_1202_3173_b200 import Plan, StrassenError, binding, inputs

pytestmark = pytest.mark.gpu


def _reference_path(n, A, B):
    # the three-launch form of the step, which is what the static entry point runs (by default the library may
    # pick its single-kernel form of a small step, whose inner sums come in another order)
    plan = Plan(n, n // 2, "B", flags=binding.STRASSEN_FLAG_NO_FUSED_STEP)
    assert plan.levels == 1
    C = plan(A, B)
    torch.cuda.synchronize()
    plan.close()
    return C


@pytest.mark.parametrize("n", [512, 511, 301, 64, 3, 2])
def test_static_entry_matches_the_planned_entry_twice_in_a_row(n):
    stream = torch.cuda.current_stream().cuda_stream
    for call, (dist, seed) in enumerate((("uniform", 71), ("int8", 72))):
        A, B = inputs.pair(n, dist, seed + n, device="cuda")
        want = _reference_path(n, A, B)
        got = torch.full_like(A, float("nan"))
        # the second call finds the first call's temporaries in the shared array
        binding.strassen_dgemm_static(n, A.data_ptr(), B.data_ptr(), got.data_ptr(), stream)
        torch.cuda.synchronize()
        assert torch.equal(got, want), "call %d differs from strassen_dgemm" % call
        ref = oracle.classical(A.cpu().numpy(), B.cpu().numpy())
        if dist == "int8":
            assert np.array_equal(got.cpu().numpy(), ref)
        else:
            lim = 1e-11 * n * float(A.abs().max()) * float(B.abs().max())
            assert float(np.abs(got.cpu().numpy() - ref).max()) <= lim


def test_static_entry_rejects_sizes_beyond_its_array():
    n = binding.STRASSEN_STATIC_MAX_N + 2
    A, B = inputs.pair(n, "uniform", 1, device="cuda")
    C = torch.empty_like(A)
    with pytest.raises(StrassenError) as e:
        binding.strassen_dgemm_static(n, A.data_ptr(), B.data_ptr(), C.data_ptr(), 0)
    assert e.value.status == -3 and "STRASSEN_STATIC_MAX_N" in str(e.value)
    with pytest.raises(StrassenError):
        binding.strassen_dgemm_static(1, A.data_ptr(), B.data_ptr(), C.data_ptr(), 0)
    with pytest.raises(StrassenError) as e:
        binding.strassen_dgemm_static(64, A.data_ptr(), B.data_ptr(), A.data_ptr(), 0)
    assert e.value.status == -4


def test_static_entry_alone_in_a_fresh_process():
    """The caller this entry point is for never creates a plan: its first call on the device must do all
    the set-up itself.  A child process calls nothing but strassen_dgemm_static, twice on one stream."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    child = textwrap.dedent("""
        import numpy as np, torch
        import oracle
        from paper_1202_3173_b200 import binding, inputs
        stream = torch.cuda.current_stream().cuda_stream
        for n, dist, seed in ((384, "int8", 5), (511, "int8", 6), (2, "int8", 7)):
            A, B = inputs.pair(n, dist, seed, device="cuda")
            for call in range(2):
                C = torch.full_like(A, float("nan"))
                binding.strassen_dgemm_static(n, A.data_ptr(), B.data_ptr(), C.data_ptr(), stream)
                torch.cuda.synchronize()
                assert np.array_equal(C.cpu().numpy(), oracle.classical(A.cpu().numpy(), B.cpu().numpy())), (n, call)
        print("static-only-ok")
    """)
    r = subprocess.run([sys.executable, "-c", child], cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "static-only-ok" in r.stdout, r.stdout + r.stderr

"""Pins for the classical oracle (the definition C = A.B): a hand-worked product,
closed forms, invariants and numpy's matmul on integer data.  A wrong index,
transposed operand, dropped term or wrong sign fails at least one of them."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(path):
    mats, cur = {}, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line in ("A", "B", "C"):
            cur = line
            mats[cur] = []
        else:
            mats[cur].append([float(x) for x in line.split()])
    return {k: np.array(v) for k, v in mats.items()}


def _ints(rng, shape, lo=-8, hi=8):
    return rng.integers(lo, hi + 1, size=shape).astype(np.float64)


def test_hand_worked_product():
    g = _read_golden(os.path.join(GOLDEN, "classical_3x3.txt"))
    assert np.array_equal(oracle.classical(g["A"], g["B"]), g["C"])
    # the operands do not commute: the transposed-operand mistake is visible
    assert not np.array_equal(oracle.classical(g["B"], g["A"]), g["C"])


@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 33])
def test_identity_and_permutation(n):
    rng = np.random.default_rng(n)
    A = rng.standard_normal((n, n))
    I = np.eye(n)
    assert np.array_equal(oracle.classical(A, I), A)
    assert np.array_equal(oracle.classical(I, A), A)
    perm = rng.permutation(n)
    P = I[perm]                                   # (P A)[i] = A[perm[i]]
    assert np.array_equal(oracle.classical(P, A), A[perm])
    assert np.array_equal(oracle.classical(A, P.T), A[:, perm])


def test_power_of_two_diagonal_scaling_is_exact():
    rng = np.random.default_rng(7)
    n = 17
    A = rng.standard_normal((n, n))
    d = 2.0 ** rng.integers(-5, 6, size=n)
    assert np.array_equal(oracle.classical(np.diag(d), A), d[:, None] * A)
    assert np.array_equal(oracle.classical(A, np.diag(d)), A * d[None, :])


def test_rank_one_closed_form():
    # (u v^T)(w z^T) = (v.w) u z^T ; integers keep every sum exact
    rng = np.random.default_rng(11)
    n = 24
    u, v, w, z = (_ints(rng, n) for _ in range(4))
    C = oracle.classical(np.outer(u, v), np.outer(w, z))
    assert np.array_equal(C, float(v @ w) * np.outer(u, z))


def test_ones_closed_form():
    m, k, n = 5, 9, 4
    C = oracle.classical(np.ones((m, k)), np.ones((k, n)))
    assert C.shape == (m, n) and np.all(C == k)


@pytest.mark.parametrize("shape", [(1, 1, 1), (2, 3, 4), (7, 5, 3), (16, 16, 16), (31, 64, 17)])
def test_against_numpy_on_integers_and_transpose(shape):
    m, k, n = shape
    rng = np.random.default_rng(m * 100 + n)
    A, B = _ints(rng, (m, k)), _ints(rng, (k, n))
    C = oracle.classical(A, B)
    assert np.array_equal(C, A @ B)               # integer data: any order is exact
    assert np.array_equal(oracle.classical(B.T.copy(), A.T.copy()), C.T)


def test_freivalds_identity():
    rng = np.random.default_rng(5)
    n = 96
    A, B = _ints(rng, (n, n)), _ints(rng, (n, n))
    x = _ints(rng, (n, 1), 0, 3)
    C = oracle.classical(A, B)
    assert np.array_equal(oracle.classical(A, oracle.classical(B, x)), oracle.classical(C, x))


def test_summation_order_is_k_ascending():
    # 1 + 2^-53 + 2^-53 evaluated left to right stays 1; any other order gives 1 + 2^-52
    e = 2.0 ** -53
    A = np.array([[1.0, e, e]])
    B = np.ones((3, 1))
    assert oracle.classical(A, B)[0, 0] == 1.0
    assert oracle.classical(A[:, ::-1].copy(), B)[0, 0] == 1.0 + 2.0 ** -52


def test_products_are_not_fused():
    # a*b + c with a*b rounded first differs from fma(a, b, c) for these values
    a = 1.0 + 2.0 ** -30
    A = np.array([[1.0, a]])
    B = np.array([[-(a * a)], [a]])
    assert oracle.classical(A, B)[0, 0] == 0.0     # fma(a, a, -fl(a*a)) would leave 2^-60


def test_empty_inner_dimension_gives_zeros():
    C = oracle.classical(np.zeros((3, 0)), np.zeros((0, 2)))
    assert C.shape == (3, 2) and np.all(C == 0)


def test_samples_match_full_product():
    rng = np.random.default_rng(3)
    n = 40
    A, B = rng.standard_normal((n, n)), rng.standard_normal((n, n))
    C = oracle.classical(A, B)
    rows = rng.integers(0, n, 200)
    cols = rng.integers(0, n, 200)
    assert np.array_equal(oracle.classical_samples(A, B, rows, cols), C[rows, cols])
    with pytest.raises(IndexError):
        oracle.classical_samples(A, B, [n], [0])


def test_thread_count_does_not_change_bits():
    import subprocess, sys
    code = ("import numpy as np, oracle, hashlib;"
            "r=np.random.default_rng(1);A=r.standard_normal((65,65));B=r.standard_normal((65,65));"
            "print(hashlib.sha1(oracle.classical(A,B).tobytes()).hexdigest())")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = set()
    for t in ("1", "3"):
        env = dict(os.environ, OMP_NUM_THREADS=t, PYTHONPATH=root)
        outs.add(subprocess.check_output([sys.executable, "-c", code], env=env, cwd=root).strip())
    assert len(outs) == 1

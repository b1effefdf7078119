"""Pins for the oracle's diagonal scaling (Section 6.1): the diagonals are powers of two (the scaling
is exact), rows / columns are brought to [1, 2), and on a badly row-scaled problem the scaled
Strassen-Winograd meets the row/column-wise bound that the plain one misses."""
import numpy as np
import pytest

import oracle


def _graded(n, seed, span=24):
    rng = np.random.default_rng(seed)
    A = rng.uniform(-1, 1, (n, n)) * 2.0 ** rng.integers(-span, span + 1, size=(n, 1))     # rows of wildly different size
    B = rng.uniform(-1, 1, (n, n)) * 2.0 ** rng.integers(-span, span + 1, size=(1, n))     # and columns of B
    return A, B


def test_exponents_bring_rows_and_columns_into_1_2():
    A, B = _graded(96, 1)
    e1, e2, e3 = oracle.scaling_exponents(A, B, inside=False, outside=True)
    assert not e2.any()
    r = np.abs(np.ldexp(A, e1[:, None])).max(axis=1)
    c = np.abs(np.ldexp(B, e3[None, :])).max(axis=0)
    assert np.all((r >= 1) & (r < 2)) and np.all((c >= 1) & (c < 2))
    # hand-checkable case: row maxima 3, 0.4, 0 -> exponents -1, 2, 0
    e1, _, e3 = oracle.scaling_exponents(np.array([[3.0, 1, 0], [0.1, -0.4, 0], [0, 0, 0]]), np.eye(3))
    assert list(e1) == [-1, 2, 0] and list(e3) == [0, 0, 0]


def test_inside_scaling_balances_columns_of_a_against_rows_of_b():
    rng = np.random.default_rng(3)
    n = 64
    A = rng.uniform(-1, 1, (n, n)) * 2.0 ** rng.integers(-20, 21, size=(1, n))
    B = rng.uniform(-1, 1, (n, n)) * 2.0 ** rng.integers(-20, 21, size=(n, 1))
    _, e2, _ = oracle.scaling_exponents(A, B, inside=True, outside=False)
    a = np.abs(np.ldexp(A, e2[None, :])).max(axis=0)
    b = np.abs(np.ldexp(B, -e2[:, None])).max(axis=1)
    ratio = np.log2(b / a)
    assert np.all(np.abs(ratio) <= 2.0)          # within a factor 4 after balancing (was up to 2^40)
    assert np.abs(np.log2(np.abs(B).max(axis=1) / np.abs(A).max(axis=0))).max() > 20


@pytest.mark.parametrize("inside,outside", [(False, True), (True, False), (True, True)])
def test_scaling_is_exact_on_integers(inside, outside):
    rng = np.random.default_rng(5)
    n = 48
    A = rng.integers(-8, 9, (n, n)).astype(float) * 2.0 ** rng.integers(-6, 7, size=(n, 1))
    B = rng.integers(-8, 9, (n, n)).astype(float) * 2.0 ** rng.integers(-6, 7, size=(1, n))
    C, cnt = oracle.scaled_strassen_winograd(A, B, 6, "BDB", inside, outside)
    assert np.array_equal(C, oracle.classical(A, B))
    assert cnt["base_calls"] == 343


def test_outside_scaling_gives_the_row_column_wise_bound():
    n = 256
    A, B = _graded(n, 7)
    ref = oracle.classical(A, B)
    plain, _ = oracle.strassen_winograd(A, B, 32)
    scaled, _ = oracle.scaled_strassen_winograd(A, B, 32)
    rows, cols = np.abs(A).max(axis=1), np.abs(B).max(axis=0)
    # |C_ij - C^_ij| <= f(n) eps ||A(i,:)|| ||B(:,j)||.  The constant: the scaled factors have every row of A and
    # column of B in [1, 2), so the norm-wise bound 1e-11 n max|A'| max|B'| is below 1e-11 n 2 2 = 4e-11 n for them;
    # scaling C back multiplies entry (i, j) by 2^-e1_i 2^-e3_j, and 2^-e1_i <= max_k|A_ik|, 2^-e3_j <= max_k|B_kj|.
    bound = 4e-11 * n * rows[:, None] * cols[None, :]
    assert np.all(np.abs(scaled - ref) <= bound)
    assert not np.all(np.abs(plain - ref) <= bound)        # the unscaled recursion only meets the norm-wise bound
    assert np.abs(plain - ref).max() <= 1e-11 * n * np.abs(A).max() * np.abs(B).max()

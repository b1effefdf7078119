"""Pins for the Strassen-Winograd oracle: the block identities of Appendix A (and the
reading of its three typos), exact equality with the classical oracle on integer data
over a sweep of sizes / cutoffs / schedules (odd sizes included), the 7^L product
count, the flop closed form, and the norm-wise error bound on float data."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _constants():
    out = {}
    for line in open(os.path.join(GOLDEN, "paper_constants.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def _ints(rng, n):
    return rng.integers(-8, 9, size=(n, n)).astype(np.float64)


# --- one step with non-commuting blocks, written from a coefficient table ----------
# Each row: which of (X11, X12, X21, X22) or an earlier sum enters with which sign.

def _one_step(A, B, t3_term, t3_sign, s2_sign, t5_sign):
    h = A.shape[0] // 2
    q = lambda X: (X[:h, :h], X[:h, h:], X[h:, :h], X[h:, h:])
    A11, A12, A21, A22 = q(A)
    B11, B12, B21, B22 = q(B)
    Aq = {"A11": A11, "A12": A12, "A21": A21, "A22": A22}
    T0, T1, T6 = A11, A12, A22
    T2 = A21 + A22
    T3 = T2 + t3_sign * Aq[t3_term]
    T4 = A11 - A21
    T5 = A12 + t5_sign * T3
    S0, S1, S5 = B11, B21, B22
    S2 = B12 + s2_sign * B11
    S3 = B22 - S2
    S4 = B22 - B12
    S6 = S3 - B21
    Q = [T @ S for T, S in ((T0, S0), (T1, S1), (T2, S2), (T3, S3), (T4, S4), (T5, S5), (T6, S6))]
    U1 = Q[0] + Q[3]
    U2 = U1 + Q[4]
    U3 = U1 + Q[2]
    return np.block([[Q[0] + Q[1], U3 + Q[5]], [U2 - Q[6], U2 + Q[2]]])


def test_block_identities_select_one_reading_of_the_printed_table():
    rng = np.random.default_rng(42)
    A, B = _ints(rng, 6), _ints(rng, 6)          # 3x3 blocks: do not commute
    want = A @ B
    printed = _one_step(A, B, "A12", -1, +1, +1)
    h = 3
    assert np.array_equal(printed[:h, :h], want[:h, :h])          # C11 survives the typos
    assert not np.array_equal(printed[:h, h:], want[:h, h:])
    assert not np.array_equal(printed[h:, :h], want[h:, :h])
    assert not np.array_equal(printed[h:, h:], want[h:, h:])
    passing = [v for v in itertools.product(("A11", "A12", "A21", "A22"), (-1, 1), (-1, 1), (-1, 1))
               if np.array_equal(_one_step(A, B, *v), want)]
    assert passing == [("A11", -1, -1, -1)]       # T3 = T2 - A11, S2 = B12 - B11, T5 = A12 - T3


# --- the C oracle against the definition ------------------------------------------

SWEEP = [(2, 1, None), (4, 1, None), (4, 2, "B"), (4, 2, "D"), (6, 3, None), (8, 1, "BDB"), (8, 2, "DB"),
         (16, 2, "DBD"), (16, 4, "BB"), (24, 3, "DDD"), (32, 8, "BD"), (64, 8, "BBB"), (64, 16, "DD"),
         (96, 12, "BDB"), (128, 16, None)]


@pytest.mark.parametrize("n,cutoff,sched", SWEEP)
def test_equals_classical_on_integers(n, cutoff, sched):
    rng = np.random.default_rng(n * 31 + cutoff)
    A, B = _ints(rng, n), _ints(rng, n)
    C, cnt = oracle.strassen_winograd(A, B, cutoff, sched)
    assert np.array_equal(C, oracle.classical(A, B))
    L = len(oracle.level_sizes(n, cutoff)) - 1
    assert cnt["base_calls"] == 7 ** L
    assert cnt["peels"] == 0


ODD = [(3, 1), (5, 2), (7, 3), (9, 2), (15, 3), (17, 4), (31, 7), (33, 8), (57, 3), (197, 12), (101, 25)]


@pytest.mark.parametrize("n,cutoff", ODD)
@pytest.mark.parametrize("mode", ["B", "D"])
def test_peeling_equals_classical_on_integers(n, cutoff, mode):
    rng = np.random.default_rng(n)
    A, B = _ints(rng, n), _ints(rng, n)
    sizes = oracle.level_sizes(n, cutoff)
    L = len(sizes) - 1
    C, cnt = oracle.strassen_winograd(A, B, cutoff, mode * L)
    assert np.array_equal(C, oracle.classical(A, B))
    assert cnt["base_calls"] == 7 ** L
    # one peel per node of every odd level above the leaves
    assert cnt["peels"] == sum(7 ** i for i, m in enumerate(sizes[:-1]) if m % 2)


def test_level_sizes_of_the_peeling_chains():
    assert oracle.level_sizes(57, 3) == [57, 28, 14, 7, 3]
    assert oracle.level_sizes(197, 12) == [197, 98, 49, 24, 12]
    assert oracle.level_sizes(12345, 771) == [12345, 6172, 3086, 1543, 771]
    assert oracle.level_sizes(512, 256) == [512, 256]
    assert oracle.level_sizes(4096, 512) == [4096, 2048, 1024, 512]
    assert oracle.level_sizes(47040, 2940) == [47040, 23520, 11760, 5880, 2940]
    assert oracle.level_sizes(300, 512) == [300]


def test_no_recursion_at_or_below_cutoff():
    rng = np.random.default_rng(0)
    A, B = rng.standard_normal((20, 20)), rng.standard_normal((20, 20))
    C, cnt = oracle.strassen_winograd(A, B, 20)
    assert np.array_equal(C, oracle.classical(A, B))      # same routine, same bits
    assert cnt == {"base_calls": 1, "mults": 8000, "adds": 400 * 19, "block_adds": 0, "peels": 0}


@pytest.mark.parametrize("n0,L", [(1, 3), (2, 4), (8, 3), (5, 2), (16, 2)])
def test_operation_counts_match_the_closed_form(n0, L):
    n = n0 * 2 ** L
    rng = np.random.default_rng(L)
    A, B = _ints(rng, n), _ints(rng, n)
    _, cnt = oracle.strassen_winograd(A, B, n0)
    total = cnt["mults"] + cnt["adds"]
    assert cnt["base_calls"] == 7 ** L
    assert cnt["mults"] == 7 ** L * n0 ** 3
    assert cnt["block_adds"] == 15 * sum(7 ** i for i in range(L))     # 15 additions per step
    assert total == oracle.flops_recurrence(n, n0)
    assert math.isclose(total, oracle.flops_closed_form(n, n0), rel_tol=1e-12)


def test_flop_numbers_of_the_paper():
    k = _constants()
    cs = lambda n0: (2 * n0 + 4) / n0 ** (math.log2(7) - 2)
    assert min(range(1, 65), key=cs) == k["flop_optimal_cutoff"]
    assert round(cs(8), 2) == k["c_s_at_optimal_cutoff"]
    # F(n) = c_s n^w0 + (quadratic coefficient) n^2 at n0 = 8, L = 3 and n0 = 512, L = 3
    for n0, L in ((8, 3), (512, 3)):
        n = n0 * 2 ** L
        assert math.isclose(oracle.flops_recurrence(n, n0),
                            cs(n0) * n ** math.log2(7) + k["quadratic_coefficient"] * n * n, rel_tol=1e-12)
    assert oracle.flops_recurrence(64, 8) == 418560
    assert oracle.flops_recurrence(4096, 512) == 92349136896


def test_depth_first_combine_uses_the_flat_contributions():
    # 8 operand sums + 10 accumulations per depth-first step
    rng = np.random.default_rng(9)
    A, B = _ints(rng, 16), _ints(rng, 16)
    _, cnt = oracle.strassen_winograd(A, B, 8, "D")
    assert cnt["block_adds"] == 18


@pytest.mark.parametrize("n,cutoff,sched,dist", [(512, 256, "B", "u"), (512, 64, "BDB", "u"),
                                                  (384, 48, "DBD", "n"), (771, 96, "BBB", "u")])
def test_float_error_within_the_norm_wise_bound(n, cutoff, sched, dist):
    rng = np.random.default_rng(1001)
    draw = (lambda: rng.uniform(-1, 1, (n, n))) if dist == "u" else (lambda: rng.standard_normal((n, n)))
    A, B = draw(), draw()
    C, _ = oracle.strassen_winograd(A, B, cutoff, sched)
    err = np.abs(C - oracle.classical(A, B)).max()
    bound = 1e-11 * n * np.abs(A).max() * np.abs(B).max()
    assert err <= bound
    assert err <= 1e-2 * bound        # a correct implementation sits orders of magnitude below
    assert err > 0                    # and it is not the classical routine in disguise


def test_effective_gflops_definition():
    # Section 5.2, values worked by hand: 2 * 1000^3 flop in 2 s is exactly 1 GFLOP/s; 2 * 2000^3 = 1.6e10 flop
    # in 4 s is 4 GFLOP/s; 2 * 2048^3 = 17 179 869 184 flop, 32 of them in half a second: 1099.511627776 GFLOP/s;
    # halving the time doubles the rate, and the rate grows with the cube of n
    assert oracle.effective_gflops(1000, 2.0) == 1.0
    assert oracle.effective_gflops(2000, 4.0) == 4.0
    assert oracle.effective_gflops(2048, 0.5, batch=32) == pytest.approx(1099.511627776, rel=1e-15)
    assert oracle.effective_gflops(94080, 1.0) == pytest.approx(1665412.890624, rel=1e-15)   # 94080^2 = 8 851 046 400; 2 * 94080^3 = 1 665 412 890 624 000
    assert oracle.effective_gflops(500, 1.0) * 8 == oracle.effective_gflops(1000, 1.0)
    assert oracle.effective_gflops(1000, 1.0) == 2 * oracle.effective_gflops(1000, 2.0)

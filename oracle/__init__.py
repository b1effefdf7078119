"""CPU oracle for the Strassen-Winograd hot path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline legs may import
this package; the product library never does, and this package never imports the
product.  It wraps ``strassen_oracle.c`` (plain C, FP64, compiled here with gcc,
``-O2 -ffp-contract=off -fopenmp``) and adds the host-side arithmetic of the
paper that needs no matrix data:

* ``classical`` / ``classical_samples`` -- the definition C = A.B (Algorithm 1,
  "Ensure C = A.B"), k ascending, multiply and add never fused.
* ``strassen_winograd`` -- the sequential Strassen-Winograd recursion of
  Appendix A (typos of the printed table corrected), cutoff to classical
  (Section 5.4), dynamic peeling for odd sizes (Section 3.1), per-level 'B'
  (U-chain combine) or 'D' (one Q at a time folded into C, Algorithm 1).
* ``level_sizes``, ``flops_recurrence``, ``flops_closed_form`` -- the cost
  F(n) = c_s n^{log2 7} - 5 n^2, c_s = (2 n0 + 4) / n0^{log2 7 - 2} (Appendix A).
* ``workspace_words`` -- the memory recurrences of Sections 3.3.1 and 3.4.1
  (a BFS step stores 7 triples S_j,T_j,Q_j of quarter size, a DFS step one),
  ``mem_um_closed_form`` -- Mem_UM = 7 n^2 / P^{2/w0} - 4 n^2 / P at P = 7^k.
* ``effective_gflops`` -- 2 n^3 / (t 10^9) (Section 5.2).
* ``bilinear_product``, ``brent_residual``, ``classical_scheme`` -- the recursion
  for any <n0, n0, n0; q> bilinear scheme (Section 6.6) on numpy blocks, the
  identities its tables must satisfy, and the table of the classical algorithm.
* ``bfs_row_blocks``, ``bfs_share``, ``bfs_unshare``, ``bfs_form_shares``,
  ``bfs_combine_shares`` -- one BFS step spread over seven processors
  (Algorithm 2 with k = 1; layout of Section 3.2) restated on numpy blocks.

Every function is pinned by tests/test_oracle_*.py to something other than
itself (closed forms, a hand-worked product, brute-force equality on integer
data, the paper's closed-form counts); none is "parity unpinned" except values at
sizes where no full classical product can be computed, where sampled entries of
the definition are used instead.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "strassen_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libstrassen_oracle.so")
_lock = threading.Lock()
_lib = None


class Counters(ctypes.Structure):
    _fields_ = [("base_calls", ctypes.c_int64), ("mults", ctypes.c_int64),
                ("adds", ctypes.c_int64), ("block_adds", ctypes.c_int64),
                ("peels", ctypes.c_int64)]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no FMA contraction, OpenMP over rows)."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                               "-std=c11", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            P = ctypes.c_void_p
            I = ctypes.c_int64
            lib.oracle_classical.argtypes = [P, I, P, I, P, I, I, I, I]
            lib.oracle_classical.restype = None
            lib.oracle_classical_samples.argtypes = [P, I, P, I, I, P, P, I, P]
            lib.oracle_classical_samples.restype = None
            lib.oracle_sw.argtypes = [P, I, P, I, P, I, I, I, ctypes.c_char_p, ctypes.POINTER(Counters)]
            lib.oracle_sw.restype = ctypes.c_int
            _lib = lib
    return _lib


def _mat(x):
    a = np.ascontiguousarray(x, dtype=np.float64)
    if a.ndim != 2:
        raise ValueError("expected a 2-D array")
    return a


def cores() -> int:
    """Threads the C oracle uses (OpenMP default = CPUs this process may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def classical(A, B):
    """C = A.B from the definition (m x k times k x n), FP64."""
    A, B = _mat(A), _mat(B)
    m, k = A.shape
    k2, n = B.shape
    if k != k2:
        raise ValueError("inner dimensions differ")
    C = np.empty((m, n), dtype=np.float64)
    _load().oracle_classical(A.ctypes.data, max(k, 1), B.ctypes.data, max(n, 1), C.ctypes.data, max(n, 1), m, n, k)
    return C


def classical_samples(A, B, rows, cols):
    """Entries C[rows[t], cols[t]] of A.B from the definition."""
    A, B = _mat(A), _mat(B)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    if rows.shape != cols.shape or A.shape[1] != B.shape[0]:
        raise ValueError("shape mismatch")
    if rows.size and (rows.min() < 0 or rows.max() >= A.shape[0] or cols.min() < 0 or cols.max() >= B.shape[1]):
        raise IndexError("sample out of range")
    out = np.empty(rows.shape, dtype=np.float64)
    _load().oracle_classical_samples(A.ctypes.data, A.shape[1], B.ctypes.data, B.shape[1], A.shape[1],
                                     rows.ctypes.data, cols.ctypes.data, rows.size, out.ctypes.data)
    return out


def strassen_winograd(A, B, cutoff, schedule=None):
    """(C, counters) with C = A.B by Strassen-Winograd, recursing while size > cutoff."""
    A, B = _mat(A), _mat(B)
    n = A.shape[0]
    if A.shape != (n, n) or B.shape != (n, n):
        raise ValueError("square matrices of equal size expected")
    C = np.empty((n, n), dtype=np.float64)
    cnt = Counters()
    sched = None if schedule is None else schedule.encode()
    rc = _load().oracle_sw(A.ctypes.data, n, B.ctypes.data, n, C.ctypes.data, n, n, int(cutoff), sched,
                           ctypes.byref(cnt))
    if rc != 0:
        raise RuntimeError("oracle_sw failed with status %d" % rc)
    return C, cnt.as_dict()


# ---------------------------------------------------------------------------
# host-side arithmetic of the paper (no matrix data)
# ---------------------------------------------------------------------------

def level_sizes(n: int, cutoff: int):
    """[m_0 = n, m_1, ..., m_L]: halve (dropping a peeled row/column) while m > cutoff."""
    if n < 1 or cutoff < 1:
        raise ValueError("n and cutoff must be positive")
    m = [n]
    while m[-1] > cutoff:
        m.append(m[-1] // 2)
    return m


def flops_recurrence(n: int, cutoff: int) -> int:
    """Flops of Strassen-Winograd for n = n0 2^L (no odd size on the way):
    7^L classical products of 2 n0^3 - n0^2 flops plus 15 quadrant additions per node."""
    m = level_sizes(n, cutoff)
    L = len(m) - 1
    if any(x % 2 for x in m[:-1]):
        raise ValueError("closed form holds only when no level is peeled")
    n0 = m[-1]
    return 7 ** L * (2 * n0 ** 3 - n0 ** 2) + 15 * sum(7 ** i * m[i + 1] ** 2 for i in range(L))


def flops_closed_form(n: int, n0: int) -> float:
    """F(n) = c_s n^{w0} - 5 n^2 with c_s = (2 n0 + 4) / n0^{w0 - 2}, w0 = log2 7 (Appendix A)."""
    w0 = math.log2(7.0)
    cs = (2 * n0 + 4) / n0 ** (w0 - 2)
    return cs * n ** w0 - 5.0 * n * n


def workspace_words(n: int, cutoff: int, schedule: str, batch: int = 1, accounting: int = 21) -> int:
    """Words beyond A, B, C for a per-level schedule string (top level first).

    Sections 3.3.1 / 3.4.1: a BFS step stores all 7 triples (S_j, T_j, Q_j) of quarter
    size per parent, a DFS step one triple.  accounting=21 counts every triple in full
    (the paper's figure); accounting=15 counts, at BFS levels, only the 4+4 operand sums
    that are not plain quadrants plus the 7 products (15 of the 21 quarter matrices).
    """
    m = level_sizes(n, cutoff)
    L = len(m) - 1
    if len(schedule) != L or any(c not in "BD" for c in schedule):
        raise ValueError("schedule must have one 'B' or 'D' per level (%d levels)" % L)
    if accounting not in (15, 21):
        raise ValueError("accounting is 21 (paper) or 15 (quadrant operands as views)")
    words, live = 0, batch
    for i, c in enumerate(schedule):
        h = m[i + 1]
        if c == "B":
            words += live * accounting * h * h
            live *= 7
        else:
            words += live * 3 * h * h
    return words


def mem_um_closed_form(n: int, k: int) -> float:
    """Mem_UM(n, P = 7^k) * P = 7 n^2 (7/4)^k - 4 n^2: total words of A, B, C plus all
    temporaries of k BFS steps, summed over the P processors (Section 3.3.1)."""
    return 7.0 * n * n * (7.0 / 4.0) ** k - 4.0 * n * n


def lm_schedule(n: int, cutoff: int, budget_words: int, batch: int = 1, accounting: int = 21) -> str:
    """Limited-Memory rule (Section 3.4): the fewest leading DFS steps, followed by
    BFS steps only, whose temporaries fit the budget."""
    L = len(level_sizes(n, cutoff)) - 1
    for ell in range(L + 1):
        s = "D" * ell + "B" * (L - ell)
        if workspace_words(n, cutoff, s, batch, accounting) <= budget_words:
            return s
    raise ValueError("even the all-DFS schedule does not fit the budget")


# ---------------------------------------------------------------------------
# diagonal scaling (Section 6.1): D1 C D3 = (D1 A D2)(D2^-1 B D3) with power-of-two diagonals
# ---------------------------------------------------------------------------

def _ilog2(x):
    """floor(log2 |x|) per element, 0 where x == 0 (exponent arithmetic, no logarithm)."""
    x = np.abs(np.asarray(x, dtype=np.float64))
    _, e = np.frexp(x)                      # x = m 2^e, 0.5 <= m < 1
    return np.where(x > 0, e - 1, 0).astype(np.int64)


def scaling_exponents(A, B, inside: bool = False, outside: bool = True):
    """Exponents (e1, e2, e3) of D1 = diag(2^e1), D2 = diag(2^e2), D3 = diag(2^e3).

    inside : balances column k of A against row k of B,
             e2_k = floor((ilog2 max_j|B_kj| - ilog2 max_i|A_ik|) / 2);
    outside: brings the largest entry of every row of A D2 and of every column of D2^-1 B into [1, 2),
             e1_i = -ilog2 max_k |A_ik| 2^e2_k,  e3_j = -ilog2 max_k |B_kj| 2^-e2_k.
    Powers of two: the scaling itself is exact, so the scaled product, unscaled, is the product."""
    A, B = _mat(A), _mat(B)
    n = A.shape[0]
    e1 = np.zeros(n, dtype=np.int64)
    e2 = np.zeros(n, dtype=np.int64)
    e3 = np.zeros(n, dtype=np.int64)
    if inside:
        e2 = (_ilog2(np.abs(B).max(axis=1)) - _ilog2(np.abs(A).max(axis=0))) // 2
    if outside:
        e1 = -_ilog2(np.abs(np.ldexp(A, e2[None, :])).max(axis=1))
        e3 = -_ilog2(np.abs(np.ldexp(B, -e2[:, None])).max(axis=0))
    return e1, e2, e3


def scaled_strassen_winograd(A, B, cutoff, schedule=None, inside: bool = False, outside: bool = True):
    """Strassen-Winograd on the diagonally scaled operands, result scaled back (Section 6.1)."""
    A, B = _mat(A), _mat(B)
    e1, e2, e3 = scaling_exponents(A, B, inside, outside)
    As = np.ldexp(A, e1[:, None] + e2[None, :])
    Bs = np.ldexp(B, -e2[:, None] + e3[None, :])
    Cs, cnt = strassen_winograd(As, Bs, cutoff, schedule)
    return np.ldexp(Cs, -e1[:, None] - e3[None, :]), cnt


def effective_gflops(n: int, seconds: float, batch: int = 1) -> float:
    """Effective GFLOPS = 2 n^3 / (seconds 10^9) (Section 5.2), times the batch size."""
    return 2.0 * n ** 3 * batch / (seconds * 1e9)


# ---- one BFS step over P = 7 processors (Algorithm 2, BFS(A, B, C, k) with k = 1) ----------------------
# Layout (Section 3.2: every processor owns the same part of each quadrant): the h = n / 2 rows of every
# quadrant are cut into seven consecutive blocks; processor r owns block r of all four quadrants.

def bfs_row_blocks(h: int, P: int = 7):
    """[(first row, rows)] of the P consecutive row blocks of a quadrant with h rows."""
    out, start = [], 0
    for r in range(P):
        rows = h // P + (1 if r < h % P else 0)
        out.append((start, rows))
        start += rows
    return out


def bfs_share(X, r: int, P: int = 7):
    """Processor r's share of the n x n matrix X: [X11_r | X12_r] stacked on [X21_r | X22_r]."""
    X = np.asarray(X)
    h = X.shape[0] // 2
    start, rows = bfs_row_blocks(h, P)[r]
    return np.vstack((X[start:start + rows], X[h + start:h + start + rows]))


def bfs_unshare(shares, n: int, P: int = 7):
    """The n x n matrix whose shares are `shares` (inverse of bfs_share over all processors)."""
    h = n // 2
    X = np.empty((n, n))
    for r, (start, rows) in enumerate(bfs_row_blocks(h, P)):
        X[start:start + rows] = shares[r][:rows]
        X[h + start:h + start + rows] = shares[r][rows:]
    return X


def bfs_form_shares(A_share, B_share):
    """Algorithm 2, "locally compute T_i, S_i": block r of the seven operand pairs of Appendix A
    (typos corrected as in the C oracle) from a processor's shares.  Returns (T, S), lists of 7 blocks."""
    A_share, B_share = np.asarray(A_share), np.asarray(B_share)
    rows, h = A_share.shape[0] // 2, A_share.shape[1] // 2
    a11, a12, a21, a22 = A_share[:rows, :h], A_share[:rows, h:], A_share[rows:, :h], A_share[rows:, h:]
    b11, b12, b21, b22 = B_share[:rows, :h], B_share[:rows, h:], B_share[rows:, :h], B_share[rows:, h:]
    t2 = a21 + a22
    t3 = t2 - a11
    s2 = b12 - b11
    s3 = b22 - s2
    T = [a11.copy(), a12.copy(), t2, t3, a11 - a21, a12 - t3, a22.copy()]
    S = [b11.copy(), b21.copy(), s2, s3, b22 - b12, b22.copy(), s3 - b21]
    return T, S


def bfs_combine_shares(Q):
    """Algorithm 2, "locally compute C from Q_i": a processor's share of C from its blocks of Q_0..Q_6."""
    q = [np.asarray(x) for x in Q]
    u1 = q[0] + q[3]
    u2 = u1 + q[4]
    u3 = u1 + q[2]
    return np.vstack((np.hstack((q[0] + q[1], u3 + q[5])), np.hstack((u2 - q[6], u2 + q[2]))))


# ---- any <n0, n0, n0; q> bilinear scheme (Section 6.6 "Parallelizing other algorithms") -------------------
# u, v: q x n0^2, w: n0^2 x q (blocks row-major):  T_j = sum_b u[j][b] A_b,  S_j = sum_b v[j][b] B_b,
# Q_j = T_j . S_j,  C_b = sum_j w[b][j] Q_j.

def brent_residual(n0, q, u, v, w):
    """Largest violation of the identities that make the tables a matrix multiplication: the coefficient of
    A_(a,b) B_(c,d) in C_(e,f) is 1 where b = c, a = e, d = f, and 0 elsewhere.  0 for a correct scheme."""
    u, v, w = np.asarray(u, dtype=np.int64), np.asarray(v, dtype=np.int64), np.asarray(w, dtype=np.int64)
    got = np.einsum("jx,jy,zj->xyz", u, v, w)
    want = np.zeros_like(got)
    for a in range(n0):
        for b in range(n0):
            for d in range(n0):
                want[a * n0 + b, b * n0 + d, a * n0 + d] = 1
    return int(np.abs(got - want).max())


def classical_scheme(n0: int):
    """The classical algorithm as a <n0, n0, n0; n0^3> scheme: product (i, k, j) is A_(i,k) B_(k,j), added to C_(i,j)."""
    q = n0 ** 3
    u, v, w = np.zeros((q, n0 * n0), dtype=int), np.zeros((q, n0 * n0), dtype=int), np.zeros((n0 * n0, q), dtype=int)
    t = 0
    for i in range(n0):
        for j in range(n0):
            for k in range(n0):
                u[t, i * n0 + k] = 1
                v[t, k * n0 + j] = 1
                w[i * n0 + j, t] = 1
                t += 1
    return n0, q, u.tolist(), v.tolist(), w.tolist()


def bilinear_product(A, B, scheme, cutoff: int):
    """C = A.B by the recursion of the scheme down to sizes <= cutoff, then the classical oracle.
    Returns (C, number of base products)."""
    n0, q, u, v, w = scheme
    u, v, w = np.asarray(u), np.asarray(v), np.asarray(w)
    A, B = np.asarray(A, dtype=np.float64), np.asarray(B, dtype=np.float64)
    m = A.shape[0]
    if m <= cutoff:
        return classical(A, B), 1
    if m % n0:
        raise ValueError("size %d is not divisible by n0 = %d" % (m, n0))
    hh = m // n0
    blk = lambda X, b: X[(b // n0) * hh:(b // n0 + 1) * hh, (b % n0) * hh:(b % n0 + 1) * hh]
    Q, calls = [], 0
    for j in range(q):
        T = sum(int(u[j, b]) * blk(A, b) for b in range(n0 * n0) if u[j, b])
        S = sum(int(v[j, b]) * blk(B, b) for b in range(n0 * n0) if v[j, b])
        Qj, c = bilinear_product(np.ascontiguousarray(T), np.ascontiguousarray(S), scheme, cutoff)
        Q.append(Qj)
        calls += c
    C = np.empty((m, m))
    for b in range(n0 * n0):
        blk(C, b)[...] = sum(int(w[b, j]) * Q[j] for j in range(q) if w[b, j])
    return C, calls

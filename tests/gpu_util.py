"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI on seeded
inputs and compare with the CPU oracle (whole matrix, or a sampled block of the definition)."""
import numpy as np
import torch

import oracle
from paper_1202_3173_b200 import Plan, inputs

TOL_FACTOR = 1e-11      # max|C - C_ref| <= 1e-11 * n * max|A| * max|B| on float inputs
SANITY_FRACTION = 0.02  # a correct Strassen-Winograd sits orders of magnitude below the bound


def absmax(X):
    """max|X| without a temporary the size of X."""
    lo, hi = torch.aminmax(X)
    return max(abs(float(lo)), abs(float(hi)))


def bound(n, A, B):
    return TOL_FACTOR * n * absmax(A) * absmax(B)


def run_plan(n, cutoff, sched, A, B, batch=1, **kw):
    plan = Plan(n, cutoff, sched, batch=batch, **kw)
    try:
        C = torch.full_like(A, float("nan"))     # every element must be overwritten
        plan(A, B, out=C)
        torch.cuda.synchronize()
    finally:
        plan.close()
    return C


def check_full(n, cutoff, sched, dist, seed, batch=1, members=None, **kw):
    """Whole-matrix comparison with the classical oracle (for a batch: every member, or those listed)."""
    A, B = inputs.pair(n, dist, seed, device="cuda", batch=None if batch == 1 else batch)
    C = run_plan(n, cutoff, sched, A, B, batch=batch, **kw)
    assert not bool(torch.isnan(C).any()), "some element of C was never written"
    if batch == 1:
        members = [(A.cpu().numpy(), B.cpu().numpy(), C.cpu().numpy())]
    else:
        members = [(A[b].cpu().numpy(), B[b].cpu().numpy(), C[b].cpu().numpy())
                   for b in (range(batch) if members is None else members)]
    worst = 0.0
    for a, b, c in members:
        ref = oracle.classical(a, b)
        if dist == "int8":
            assert np.array_equal(c, ref), "integer-valued inputs must give equal values (max diff %g)" % np.abs(c - ref).max()
        else:
            err = float(np.abs(c - ref).max())
            lim = TOL_FACTOR * n * np.abs(a).max() * np.abs(b).max()
            assert err <= lim, (err, lim)
            assert err <= SANITY_FRACTION * lim, (err, lim)
            worst = max(worst, err / lim)
    return worst


def boundary_indices(level_sizes, extra, seed):
    """Row/column indices that touch every recursion boundary (first/last row of each quadrant
    at every level, the peeled last row) plus random ones."""
    n = level_sizes[0]
    idx = {0, n - 1}
    starts = [0]
    for m, h in zip(level_sizes[:-1], level_sizes[1:]):
        new = []
        for s in starts[:64]:
            for q in (0, 1):
                o = s + q * h
                new.append(o)
                idx.update(i for i in (o, o + h - 1, o + h, s + m - 1) if 0 <= i < n)
        starts = new
    # last rows/columns of the base-product tiles (128 wide) and their ragged tail
    base = level_sizes[-1]
    for t in (127, 128, base - 1, (base // 128) * 128, (base // 128) * 128 - 1):
        if 0 <= t < n:
            idx.add(t)
    rng = np.random.default_rng(seed)
    idx.update(int(i) for i in rng.integers(0, n, extra))
    return np.array(sorted(idx), dtype=np.int64)


def check_sampled(n, cutoff, sched, dist, seed, batch=1, members=(0,), samples=96, **kw):
    """Sampled comparison for sizes where a full classical product is too slow: the block
    C[R, S] for index sets R, S that include every recursion boundary."""
    A, B = inputs.pair(n, dist, seed, device="cuda", batch=None if batch == 1 else batch)
    C = run_plan(n, cutoff, sched, A, B, batch=batch, **kw)
    assert float(C.sum()) == float(C.sum()), "some element of C was never written (NaN fill survives)"
    sizes = oracle.level_sizes(n, cutoff)
    amax, bmax = absmax(A), absmax(B)
    worst = 0.0
    for mb in members:
        a, b, c = (A, B, C) if batch == 1 else (A[mb], B[mb], C[mb])
        R = boundary_indices(sizes, samples, seed + 17 + mb)
        S = boundary_indices(sizes, samples, seed + 29 + mb)
        Rt, St = torch.from_numpy(R).cuda(), torch.from_numpy(S).cuda()
        rows = a.index_select(0, Rt).cpu().numpy()
        cols = b.index_select(1, St).cpu().numpy()
        got = c.index_select(0, Rt).index_select(1, St).cpu().numpy()
        ref = oracle.classical(rows, cols)
        if dist == "int8":
            assert np.array_equal(got, ref), "integer-valued inputs must give equal values"
        else:
            err = float(np.abs(got - ref).max())
            lim = TOL_FACTOR * n * amax * bmax
            assert err <= lim, (err, lim)
            assert err <= SANITY_FRACTION * lim, (err, lim)
            worst = max(worst, err / lim)
    if dist == "int8" and batch == 1:
        # Freivalds on the whole matrix: C x == A (B x) exactly for small integer x
        x = torch.randint(0, 3, (n, 1), device="cuda", generator=torch.Generator("cuda").manual_seed(seed)).double()
        assert torch.equal(C @ x, A @ (B @ x))
    return worst

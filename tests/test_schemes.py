"""Other bilinear schemes through the same BFS / DFS traversal (Section 6.6): the oracle's restatement pinned to the
identities a scheme must satisfy and to the definition of the product; the library's table check and plans on the
host; and the CUDA path against the classical oracle."""
import itertools

import numpy as np
import pytest

import oracle
from paper_1202_3173_b200 import Plan, StrassenError, binding

# the three built-in tables as the header documents them, written down independently of the library
CLASSICAL = (2, 8,
             [[1, 0, 0, 0], [0, 1, 0, 0], [1, 0, 0, 0], [0, 1, 0, 0], [0, 0, 1, 0], [0, 0, 0, 1], [0, 0, 1, 0], [0, 0, 0, 1]],
             [[1, 0, 0, 0], [0, 0, 1, 0], [0, 1, 0, 0], [0, 0, 0, 1], [1, 0, 0, 0], [0, 0, 1, 0], [0, 1, 0, 0], [0, 0, 0, 1]],
             [[1, 1, 0, 0, 0, 0, 0, 0], [0, 0, 1, 1, 0, 0, 0, 0], [0, 0, 0, 0, 1, 1, 0, 0], [0, 0, 0, 0, 0, 0, 1, 1]])
STRASSEN = (2, 7,
            [[1, 0, 0, 1], [0, 0, 1, 1], [1, 0, 0, 0], [0, 0, 0, 1], [1, 1, 0, 0], [-1, 0, 1, 0], [0, 1, 0, -1]],
            [[1, 0, 0, 1], [1, 0, 0, 0], [0, 1, 0, -1], [-1, 0, 1, 0], [0, 0, 0, 1], [1, 1, 0, 0], [0, 0, 1, 1]],
            [[1, 0, 0, 1, -1, 0, 1], [0, 0, 1, 0, 1, 0, 0], [0, 1, 0, 1, 0, 0, 0], [1, -1, 1, 0, 0, 1, 0]])
WINOGRAD = (2, 7,
            [[1, 0, 0, 0], [0, 1, 0, 0], [0, 0, 1, 1], [-1, 0, 1, 1], [1, 0, -1, 0], [1, 1, -1, -1], [0, 0, 0, 1]],
            [[1, 0, 0, 0], [0, 0, 1, 0], [-1, 1, 0, 0], [1, -1, 0, 1], [0, -1, 0, 1], [0, 0, 0, 1], [1, -1, -1, 1]],
            [[1, 1, 0, 0, 0, 0, 0], [1, 0, 1, 1, 0, 1, 0], [1, 0, 0, 1, 1, 0, -1], [1, 0, 1, 1, 1, 0, 0]])
SCHEMES = {"classical": CLASSICAL, "strassen": STRASSEN, "winograd": WINOGRAD}


def redundant_classical():
    """The <2,2,2;8> classical products repeated (12, 8, 4, 4, 9, 9, 9, 9 copies: q = 64) with coefficients that sum to 1 per
    product (+1 / -1 alternating for an odd count, one coefficient 2 for an even one): a legal scheme whose first block of
    C adds 20 products -- more than one launch of the linear-combination kernel takes."""
    n0, q8, u8, v8, w8 = CLASSICAL
    copies = [12, 8, 4, 4, 9, 9, 9, 9]
    u, v, w = [], [], [[] for _ in range(4)]
    for j, n in enumerate(copies):
        coef = [1 if i % 2 == 0 else -1 for i in range(n)]
        if n % 2 == 0:
            coef[0] = 2
        assert sum(coef) == 1
        for c in coef:
            u.append(u8[j]); v.append(v8[j])
            for b in range(4):
                w[b].append(c * w8[b][j])
    return 2, sum(copies), u, v, w


def _ints(n, seed):
    rng = np.random.default_rng(seed)
    return rng.integers(-8, 9, (n, n)).astype(float), rng.integers(-8, 9, (n, n)).astype(float)


# ---- oracle pins ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("scheme", [CLASSICAL, STRASSEN, WINOGRAD, oracle.classical_scheme(2), oracle.classical_scheme(3),
                                    oracle.classical_scheme(4), redundant_classical()])
def test_tables_satisfy_the_bilinear_identities(scheme):
    assert oracle.brent_residual(*scheme) == 0
    n0, q, u, v, w = scheme
    # hand-checkable corner of the identities: exactly n0 products carry A_(0,k) B_(k,0) into C_(0,0)
    coeff = [sum(u[j][k] * v[j][k * n0] * w[0][j] for j in range(q)) for k in range(n0)]
    assert coeff == [1] * n0


def test_a_wrong_sign_or_a_dropped_term_is_seen():
    n0, q, u, v, w = STRASSEN
    bad = [row[:] for row in w]
    bad[0][4] = 1                                   # C11 = M1 + M4 + M5 + M7: wrong sign
    assert oracle.brent_residual(n0, q, u, v, bad) > 0
    bad = [row[:] for row in u]
    bad[5][0] = 0                                   # M6 = A21 (B11 + B12): dropped term
    assert oracle.brent_residual(n0, q, bad, v, w) > 0
    assert oracle.brent_residual(n0, q, v, u, w) > 0          # the two sides are not interchangeable


@pytest.mark.parametrize("scheme,n,cutoff,calls", [(CLASSICAL, 16, 2, 8 ** 3), (STRASSEN, 16, 2, 7 ** 3), (WINOGRAD, 24, 3, 7 ** 3),
                                                   (oracle.classical_scheme(3), 27, 3, 27 ** 2), (STRASSEN, 20, 5, 49),
                                                   (oracle.classical_scheme(4), 16, 4, 64)])
def test_oracle_recursion_equals_the_definition_on_integers(scheme, n, cutoff, calls):
    A, B = _ints(n, n + cutoff)
    C, count = oracle.bilinear_product(A, B, scheme, cutoff)
    assert count == calls                            # q^L base products (Section 6.6: omega_0 = log_n0 q)
    assert np.array_equal(C, oracle.classical(A, B))
    # the Winograd table is Appendix A written out: on integers it agrees with the chained form as well
    if scheme is WINOGRAD:
        C2, cnt = oracle.strassen_winograd(A, B, cutoff)
        assert np.array_equal(C, C2) and cnt["base_calls"] == calls


# ---- the library's host side ----------------------------------------------------------------------------------

def test_library_accepts_correct_tables_and_names_the_broken_identity():
    for s in (CLASSICAL, STRASSEN, WINOGRAD, oracle.classical_scheme(3), redundant_classical()):
        binding.strassen_scheme_check(*s)
    p = Plan(64, 32, "B", scheme=redundant_classical())        # 20, 8, 18, 18 products per block of C: 2 + 1 + 2 + 2 launches
    assert p.launches_by_kind()["lincomb"] == 7 and p.base_products == 64
    p.close()
    n0, q, u, v, w = STRASSEN
    bad = [row[:] for row in w]
    bad[3][1] = 1
    with pytest.raises(StrassenError) as e:
        binding.strassen_scheme_check(n0, q, u, v, bad)
    assert "coefficient" in str(e.value)
    with pytest.raises(StrassenError):
        Plan(64, 16, "BB", scheme=(n0, q, u, v, bad))
    with pytest.raises(StrassenError):
        Plan(64, 16, "BB", scheme="karatsuba")


def test_scheme_plans_on_the_host():
    for name, (n0, q, u, v, w) in SCHEMES.items():
        p = Plan(512, 64, "BDB", scheme=name)
        assert p.level_sizes == [512, 256, 128, 64] and p.schedule == "BDB" and p.base_products == q ** 3
        k = p.launches_by_kind()
        assert k["lincomb"] > 0 and k["form"] == 0 and k["recombine"] == 0 and k["gemm"] == q      # one product launch per DFS sub-tree
        # a table given explicitly plans like the built-in of the same name
        p2 = Plan(512, 64, "BDB", scheme=(n0, q, u, v, w))
        assert p2.workspace_bytes == p.workspace_bytes and p2.launch_count == p.launch_count
        p.close(); p2.close()
    # the recursive classical algorithm needs no sums: every operand is a block used in place, only products are stored
    p = Plan(256, 128, "B", scheme="classical")
    assert p.workspace_bytes == 8 * 8 * 128 * 128 and p.launches_by_kind()["lincomb"] == 4
    p.close()
    p = Plan(243, 9, "BBB", scheme=oracle.classical_scheme(3))
    assert p.level_sizes == [243, 81, 27, 9] and p.base_products == 27 ** 3
    p.close()
    with pytest.raises(StrassenError) as e:
        Plan(250, 9, "BBB", scheme=oracle.classical_scheme(3))          # 250 is not divisible by 3: no peeling
    assert "divisible" in str(e.value)
    with pytest.raises(StrassenError):
        Plan(512, 64, "BB", scheme="strassen")                          # three levels need three characters
    # Limited-Memory rule for a scheme: the fewest leading DFS steps whose workspace fits
    p = Plan(1024, 128, None, scheme="strassen", workspace_budget_bytes=int(40e6))
    assert p.schedule in ("DBB", "DDB", "DDD") and p.workspace_bytes <= 40e6
    q = Plan(1024, 128, None, scheme="strassen", workspace_budget_bytes=int(1e9))
    assert q.schedule == "BBB"
    p.close(); q.close()


# ---- CUDA path -------------------------------------------------------------------------------------------------

@pytest.mark.gpu
@pytest.mark.parametrize("name,n,cutoff", [("classical", 256, 32), ("strassen", 256, 32), ("winograd", 264, 33), ("strassen", 40, 5)])
def test_built_in_schemes_give_the_product_for_every_schedule(name, n, cutoff):
    import torch
    from paper_1202_3173_b200 import inputs
    L = len(oracle.level_sizes(n, cutoff)) - 1
    A, B = inputs.pair(n, "int8", 70 + n, device="cuda")
    ref = oracle.classical(A.cpu().numpy(), B.cpu().numpy())
    for sched in ("".join(s) for s in itertools.product("BD", repeat=L)):
        plan = Plan(n, cutoff, sched, scheme=name)
        C = torch.full_like(A, float("nan"))
        plan(A, B, out=C)
        torch.cuda.synchronize()
        plan.close()
        assert np.array_equal(C.cpu().numpy(), ref), (name, sched)


@pytest.mark.gpu
@pytest.mark.parametrize("scheme,n,cutoff,sched,batch", [("strassen", 1024, 128, "BBB", 1), ("classical", 1024, 256, "BD", 1),
                                                         (oracle.classical_scheme(3), 729, 81, "BD", 1),
                                                         (oracle.classical_scheme(4), 512, 32, "DB", 2),
                                                         ("winograd", 1030, 515, "B", 3), ("strassen", 2048, 256, "DBB", 1),
                                                         (redundant_classical(), 256, 64, "BD", 1)])
def test_schemes_on_float_data_meet_the_bound(scheme, n, cutoff, sched, batch):
    import torch
    from paper_1202_3173_b200 import inputs
    A, B = inputs.pair(n, "uniform", 90 + n, device="cuda", batch=None if batch == 1 else batch)
    plan = Plan(n, cutoff, sched, batch=batch, scheme=scheme)
    C = torch.full_like(A, float("nan"))
    plan(A, B, out=C)
    torch.cuda.synchronize()
    plan.close()
    members = [(A, B, C)] if batch == 1 else [(A[b], B[b], C[b]) for b in range(batch)]
    for a, b, c in members:
        ref = oracle.classical(a.cpu().numpy(), b.cpu().numpy())
        err = float(np.abs(c.cpu().numpy() - ref).max())
        lim = 1e-11 * n * float(a.abs().max()) * float(b.abs().max())
        assert err <= 0.02 * lim, (err, lim)
    # the oracle's recursion of the same scheme lands within the same bound of the CUDA result
    if batch == 1 and n <= 1100:
        sch = SCHEMES[scheme] if isinstance(scheme, str) else scheme
        want, _ = oracle.bilinear_product(A.cpu().numpy(), B.cpu().numpy(), sch, cutoff)
        assert float(np.abs(C.cpu().numpy() - want).max()) <= 0.02 * lim


@pytest.mark.gpu
def test_winograd_table_agrees_with_the_chained_plan_on_integers_and_graph_replay_works():
    import torch
    from paper_1202_3173_b200 import inputs
    n, cutoff, sched = 512, 64, "BDB"
    A, B = inputs.pair(n, "int8", 5, device="cuda")
    chained = Plan(n, cutoff, sched)
    table = Plan(n, cutoff, sched, scheme="winograd", flags=binding.STRASSEN_FLAG_CUDA_GRAPH)
    want = chained(A, B).clone()
    for _ in range(3):
        got = table(A, B)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
    chained.close(); table.close()


@pytest.mark.gpu
def test_scheme_plan_through_the_host_entry_point():
    import torch
    from paper_1202_3173_b200 import inputs
    n = 192
    A, B = inputs.pair(n, "int8", 77, device="cpu")
    A, B = A.pin_memory(), B.pin_memory()
    for flags in (0, binding.STRASSEN_FLAG_HOST_PIPELINE):
        plan = Plan(n, 24, "BDB", scheme="classical", flags=flags)
        C = torch.full((n, n), float("nan"), dtype=torch.float64).pin_memory()
        for _ in range(2):
            plan.run_host(A, B, C)
        torch.cuda.synchronize()
        plan.close()
        assert np.array_equal(C.numpy(), oracle.classical(A.numpy(), B.numpy()))
    with pytest.raises(StrassenError):
        Plan(n, 24, "BDB", scheme="classical", flags=binding.STRASSEN_FLAG_SCALE_OUTSIDE)     # not for generic schemes

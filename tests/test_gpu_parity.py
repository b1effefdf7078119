"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Integer-valued inputs in [-8, 8]: every intermediate is an exact integer, values must be
equal.  Float inputs: max|C - C_ref| <= 1e-11 * n * max|A| * max|B|, the reference being the
classical definition computed by the oracle."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_1202_3173_b200 import Plan, StrassenError, binding, inputs
from tests.gpu_util import bound, check_full, check_sampled, run_plan

pytestmark = pytest.mark.gpu
GB = 1e9


def _free_bytes():
    torch.cuda.empty_cache()        # memory cached by earlier tests counts as free
    return torch.cuda.mem_get_info()[0]


# ---- base products alone (zero levels), ragged sizes, one and many per launch ----------

@pytest.mark.parametrize("n", [1, 2, 3, 7, 16, 17, 100, 127, 128, 129, 255, 256, 300, 515])
@pytest.mark.parametrize("dist", ["int8", "uniform"])
def test_base_product_sizes(n, dist):
    check_full(n, max(n, 1), "", dist, 100 + n)


@pytest.mark.parametrize("n", [65, 72, 136, 194, 260, 388, 771])
def test_base_product_thin_remainders(n):
    """Sizes 1..8 past a multiple of 64: tiled bulk plus thin products for the last rows / columns."""
    check_full(n, n, "", "int8", 300 + n)
    check_full(n, n, "", "normal", 301 + n, batch=3)


@pytest.mark.parametrize("n,cutoff,sched,batch", [(262, 131, "B", 1), (1542, 771, "B", 2), (393, 196, "B", 1), (526, 131, "BB", 3),
                                                  (1050, 131, "BBB", 1), (524, 131, "BB", 1), (1048, 131, "BBB", 2), (525, 131, "DB", 1)])
def test_thin_remainders_of_sibling_base_products(n, cutoff, sched, batch):
    """Base products that are the seven children of BFS parents get their remainder rows and columns per parent, from
    the parent's quadrants: after a BFS step of its own (262, 1542, odd parent 393, below a DFS step 525) and after the
    pair with an odd lower member (526: 263 odd).  The even two- and three-level passes (524, 1048) leave one
    quadrant of the intermediate sums unwritten, so their leaves keep the per-leaf products.  Three-launch path."""
    no_fused_step = 128
    p = Plan(n, cutoff, sched, batch=batch, flags=no_fused_step)
    assert p.launches_by_kind()["gemm"] >= 3          # tiled bulk + two thin launches
    p.close()
    check_full(n, cutoff, sched, "int8", 330 + n, batch=batch, flags=no_fused_step)
    check_full(n, cutoff, sched, "uniform", 331 + n, batch=batch, flags=no_fused_step)


@pytest.mark.parametrize("n,cutoff,sched", [(4100, 4100, ""), (8197, 4100, "B")])
def test_thin_products_over_one_large_node(n, cutoff, sched):
    """A single node with an inner dimension of 4096 or more: its thin products give each CTA 8 rows (columns) and split
    the inner dimension over the CTA's warps.  4100 = 64 x 64 + 4: remainder columns and rows of one base product;
    8197: the peeled last column and row of the root (its children, 4098 = 64 x 64 + 2, are one set of siblings)."""
    check_sampled(n, cutoff, sched, "int8", 350 + n)
    check_sampled(n, cutoff, sched, "uniform", 351 + n)


@pytest.mark.parametrize("n,cutoff,sched,batch", [(4480, 560, "BBB", 1), (2400, 300, "BBB", 2), (4481, 560, "BBB", 1)])
def test_base_product_margin_strips(n, cutoff, sched, batch):
    # a base size 1..64 past a multiple of 128 with hundreds of leaves: 128 x 128 tiles over the multiple, a right
    # and a bottom strip of 64 x 64 tiles over the margin (560 = 512 + 48, 300 = 256 + 44; 4481: leaves that are
    # views with an odd leading dimension)
    p = Plan(n, cutoff, sched, batch=batch)
    assert p.launches_by_kind()["gemm"] >= 3
    p.close()
    members = (0,) if batch == 1 else (0, batch - 1)
    check_sampled(n, cutoff, sched, "int8", 640 + n, batch=batch, members=members)
    check_sampled(n, cutoff, sched, "uniform", 641 + n, batch=batch, members=members)


@pytest.mark.parametrize("n,batch,dist", [(300, 70, "int8"), (192, 100, "uniform"), (560, 40, "int8")])
def test_base_product_batches_with_a_margin(n, batch, dist):
    check_full(n, n, "", dist, 650 + n, batch=batch)


def test_base_product_split_between_tile_shapes():
    # 5 x 30 x 30... enough 128-tiles for >= 4 full rounds of 148 plus a short tail that moves to 64 x 64 tiles
    check_full(512, 512, "", "int8", 77, batch=38)       # 608 tiles = 4 rounds + 16
    check_full(256, 256, "", "uniform", 78, batch=150)   # 600 tiles = 4 rounds + 8


def test_base_product_batch_spans_many_tiles():
    check_full(200, 256, "", "int8", 7, batch=40)
    check_full(384, 512, "", "uniform", 8, batch=9)


# ---- tiny recursions: every schedule string -----------------------------------------------

@pytest.mark.parametrize("n,cutoff", [(2, 1), (4, 1), (8, 2), (16, 2), (24, 3), (64, 8)])
def test_every_schedule_string_small(n, cutoff):
    L = len(oracle.level_sizes(n, cutoff)) - 1
    for sched in ("".join(s) for s in itertools.product("BD", repeat=L)):
        check_full(n, cutoff, sched, "int8", 11 * n + L)
    check_full(n, cutoff, "B" * L, "uniform", 5 * n)
    check_full(n, cutoff, "D" * L, "normal", 5 * n + 1)


@pytest.mark.parametrize("n,cutoff", [(3, 1), (5, 2), (7, 3), (9, 2), (15, 3), (17, 4), (31, 7), (33, 8), (57, 3),
                                      (197, 12), (101, 25)])
def test_peeling_small(n, cutoff):
    L = len(oracle.level_sizes(n, cutoff)) - 1
    for sched in {"B" * L, "D" * L, ("BD" * L)[:L], ("DB" * L)[:L]}:
        check_full(n, cutoff, sched, "int8", 3 * n)
    check_full(n, cutoff, "B" * L, "uniform", 3 * n + 1)


# ---- the small configuration and mid sizes spanning several tiles ---------------------------

def test_config_n512_one_level():
    check_full(512, 256, "B", "int8", 1002)
    r = check_full(512, 256, "B", "uniform", 1001)
    assert r < 1e-3        # calibration: about 1e-5 of the bound at one level
    check_full(512, 256, "D", "int8", 1002)


@pytest.mark.parametrize("n,cutoff,sched", [(1024, 128, "BBB"), (1024, 128, "DBD"), (1024, 128, "BDB"),
                                            (1024, 256, "DD"), (768, 96, "BBB"), (1000, 125, "DBB"),
                                            (771, 96, "BBB"), (1543, 192, "BDB"), (2048, 512, "BB")])
def test_mid_sizes(n, cutoff, sched):
    check_full(n, cutoff, sched, "int8", n + 1)
    check_full(n, cutoff, sched, "uniform", n + 2)


def test_batch_of_products():
    check_full(256, 64, "BB", "int8", 21, batch=4)
    check_full(320, 80, "DB", "uniform", 22, batch=3)
    check_full(129, 32, "BB", "int8", 23, batch=5)      # odd size inside a batch


def test_leading_dimensions_and_strides():
    n, ld, batch = 96, 101, 2            # odd leading dimension: 8-byte-aligned rows only
    g = torch.Generator("cuda").manual_seed(5)
    A = torch.randint(-8, 9, (batch, n + 3, ld), device="cuda", generator=g).double()
    B = torch.randint(-8, 9, (batch, n + 3, ld), device="cuda", generator=g).double()
    C = torch.full((batch, n + 3, ld), 777.0, device="cuda", dtype=torch.float64)
    stride = (n + 3) * ld
    plan = Plan(n, 12, "BDB", batch=batch, lda=ld, ldb=ld, ldc=ld, stride_a=stride, stride_b=stride, stride_c=stride)
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device="cuda")
    binding.strassen_plan_set_workspace(plan.handle, ws.data_ptr(), plan.workspace_bytes)
    binding.strassen_dgemm(plan.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    plan.close()
    for b in range(batch):
        ref = oracle.classical(A[b, :n, :n].cpu().numpy(), B[b, :n, :n].cpu().numpy())
        assert np.array_equal(C[b, :n, :n].cpu().numpy(), ref)
    assert bool((C[:, n:, :] == 777.0).all()) and bool((C[:, :, n:] == 777.0).all())   # nothing outside n x n


def test_random_sizes_cutoffs_and_schedules():
    """Seeded sweep over odd and even sizes, cutoffs and B/D strings: exact on integer inputs."""
    rng = np.random.default_rng(2024)
    for case in range(48):
        n = int(rng.integers(1, 420))
        cutoff = int(rng.integers(1, max(2, n)))
        if n // max(cutoff, 1) > 64:            # keep the tree small: at most 6 levels
            cutoff = max(cutoff, n // 64 + 1)
        L = len(oracle.level_sizes(n, cutoff)) - 1
        sched = "".join(rng.choice(list("BD"), size=L))
        batch = int(rng.integers(1, 4))
        # alternate between the default plan (small deepest BFS steps run fused), the three-launch form of every step,
        # and separate fold passes in every DFS step
        flags = (0, binding.STRASSEN_FLAG_NO_FUSED_STEP, binding.STRASSEN_FLAG_NO_FUSED_STEP | binding.STRASSEN_FLAG_NO_DFS_FOLD,
                 binding.STRASSEN_FLAG_FUSED_STEP)[case % 4]
        check_full(n, cutoff, sched, "int8", 9000 + case, batch=batch, flags=flags)


def test_timed_random_sweep_over_plan_variants():
    """Random sizes, cutoffs, B/D strings, batches, padded leading dimensions and plan flags (multi-level pass caps, fused
    step on / off, separate fold passes, graph replay) against the classical oracle, for STRASSEN_FUZZ_SECONDS seconds
    (default 5; the build's long runs used 300 per seed).  Exact on integer data, within 2 % of the bound on floats."""
    import os
    import time
    budget = float(os.environ.get("STRASSEN_FUZZ_SECONDS", "5"))
    rng = np.random.default_rng(int(os.environ.get("STRASSEN_FUZZ_SEED", "3")))
    flag_sets = [0, 1, 32, 64, 128, 256, 64 | 256, 128 | 256, 1 | 128, 32 | 64, 2, 2 | 64]
    stream = torch.cuda.current_stream().cuda_stream
    t0, cases = time.time(), 0
    while time.time() - t0 < budget or cases < 20:
        n = int(rng.integers(1, 900)) if rng.integers(0, 4) else int(rng.integers(1, 70))
        cutoff = int(rng.integers(1, max(2, n)))
        if n // max(cutoff, 1) > 48:
            cutoff = max(cutoff, n // 48 + 1)
        L = len(oracle.level_sizes(n, cutoff)) - 1
        sched = "".join(rng.choice(list("BD"), size=L))
        flags = int(rng.choice(flag_sets))
        batch = int(rng.integers(1, 4))
        pad = int(rng.integers(0, 3)) if batch == 1 else 0
        dist = "int8" if rng.integers(0, 5) else "uniform"
        what = (n, cutoff, sched, batch, flags, pad, dist)
        if pad:
            ld = n + pad
            g = torch.Generator("cuda").manual_seed(int(rng.integers(1 << 30)))
            A = torch.randint(-8, 9, (n, ld), device="cuda", generator=g).double()
            B = torch.randint(-8, 9, (n, ld), device="cuda", generator=g).double()
            C = torch.full((n, ld), 7.5, device="cuda", dtype=torch.float64)
            plan = Plan(n, cutoff, sched, lda=ld, ldb=ld, ldc=ld, flags=flags)
            ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
            binding.strassen_plan_set_workspace(plan.handle, ws.data_ptr(), plan.workspace_bytes)
            binding.strassen_dgemm(plan.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), stream)
            torch.cuda.synchronize()
            plan.close()
            ref = oracle.classical(A[:, :n].cpu().numpy().copy(), B[:, :n].cpu().numpy().copy())
            assert np.array_equal(C[:, :n].cpu().numpy(), ref) and bool((C[:, n:] == 7.5).all()), what
        else:
            check_full(n, cutoff, sched, dist, int(rng.integers(1 << 30)), batch=batch, flags=flags)
        cases += 1


def test_pointers_that_are_only_8_byte_aligned():
    n = 258
    g = torch.Generator("cuda").manual_seed(77)
    store = [torch.randint(-8, 9, (n * n + 1,), device="cuda", generator=g).double() for _ in range(2)]
    out = torch.zeros(n * n + 1, device="cuda", dtype=torch.float64)
    A, B, C = store[0][1:].view(n, n), store[1][1:].view(n, n), out[1:].view(n, n)     # offset by one element
    assert A.data_ptr() % 16 == 8
    for cutoff, sched in ((n, ""), (129, "B"), (33, "BBB"), (65, "DB")):
        plan = Plan(n, cutoff, sched)
        C.fill_(float("nan"))
        binding.strassen_dgemm(plan.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        plan.close()
        assert np.array_equal(C.cpu().numpy(), oracle.classical(A.cpu().numpy(), B.cpu().numpy())), (cutoff, sched)
    assert float(out[0]) == 0.0


@pytest.mark.parametrize("n,cutoff,sched,batch", [(771, 96, "BBB", 1), (520, 65, "DBB", 2), (1000, 125, "BDB", 1), (301, 80, "DB", 3)])
def test_nothing_is_written_outside_the_workspace_or_c(n, cutoff, sched, batch):
    """Guard words before and after the workspace and after C keep their pattern; padding inside the
    workspace rows aside, every byte the library may touch is inside what it was given."""
    plan = Plan(n, cutoff, sched, batch=batch)
    need = plan.workspace_bytes
    guard = 4096
    raw = torch.full((need + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    ws = raw[guard:guard + need]
    assert ws.data_ptr() % 256 == 0
    binding.strassen_plan_set_workspace(plan.handle, ws.data_ptr(), need)
    A, B = inputs.pair(n, "int8", 31 + n, device="cuda", batch=None if batch == 1 else batch)
    cbuf = torch.full((batch * n * n + 512,), -123.0, dtype=torch.float64, device="cuda")
    C = cbuf[:batch * n * n].view(A.shape)
    binding.strassen_dgemm(plan.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    plan.close()
    assert bool((raw[:guard] == 0x5A).all()) and bool((raw[guard + need:] == 0x5A).all())
    assert bool((cbuf[batch * n * n:] == -123.0).all())
    members = [(A, B, C)] if batch == 1 else [(A[b], B[b], C[b]) for b in range(batch)]
    for a, b, c in members:
        assert np.array_equal(c.cpu().numpy(), oracle.classical(a.cpu().numpy(), b.cpu().numpy()))


def test_inputs_are_not_written_and_calls_repeat():
    A, B = inputs.pair(640, "uniform", 31, device="cuda")
    A0, B0 = A.clone(), B.clone()
    plan = Plan(640, 80, "BDB")
    C1 = plan(A, B).clone()
    C2 = plan(A, B)
    torch.cuda.synchronize()
    plan.close()
    assert torch.equal(A, A0) and torch.equal(B, B0)
    assert torch.equal(C1, C2)          # same plan, same inputs: same bits


@pytest.mark.parametrize("n,cutoff,sched,dist", [(1024, 128, "BBB", "uniform"), (1024, 256, "BB", "normal"),
                                                 (512, 32, "BBBB", "uniform"), (520, 65, "BBB", "uniform"),
                                                 (1030, 64, "BDBB", "uniform"), (771, 96, "BBB", "uniform"),
                                                 (197, 12, "BBBB", "uniform"), (36, 9, "BB", "int8"),
                                                 (1544, 193, "DBB", "normal")])
def test_two_level_passes_give_the_same_bits_as_single_level_passes(n, cutoff, sched, dist):
    A, B = inputs.pair(n, dist, n + 7, device="cuda")
    fused = run_plan(n, cutoff, sched, A, B)
    two = run_plan(n, cutoff, sched, A, B, flags=binding.STRASSEN_FLAG_TWO_LEVEL_PASSES)
    single = run_plan(n, cutoff, sched, A, B, flags=binding.STRASSEN_FLAG_SINGLE_LEVEL_PASSES)
    assert torch.equal(fused, single)      # same operations in the same order
    assert torch.equal(two, single)
    p1, p2 = Plan(n, cutoff, sched), Plan(n, cutoff, sched, flags=binding.STRASSEN_FLAG_SINGLE_LEVEL_PASSES)
    assert p1.launch_count <= p2.launch_count
    p1.close(); p2.close()


@pytest.mark.parametrize("n,cutoff,sched,dist", [(2048, 256, "BBB", "uniform"), (1025, 128, "BBB", "normal"),
                                                 (72, 9, "BBB", "int8"), (2064, 129, "BBBB", "uniform"),
                                                 (1536, 24, "BBBBBB", "uniform"), (1041, 65, "DBBB", "uniform")])
def test_three_level_passes_cover_odd_parents_ragged_tiles_and_stacked_groups(n, cutoff, sched, dist):
    # 1025, 1041: odd size at or above the group (rank-one term inside the three-level recombination); 72: a lattice
    # block of 9 x 9, far below one CTA tile; 2064 -> 129: a single level above a group of three with odd base;
    # 1536 -> 24: two groups of three on top of each other
    A, B = inputs.pair(n, dist, n + 11, device="cuda")
    fused = run_plan(n, cutoff, sched, A, B)
    single = run_plan(n, cutoff, sched, A, B, flags=binding.STRASSEN_FLAG_SINGLE_LEVEL_PASSES)
    assert torch.equal(fused, single)
    check_full(n, cutoff, sched, dist, n + 11)          # and the oracle's definition, whole matrix


@pytest.mark.parametrize("n,cutoff,sched,batch,dist", [
    (6, 1, "BB", 2, "int8"),            # children of size 3, grandchildren of size 1
    (14, 3, "BB", 1, "int8"), (1030, 257, "BB", 1, "uniform"), (1542, 385, "BB", 2, "normal"),
    (771, 96, "BBB", 1, "uniform"),     # odd parent with odd children: both rank-one terms in one recombination
    (2060, 128, "BBBB", 1, "int8"),     # 2060 -> 1030 -> 515 (odd) -> 257 (odd) -> 128: pair (1,2), level 3 alone below it
    (3086, 771, "BB", 1, "uniform"),    # the deepest pair of the n=12345 tree
    (1034, 129, "DBB", 1, "int8"), (2068, 129, "BDBB", 1, "int8"),
])
def test_pair_of_levels_with_odd_children_gives_the_bits_of_single_level_passes(n, cutoff, sched, batch, dist):
    A, B = inputs.pair(n, dist, n + 13, device="cuda", batch=None if batch == 1 else batch)
    paired = run_plan(n, cutoff, sched, A, B, batch=batch, flags=UNFUSED)
    single = run_plan(n, cutoff, sched, A, B, batch=batch, flags=UNFUSED | binding.STRASSEN_FLAG_SINGLE_LEVEL_PASSES)
    assert torch.equal(paired, single)
    p, q = Plan(n, cutoff, sched, batch=batch, flags=UNFUSED), Plan(n, cutoff, sched, batch=batch,
                                                                  flags=UNFUSED | binding.STRASSEN_FLAG_SINGLE_LEVEL_PASSES)
    assert p.launches_by_kind()["form"] < q.launches_by_kind()["form"]
    p.close(); q.close()
    check_full(n, cutoff, sched, dist, n + 13, batch=batch, flags=UNFUSED)


def test_batch_with_two_level_passes():
    check_full(256, 64, "BB", "uniform", 121, batch=6)
    check_full(260, 65, "BB", "int8", 122, batch=3)      # odd quarter size: 8-byte accesses


# ---- the deepest BFS step as one fused kernel ------------------------------------------------

FUSED, UNFUSED = binding.STRASSEN_FLAG_FUSED_STEP, binding.STRASSEN_FLAG_NO_FUSED_STEP


@pytest.mark.parametrize("n,cutoff,sched,batch,dist", [
    (512, 256, "B", 1, "uniform"), (512, 256, "B", 1, "int8"),      # the small configuration: 128 CTAs of the small tile
    (64, 32, "B", 1, "int8"), (2, 1, "B", 3, "int8"), (6, 3, "B", 1, "int8"), (3, 1, "B", 2, "int8"), (7, 3, "B", 1, "int8"),
    (33, 16, "B", 1, "normal"),
    (100, 50, "B", 2, "normal"),        # ragged tiles in both directions, inner dimension not a multiple of 16
    (101, 50, "B", 2, "int8"),          # odd parent: rank-one term inside the kernel, then the peeled column and row
    (258, 129, "B", 1, "int8"),         # odd quadrant size: 8-byte copies only
    (1024, 512, "B", 1, "uniform"),     # the wide tile
    (1030, 515, "B", 1, "int8"), (777, 388, "B", 1, "uniform"),
    (1024, 128, "BBB", 1, "uniform"),   # two-level pass above a fused deepest step
    (1000, 125, "DBB", 1, "int8"), (520, 65, "BDB", 2, "int8"), (771, 96, "BBB", 1, "int8"),
    (4096, 512, "BBB", 1, "uniform"),
])
def test_fused_step_agrees_with_the_three_launch_path(n, cutoff, sched, batch, dist):
    A, B = inputs.pair(n, dist, 40 + n, device="cuda", batch=None if batch == 1 else batch)
    fused = run_plan(n, cutoff, sched, A, B, batch=batch, flags=FUSED)
    plain = run_plan(n, cutoff, sched, A, B, batch=batch, flags=UNFUSED)
    if dist == "int8":
        assert torch.equal(fused, plain)             # same operations on every element, exact on integers
    else:       # the inner dimension is summed in another order (two partial sums per product; thin remainders)
        assert float((fused - plain).abs().max()) <= 1e-4 * bound(n, A, B)
    p = Plan(n, cutoff, sched, batch=batch, flags=FUSED)
    assert p.launches_by_kind()["fused_step"] >= 1 and p.launches_by_kind()["gemm"] == 0
    p.close()
    if n <= 2100:
        check_full(n, cutoff, sched, dist, 40 + n, batch=batch, flags=FUSED)
    else:
        check_sampled(n, cutoff, sched, dist, 40 + n, batch=batch, flags=FUSED)


def test_fused_step_launched_as_a_dependent_keeps_stream_order():
    """The fused step is launched with programmatic stream serialisation: its CTAs may be placed while the launch
    before it still runs, but every global access waits for that launch.  Inputs rewritten by other kernels between
    products, outputs overwritten by the next product, and a consumer kernel behind each product must all see
    stream order."""
    n, steps = 512, 24
    g = torch.Generator("cuda").manual_seed(5)
    A = torch.randint(-3, 4, (n, n), device="cuda", generator=g).double()
    B = torch.randint(-3, 4, (n, n), device="cuda", generator=g).double()
    A0, B0 = A.cpu().numpy().copy(), B.cpu().numpy().copy()
    plan = Plan(n, 256, "B", flags=FUSED)
    assert plan.launches_by_kind() == {**{k: 0 for k in plan.launches_by_kind()}, "fused_step": 1}
    C = torch.empty_like(A)
    sums = torch.zeros(steps, dtype=torch.float64, device="cuda")
    kept = []
    for i in range(steps):
        A.add_(1.0)                      # another kernel rewrites an input right before the product ...
        plan(A, B, out=C)                # ... the product overwrites the output of the one before it ...
        sums[i] = C.sum()                # ... and a consumer reads it right behind
        if i % 8 == 7:
            kept.append((i, C.clone()))
        B.sub_(1.0)                      # and the other input changes before the next product
    torch.cuda.synchronize()
    plan.close()
    for i in range(steps):
        ref = oracle.classical(A0 + (i + 1), B0 - i)
        assert float(sums[i]) == float(ref.sum()), i
        for k, c in kept:
            if k == i:
                assert np.array_equal(c.cpu().numpy(), ref), i


def test_fused_step_on_pointers_that_are_only_8_byte_aligned_and_strided_views():
    n, ld = 130, 137
    g = torch.Generator("cuda").manual_seed(9)
    Abuf = torch.randint(-8, 9, (n * ld + 1,), device="cuda", generator=g).double()
    Bbuf = torch.randint(-8, 9, (n * ld + 1,), device="cuda", generator=g).double()
    Cbuf = torch.full((n * ld + 1,), 55.0, device="cuda", dtype=torch.float64)
    A, B, C = (x[1:].view(n, ld) for x in (Abuf, Bbuf, Cbuf))
    plan = Plan(n, 65, "B", lda=ld, ldb=ld, ldc=ld, flags=FUSED)
    assert plan.launches_by_kind()["fused_step"] == 1
    binding.strassen_dgemm(plan.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    plan.close()
    ref = oracle.classical(A[:, :n].cpu().numpy().copy(), B[:, :n].cpu().numpy().copy())
    assert np.array_equal(C[:, :n].cpu().numpy(), ref)
    assert bool((C[:, n:] == 55.0).all()) and float(Cbuf[0]) == 55.0


def test_cuda_graph_replay_matches_launch_by_launch():
    n = 512
    A, B = inputs.pair(n, "uniform", 131, device="cuda")
    A2, B2 = inputs.pair(n, "int8", 133, device="cuda")
    for cutoff, sched in ((256, "B"), (64, "DBD"), (32, "DDDD")):
        eager = Plan(n, cutoff, sched)
        graph = Plan(n, cutoff, sched, flags=binding.STRASSEN_FLAG_CUDA_GRAPH)
        want = eager(A, B).clone()
        C = torch.empty_like(A)
        for _ in range(3):                       # capture on the first call, replay afterwards
            C.fill_(float("nan"))
            graph(A, B, out=C)
            torch.cuda.synchronize()
            assert torch.equal(C, want)
        # other pointers: the graph is captured again and stays correct
        C2 = graph(A2, B2)
        torch.cuda.synchronize()
        assert np.array_equal(C2.cpu().numpy(), oracle.classical(A2.cpu().numpy(), B2.cpu().numpy()))
        graph(A, B, out=C)
        torch.cuda.synchronize()
        assert torch.equal(C, want)
        eager.close(); graph.close()


@pytest.mark.parametrize("n,cutoff,sched,dist", [
    (1024, 256, "DB", "uniform"),       # sub-problems end in a one-level recombination
    (4128, 129, "DBBBB", "uniform"),    # ... one level above a three-level pass
    (4129, 129, "DBBBB", "int8"),       # odd DFS parent: the first fold carries the rank-one term of the peeled split
    (1025, 256, "DB", "int8"), (1028, 257, "DB", "normal"),
    (520, 65, "DDB", "int8"), (1024, 128, "BDB", "uniform"), (260, 65, "DB", "int8"),
])
def test_dfs_fold_inside_the_recombination_matches_the_separate_fold_pass(n, cutoff, sched, dist):
    A, B = inputs.pair(n, dist, 60 + n, device="cuda")
    through = run_plan(n, cutoff, sched, A, B, flags=UNFUSED)
    separate = run_plan(n, cutoff, sched, A, B, flags=UNFUSED | binding.STRASSEN_FLAG_NO_DFS_FOLD)
    assert torch.equal(through, separate)          # the same operations in the same order on every element of C
    p, q = Plan(n, cutoff, sched, flags=UNFUSED), Plan(n, cutoff, sched, flags=UNFUSED | binding.STRASSEN_FLAG_NO_DFS_FOLD)
    assert p.launches_by_kind()["accumulate"] < q.launches_by_kind()["accumulate"]
    p.close(); q.close()
    check_full(n, cutoff, sched, dist, 60 + n, flags=UNFUSED)


def test_schedules_agree_exactly_on_integers():
    A, B = inputs.pair(512, "int8", 41, device="cuda")
    outs = [run_plan(512, 64, s, A, B) for s in ("BBB", "DDD", "BDB", "DBD")]
    for o in outs[1:]:
        assert torch.equal(outs[0], o)


def test_errors_on_device():
    A, B = inputs.pair(64, "uniform", 1, device="cuda")
    plan = Plan(64, 16, "BB")
    with pytest.raises(StrassenError) as e:
        binding.strassen_dgemm(plan.handle, A.data_ptr(), B.data_ptr(), A.data_ptr(), 0)
    assert e.value.status == -4
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(StrassenError) as e:
        binding.strassen_plan_set_workspace(plan.handle, small.data_ptr(), 1024)
    assert e.value.status == -3
    # a workspace that overlaps an operand is refused before anything is launched
    need = plan.workspace_bytes
    big = torch.zeros(need // 8 + 64 * 64 + 64, dtype=torch.float64, device="cuda")
    Ain = big[need // 8 - 32: need // 8 - 32 + 64 * 64].view(64, 64)        # starts inside the workspace range
    assert big.data_ptr() % 256 == 0
    binding.strassen_plan_set_workspace(plan.handle, big.data_ptr(), need)
    C = torch.empty_like(B)
    with pytest.raises(StrassenError) as e:
        binding.strassen_dgemm(plan.handle, Ain.data_ptr(), B.data_ptr(), C.data_ptr(), 0)
    assert e.value.status == -4 and "workspace" in str(e.value)
    plan.close()


@pytest.mark.parametrize("n,cutoff,sched,flags", [(2048, 16, "BBBBBBB", 0), (2048, 16, "BBBBBBB", 1), (1024, 8, "BBBBBBB", 32),
                                                  (2048, 16, "BBBBBBB", 64)])      # 64: 117 649 parents through the fused step
def test_item_lists_longer_than_one_launch_covers(n, cutoff, sched, flags):
    # 7^6 = 117 649 parents at the deepest level and 7^7 = 823 543 leaves: the streaming kernels and the thin
    # products (8 x 8 leaves are all remainder) cut their item lists into launches of at most 32 768 items
    if _free_bytes() < 12 * GB:
        pytest.skip("needs 8 GB")
    A, B = inputs.pair(n, "int8", 900 + n + flags, device="cuda")
    C = run_plan(n, cutoff, sched, A, B, flags=flags)
    assert np.array_equal(C.cpu().numpy(), oracle.classical(A.cpu().numpy(), B.cpu().numpy()))


@pytest.mark.parametrize("n", [700, 1500, 3001])
def test_library_chosen_plan_gives_the_product(n):
    # cutoff 0, schedule None: steps and interleaving picked by the cost model against the free device memory
    from paper_1202_3173_b200 import matmul
    A, B = inputs.pair(n, "int8", 2900 + n, device="cuda")
    C = matmul(A, B)
    x = torch.randint(0, 3, (n, 1), device="cuda", generator=torch.Generator("cuda").manual_seed(n)).double()
    assert torch.equal(C @ x, A @ (B @ x))              # Freivalds, exact on small integers
    if n <= 1500:
        assert np.array_equal(C.cpu().numpy(), oracle.classical(A.cpu().numpy(), B.cpu().numpy()))


def test_first_call_on_a_side_stream_sees_its_node_tables():
    # 137 257 nodes (6.6 MB of tables) uploaded by the first call, which is made on a non-blocking stream while
    # another stream keeps the host-to-device copy engine busy: the product must wait for its own tables
    n, cutoff, sched = 1024, 16, "BBBBBB"
    A, B = inputs.pair(n, "int8", 4242, device="cuda")
    torch.cuda.synchronize()
    side, copier = torch.cuda.Stream(), torch.cuda.Stream()
    host = torch.empty(1 << 28, dtype=torch.uint8).pin_memory()
    dev = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    with torch.cuda.stream(copier):
        for _ in range(8):
            dev.copy_(host, non_blocking=True)
    plan = Plan(n, cutoff, sched)
    with torch.cuda.stream(side):
        C = plan(A, B)
    torch.cuda.synchronize()
    plan.close()
    assert np.array_equal(C.cpu().numpy(), oracle.classical(A.cpu().numpy(), B.cpu().numpy()))


def test_host_entry_point_copies_in_and_out():
    n = 384
    A, B = inputs.pair(n, "int8", 51, device="cpu")
    A, B = A.pin_memory(), B.pin_memory()
    C = torch.empty((n, n), dtype=torch.float64).pin_memory()
    plan = Plan(n, 96, "BB")
    plan.run_host(A, B, C)
    torch.cuda.synchronize()
    plan.close()
    assert np.array_equal(C.numpy(), oracle.classical(A.numpy(), B.numpy()))


def test_host_pipeline_keeps_every_result_separate():
    n, calls = 320, 5
    plan = Plan(n, 80, "BB", flags=binding.STRASSEN_FLAG_HOST_PIPELINE)
    As, Bs, Cs = [], [], []
    for k in range(calls):
        A, B = inputs.pair(n, "int8", 700 + 2 * k, device="cpu")
        As.append(A.pin_memory()); Bs.append(B.pin_memory())
        Cs.append(torch.full((n, n), float("nan"), dtype=torch.float64).pin_memory())
    for k in range(calls):                                    # enqueue all calls back to back, no sync in between
        plan.run_host(As[k], Bs[k], Cs[k])
    torch.cuda.synchronize()
    plan.close()
    for k in range(calls):
        assert np.array_equal(Cs[k].numpy(), oracle.classical(As[k].numpy(), Bs[k].numpy())), k


def _graded_pair(n, seed, span=24):
    g = torch.Generator("cuda").manual_seed(seed)
    A = (torch.rand((n, n), generator=g, device="cuda", dtype=torch.float64) * 2 - 1)
    B = (torch.rand((n, n), generator=g, device="cuda", dtype=torch.float64) * 2 - 1)
    ra = torch.randint(-span, span + 1, (n, 1), generator=g, device="cuda")
    cb = torch.randint(-span, span + 1, (1, n), generator=g, device="cuda")
    return torch.ldexp(A, ra), torch.ldexp(B, cb)


def test_outside_scaling_meets_the_row_column_wise_bound():
    """Section 6.1: with D1, D3 the error of C_ij scales with max_k|A_ik| max_k|B_kj|; without scaling only
    the norm-wise bound holds.  Rows of A and columns of B spread over 2^-24 .. 2^24."""
    n, cutoff, sched = 512, 64, "BBB"
    A, B = _graded_pair(n, 11)
    ref = oracle.classical(A.cpu().numpy(), B.cpu().numpy())
    plain = run_plan(n, cutoff, sched, A, B).cpu().numpy()
    scaled = run_plan(n, cutoff, sched, A, B, flags=binding.STRASSEN_FLAG_SCALE_OUTSIDE).cpu().numpy()
    rows = A.abs().amax(dim=1).cpu().numpy()
    cols = B.abs().amax(dim=0).cpu().numpy()
    # 4e-11 = 1e-11 (the norm-wise constant) x 2 x 2: the scaled factors have rows of A and columns of B in [1, 2),
    # and scaling back multiplies entry (i, j) by factors that are at most max_k|A_ik| and max_k|B_kj|
    entry_bound = 4e-11 * n * rows[:, None] * cols[None, :]
    assert np.all(np.abs(scaled - ref) <= entry_bound)
    assert not np.all(np.abs(plain - ref) <= entry_bound)
    assert np.abs(plain - ref).max() <= bound(n, A, B)
    # the oracle's scaled recursion agrees to within the same bound (different summation order in the leaves)
    want, _ = oracle.scaled_strassen_winograd(A.cpu().numpy(), B.cpu().numpy(), cutoff, sched)
    assert np.all(np.abs(scaled - want) <= 2 * entry_bound)


@pytest.mark.parametrize("flags", [8, 16, 24])
def test_scaling_is_exact_on_scaled_integers(flags):
    n, batch = 260, 2
    g = torch.Generator("cuda").manual_seed(5)
    A = torch.ldexp(torch.randint(-8, 9, (batch, n, n), generator=g, device="cuda").double(),
                    torch.randint(-9, 10, (batch, n, 1), generator=g, device="cuda"))
    B = torch.ldexp(torch.randint(-8, 9, (batch, n, n), generator=g, device="cuda").double(),
                    torch.randint(-9, 10, (batch, 1, n), generator=g, device="cuda"))
    A0, B0 = A.clone(), B.clone()
    C = run_plan(n, 65, "BD", A, B, batch=batch, flags=flags)
    assert torch.equal(A, A0) and torch.equal(B, B0)                    # inputs are scaled into copies, never in place
    for b in range(batch):
        assert np.array_equal(C[b].cpu().numpy(), oracle.classical(A[b].cpu().numpy(), B[b].cpu().numpy()))


def test_timing_split_sums_to_about_the_total():
    A, B = inputs.pair(2048, "uniform", 61, device="cuda")
    plan = Plan(2048, 512, "BB")
    plan(A, B)
    torch.cuda.synchronize()
    plan.set_timing(True)
    plan(A, B)
    t = plan.timings_ms()
    plan.close()
    assert t["gemm"] > 0 and t["form"] > 0 and t["recombine"] > 0 and t["peel"] == 0


def test_autotune_returns_a_valid_fastest_candidate():
    from paper_1202_3173_b200 import autotune
    n = 1024
    A, B = inputs.pair(n, "uniform", 91, device="cuda")
    best, log, C = autotune(A, B, workspace_budget_bytes=int(1e9), min_base=128, repetitions=2)
    assert len(log) == 1 + 2 + 4 + 8                       # L = 0..3, every B/D string
    assert {e["levels"] for e in log} == {0, 1, 2, 3}
    assert best["ms"] == min(e["ms"] for e in log) and best["ms"] > 0
    models = [e["model_ms"] for e in log]
    assert models == sorted(models) and models[0] > 0       # tried in the order of the cost model
    assert len(best["schedule"]) == best["levels"] and set(best["schedule"]) <= set("BD")
    # the tuned pair recreates a plan, and C holds that plan's (correct) product
    plan = Plan(n, best["cutoff"], best["schedule"])
    assert plan.levels == best["levels"]
    plan.close()
    ref = oracle.classical(A.cpu().numpy(), B.cpu().numpy())
    assert float(np.abs(C.cpu().numpy() - ref).max()) <= bound(n, A, B)
    # a budget too small for any recursion leaves only the classical product
    best0, log0, _ = autotune(A, B, workspace_budget_bytes=0, min_base=128)
    assert best0["levels"] == 0 and len(log0) == 1


# ---- full-size configurations --------------------------------------------------------------
# n <= 4096: the whole matrix against the classical oracle (a few seconds of host time each); larger n:
# sampled blocks of the definition that contain every recursion boundary, exact on the integer variant,
# plus Freivalds over the whole matrix.

def test_config_n4096_bbb_full_size():
    check_full(4096, 512, "BBB", "int8", 2501)
    r = check_full(4096, 512, "BBB", "uniform", 2001)
    assert r < 1e-2
    check_sampled(4096, 512, "BBB", "int8", 2501)       # the sampled checker itself, where the full answer is known


def test_config_batch32_n2048_bb_full_size():
    if _free_bytes() < 20 * GB:
        pytest.skip("needs 15 GB")
    check_full(2048, 512, "BB", "int8", 5502, batch=32, members=(0, 13, 31))
    check_full(2048, 512, "BB", "uniform", 5002, batch=32, members=(0, 31))
    check_sampled(2048, 512, "BB", "int8", 5502, batch=32, members=tuple(range(1, 31, 4)))


def test_config_n12345_peeling_full_size():
    if _free_bytes() < 20 * GB:
        pytest.skip("needs 12 GB")
    check_sampled(12345, 771, "DBBB", "int8", 5501)
    check_sampled(12345, 771, "DBBB", "uniform", 5001)


def test_config_n16384_dbbbb_full_size():
    if _free_bytes() < 50 * GB:
        pytest.skip("needs 31 GB")
    plan = Plan(16384, 512, "auto", workspace_budget_bytes=int(40 * GB))
    assert plan.schedule == "DBBBB"
    plan.close()
    check_sampled(16384, 512, "DBBBB", "int8", 3501)
    check_sampled(16384, 512, "DBBBB", "uniform", 3001)


def test_config_n47040_full_size():
    n, cutoff = 47040, 2940
    abc = 3 * n * n * 8
    free = _free_bytes()
    if free < 170 * GB:
        pytest.skip("needs about 165 GB of device memory")
    room = int(min(180 * GB, free - 4 * GB) - abc)
    plan = Plan(n, cutoff, "auto", workspace_budget_bytes=room)
    sched = plan.schedule
    plan.close()
    assert sched in ("DBBB", "DDBB")
    check_sampled(n, cutoff, sched, "normal", 4001, samples=48)
    torch.cuda.empty_cache()
    check_sampled(n, cutoff, sched, "int8", 4501, samples=48)

"""Host-side plan logic through the C ABI (no GPU needed): level sizes, schedule strings,
the Limited-Memory rule, workspace arithmetic against the oracle's memory model and the
paper's closed forms, launch lists, and error reporting."""
import itertools

import pytest

import oracle
from paper_1202_3173_b200 import Plan, StrassenError, binding

GB = 1e9


@pytest.mark.parametrize("n,cutoff,L,base", [(512, 256, 1, 256), (4096, 512, 3, 512), (16384, 512, 5, 512),
                                             (47040, 2940, 4, 2940), (12345, 771, 4, 771), (2048, 512, 2, 512),
                                             (300, 512, 0, 300), (1, 1, 0, 1), (2, 1, 1, 1)])
def test_levels_follow_the_cutoff_rule(n, cutoff, L, base):
    p = Plan(n, cutoff, "B" * L)
    assert p.levels == L and p.base_size == base
    assert p.level_sizes == oracle.level_sizes(n, cutoff)
    assert p.base_products == 7 ** L
    p.close()


def test_schedule_errors():
    for bad in ("BB", "BBBB", "BXB", "bbb", ""):
        with pytest.raises(StrassenError) as e:
            Plan(4096, 512, bad)
        assert "schedule" in str(e.value)
    with pytest.raises(StrassenError):
        Plan(0, 512, "")
    with pytest.raises(StrassenError):
        Plan(64, -1, "")
    with pytest.raises(StrassenError):
        Plan(64, 8, "BBB", lda=32)
    with pytest.raises(StrassenError):
        Plan(64, 8, "BBB", batch=-1)


def test_null_arguments_are_reported_not_crashed():
    l = binding.lib()
    assert l.strassen_dgemm(None, None, None, None, None) == -1
    assert b"non-NULL" in l.strassen_last_error()
    assert l.strassen_plan_create_ex(None) is None
    l.strassen_plan_destroy(None)
    assert l.strassen_plan_levels(None) == -1
    assert l.strassen_plan_workspace_bytes(None) == 0


def test_autotune_rejects_bad_requests_without_a_device():
    l = binding.lib()
    assert l.strassen_autotune(None, None, None, 0, None) == -1
    req = binding.strassen_tune_request(64, 1, 0, 0, 0.0, None, None, None, None, 0, None)
    best = binding.strassen_tune_entry()
    import ctypes
    assert l.strassen_autotune(ctypes.byref(req), ctypes.byref(best), None, 0, None) == -1
    assert b"non-NULL" in l.strassen_last_error()


def test_alias_and_alignment_checks_come_before_any_device_work():
    p = Plan(64, 16, "BB")
    l = binding.lib()
    buf = 1 << 20
    n2 = 64 * 64 * 8
    assert l.strassen_dgemm(p.handle, buf, buf + n2, buf + n2 // 2, None) == -4      # C overlaps A and B
    assert l.strassen_dgemm(p.handle, buf, buf + n2, buf + 4, None) == -5          # 4-byte aligned
    import torch
    if not torch.cuda.is_available():   # made-up addresses: only where no kernel can run
        assert l.strassen_dgemm(p.handle, buf, buf, buf + 2 * n2, None) == -6   # A == B is legal; no device
        assert "cuda" in l.strassen_last_error().decode().lower()
    p.close()


@pytest.mark.parametrize("n,cutoff,batch", [(4096, 512, 1), (16384, 512, 1), (2048, 512, 32), (512, 256, 1)])
def test_workspace_model_matches_oracle_and_closed_form(n, cutoff, batch):
    L = len(oracle.level_sizes(n, cutoff)) - 1
    for sched in ("".join(s) for s in itertools.product("BD", repeat=L)):
        for acc in (15, 21):
            assert binding.strassen_schedule_model_bytes(n, cutoff, batch, sched, acc) == \
                8 * oracle.workspace_words(n, cutoff, sched, batch, acc)
        p = Plan(n, cutoff, sched, batch=batch)
        # power-of-two sizes need no padding: the library allocates exactly the 15-matrix figure
        assert p.workspace_bytes == 8 * oracle.workspace_words(n, cutoff, sched, batch, 15)
        assert p.schedule == sched
        p.close()
    all_b = binding.strassen_schedule_model_bytes(n, cutoff, 1, "B" * L, 21)
    assert 3 * n * n * 8 + all_b == pytest.approx(8 * oracle.mem_um_closed_form(n, L), rel=1e-13)


def test_padded_workspace_for_odd_sizes():
    n, cutoff, sched = 12345, 771, "DBBB"
    p = Plan(n, cutoff, sched)
    lo = 8 * oracle.workspace_words(n, cutoff, sched, 1, 15)
    assert lo <= p.workspace_bytes <= lo * 1.01
    assert p.workspace_bytes % 256 == 0
    p.close()


def test_limited_memory_rule():
    # 16384 under 40 GB: DFS at the top, BFS below
    p = Plan(16384, 512, "auto", workspace_budget_bytes=int(40 * GB))
    assert p.schedule == "DBBBB" and p.workspace_bytes <= 40 * GB
    assert round(p.workspace_bytes / GB, 1) == 24.1
    p.close()
    # 47040 with what is left of 180 GB after A, B, C
    room = int(180 * GB - 3 * 47040 ** 2 * 8)
    p = Plan(47040, 2940, None, workspace_budget_bytes=room)
    assert p.schedule == "DBBB" and p.workspace_bytes <= room
    p.close()
    # plenty of room: all BFS; tiny room: all DFS; none: error
    p = Plan(4096, 512, "auto", workspace_budget_bytes=int(10 * GB))
    assert p.schedule == "BBB"
    p.close()
    p = Plan(4096, 512, "auto", workspace_budget_bytes=int(0.14 * GB))
    assert p.schedule == "DDD"
    p.close()
    with pytest.raises(StrassenError):
        Plan(4096, 512, "auto", workspace_budget_bytes=1000)
    # an explicit schedule is checked against an explicit budget
    with pytest.raises(StrassenError):
        Plan(4096, 512, "BBB", workspace_budget_bytes=int(1 * GB))
    # same choice as the oracle's statement of the rule, under the library's own accounting
    for budget_gb in (0.2, 0.5, 1.0, 2.0, 3.0, 5.0):
        p = Plan(4096, 512, "auto", workspace_budget_bytes=int(budget_gb * GB))
        assert p.schedule == oracle.lm_schedule(4096, 512, int(budget_gb * GB) // 8, accounting=15)
        p.close()


def test_auto_without_budget_or_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(StrassenError) as e:
        Plan(4096, 512, "auto")
    assert "CUDA" in str(e.value)


def test_cutoff_zero_lets_the_cost_model_choose():
    GBb = int(1e9)
    # the choices the measurements on a B200 confirmed (autotune finds the same plans)
    for n, batch, budget, sched, base in [(4096, 1, 40, "BBB", 512), (16384, 1, 40, "DBBBB", 512), (12345, 1, 40, "BBB", 1543),
                                          (47040, 1, 125, "DDBBB", 1470), (2048, 32, 40, "BBB", 256), (512, 1, 1, "B", 256),
                                          (1000, 1, 1, "", 1000), (300, 1, 1, "", 300)]:
        p = Plan(n, 0, None, batch=batch, workspace_budget_bytes=budget * GBb)
        assert (p.schedule, p.base_size) == (sched, base), (n, p.schedule, p.base_size)
        assert p.workspace_bytes <= budget * GBb
        p.close()
    # a tighter budget trades BFS steps for DFS steps or a larger base; nothing that does not fit is chosen
    p = Plan(16384, 0, None, workspace_budget_bytes=2 * GBb)
    assert p.workspace_bytes <= 2 * GBb and p.levels >= 1
    p.close()
    p = Plan(4096, 0, None, workspace_budget_bytes=1)       # no room at all: the classical product
    assert p.levels == 0
    p.close()
    # an explicit schedule with cutoff 0 fixes the number of steps by its length
    p = Plan(4096, 0, "BD")
    assert p.level_sizes == [4096, 2048, 1024] and p.schedule == "BD"
    p.close()
    with pytest.raises(StrassenError):
        Plan(8, 0, "BBBB")
    with pytest.raises(StrassenError):
        Plan(4096, -1, "B")


def test_launch_lists():
    # all BFS, one pass per level: one form and one recombine per level, one batched product launch
    single = binding.STRASSEN_FLAG_SINGLE_LEVEL_PASSES
    p = Plan(4096, 512, "BBB", flags=single)
    # (343 x 16 tiles = 37 full rounds of 148 + 12: the leaf owning the leftover runs as a second, small-tile launch)
    assert p.launches_by_kind() == {"form": 3, "gemm": 2, "recombine": 3, "form_one": 0, "accumulate": 0, "peel": 0, "scale": 0, "fused_step": 0, "lincomb": 0}
    assert p.launch_count == 8
    p.close()
    # default: up to three BFS levels share one formation pass and one recombination pass
    p = Plan(4096, 512, "BBB")
    assert p.launches_by_kind() == {"form": 1, "gemm": 2, "recombine": 1, "form_one": 0, "accumulate": 0, "peel": 0, "scale": 0, "fused_step": 0, "lincomb": 0}
    p.close()
    # at most two levels per pass: the two deepest levels pair up
    two = binding.STRASSEN_FLAG_TWO_LEVEL_PASSES
    p = Plan(4096, 512, "BBB", flags=two)
    assert p.launches_by_kind() == {"form": 2, "gemm": 2, "recombine": 2, "form_one": 0, "accumulate": 0, "peel": 0, "scale": 0, "fused_step": 0, "lincomb": 0}
    p.close()
    # DFS on top: 7 x (form_one [not for j = 0, 1], sub-tree, accumulate)
    p = Plan(16384, 512, "DBBBB", flags=single)
    k = p.launches_by_kind()
    # (the recombination pass that ends each sub-problem folds its product into C: no separate fold passes)
    assert k["form_one"] == 5 and k["accumulate"] == 0 and k["gemm"] == 7 and k["form"] == 28 and k["recombine"] == 28
    assert p.base_products == 7 ** 5
    p.close()
    p = Plan(16384, 512, "DBBBB", flags=single | binding.STRASSEN_FLAG_NO_DFS_FOLD)
    assert p.launches_by_kind()["accumulate"] == 7
    p.close()
    # the upper DFS step's sub-problems end in a DFS step (separate fold passes), the lower one's in a recombination
    p = Plan(1024, 128, "DDB", flags=binding.STRASSEN_FLAG_NO_FUSED_STEP)
    k = p.launches_by_kind()
    assert k["accumulate"] == 7 and k["recombine"] == 49
    p.close()
    p = Plan(1024, 128, "DDB")          # ... or, by default at this size, in a fused step: separate fold passes again
    k = p.launches_by_kind()
    assert k["accumulate"] == 7 + 49 and k["fused_step"] == 49 and k["recombine"] == 0
    p.close()
    p = Plan(1026, 256, "DB")           # sub-problems of odd size (513) end in their peeling fix-ups: separate fold passes
    assert p.launches_by_kind()["accumulate"] == 7
    p.close()
    p = Plan(16384, 512, "DBBBB", flags=two)          # four BFS levels below the DFS step: two pairs
    k = p.launches_by_kind()
    assert k["form"] == 14 and k["recombine"] == 14 and k["gemm"] == 7 and p.base_products == 7 ** 5
    p.close()
    p = Plan(16384, 512, "DBBBB")          # ... or one level on its own above a group of three (the bytes are at the bottom)
    k = p.launches_by_kind()
    assert k["form"] == 14 and k["recombine"] == 14 and k["gemm"] == 7
    p.close()
    p = Plan(16384, 256, "BBBBBB")         # six BFS levels: two groups of three
    k = p.launches_by_kind()
    assert k["form"] == 2 and k["recombine"] == 2
    p.close()
    p = Plan(8192, 256, "BBBBB")           # five: a pair above a group of three
    k = p.launches_by_kind()
    assert k["form"] == 2 and k["recombine"] == 2
    p.close()
    # a level of odd size cannot be a lower member of an ordinary group (its fix-ups need the children's products), but it
    # can be the lower member of a pair: sizes 12345, 6172, 3086, 1543 (odd), 771 -> pairs (0,1) and (2,3)
    p = Plan(12345, 771, "BBBB")
    k = p.launches_by_kind()
    assert k["form"] == 2 and k["recombine"] == 2 and k["peel"] == 4      # last column + last row at levels 0 and 3
    p.close()
    p = Plan(12345, 771, "BBBB", flags=two)
    k = p.launches_by_kind()
    assert k["form"] == 2 and k["recombine"] == 2
    p.close()
    p = Plan(12345, 771, "BBBB", flags=single)
    k = p.launches_by_kind()
    assert k["form"] == 4 and k["recombine"] == 4 and k["peel"] == 4
    p.close()
    p = Plan(12345, 771, "DBBB")           # below the DFS step: level 1 alone (it folds its products into C), pair (2,3)
    k = p.launches_by_kind()
    assert k["form"] == 14 and k["recombine"] == 14 and k["accumulate"] == 0 and k["form_one"] == 5
    p.close()
    # a deepest BFS step whose products would leave most SMs idle runs as one fused kernel (no sums, no products in memory)
    p = Plan(512, 256, "B")
    assert p.launches_by_kind() == {"form": 0, "gemm": 0, "recombine": 0, "form_one": 0, "accumulate": 0, "peel": 0,
                                    "scale": 0, "fused_step": 1, "lincomb": 0}
    assert p.base_products == 7
    p.close()
    p = Plan(512, 256, "B", flags=binding.STRASSEN_FLAG_NO_FUSED_STEP)
    k = p.launches_by_kind()
    assert k["fused_step"] == 0 and k["form"] == 1 and k["gemm"] == 1 and k["recombine"] == 1
    p.close()
    p = Plan(4096, 512, "BBB", flags=binding.STRASSEN_FLAG_FUSED_STEP)     # forced: a two-level pass above the fused deepest step
    k = p.launches_by_kind()
    assert k == {"form": 1, "gemm": 0, "recombine": 1, "form_one": 0, "accumulate": 0, "peel": 0, "scale": 0, "fused_step": 1, "lincomb": 0}
    assert p.base_products == 343
    p.close()
    p = Plan(1025, 512, "D", flags=binding.STRASSEN_FLAG_FUSED_STEP)       # only a BFS step can be fused
    assert p.launches_by_kind()["fused_step"] == 0
    p.close()
    p = Plan(1025, 512, "B", flags=binding.STRASSEN_FLAG_FUSED_STEP)       # odd parent: the peeled column and row follow
    k = p.launches_by_kind()
    assert k["fused_step"] == 1 and k["peel"] == 2 and k["gemm"] == 0
    p.close()
    # all DFS: 7^L single products
    p = Plan(64, 8, "DDD")
    assert p.launches_by_kind()["gemm"] == 343 and p.base_products == 343
    p.close()
    # peeling adds two fix-up kernels per odd level (last column, last row; the rank-one term rides in the
    # recombination)
    p = Plan(12345, 771, "BBBB")
    assert p.launches_by_kind()["peel"] == 4
    p.close()
    # zero levels: a single classical product
    p = Plan(300, 512, "")
    assert p.launch_count == 1 and p.workspace_bytes == 0
    p.close()


def test_diagonal_scaling_adds_passes_and_workspace():
    plain = Plan(4096, 512, "BBB")
    out = Plan(4096, 512, "BBB", flags=binding.STRASSEN_FLAG_SCALE_OUTSIDE)
    both = Plan(4096, 512, "BBB", flags=binding.STRASSEN_FLAG_SCALE_OUTSIDE | binding.STRASSEN_FLAG_SCALE_INSIDE)
    assert out.launches_by_kind()["scale"] == 6 and both.launches_by_kind()["scale"] == 8
    extra = out.workspace_bytes - plain.workspace_bytes
    assert 2 * 4096 ** 2 * 8 <= extra <= 2 * 4096 ** 2 * 8 + 3 * 4096 * 4 + 1024      # two scaled copies + exponents
    assert both.workspace_bytes == out.workspace_bytes
    for p in (plain, out, both):
        p.close()


def test_batch_is_extra_live_nodes():
    p = Plan(2048, 512, "BB", batch=32)
    assert p.base_products == 32 * 49
    assert p.launches_by_kind()["gemm"] == 1
    p.close()


def test_python_plan_checks_shapes_before_any_pointer_reaches_the_library():
    """The kernels index their operands by the plan's n and batch only, so a smaller tensor would be read or
    written out of bounds on the device: the Python layer must refuse it (host-only: nothing is launched)."""
    import torch
    from paper_1202_3173_b200 import Plan, matmul
    plan = Plan(64, 16, "BB")
    ok = torch.zeros((64, 64), dtype=torch.float64)
    with pytest.raises(ValueError, match="CUDA"):
        plan(ok, ok)                                            # host tensors on the device entry point
    for bad in (torch.zeros((32, 64), dtype=torch.float64), torch.zeros((64, 64), dtype=torch.float32),
                torch.zeros((64, 128), dtype=torch.float64)[:, ::2], torch.zeros((2, 64, 64), dtype=torch.float64)):
        with pytest.raises(ValueError):
            plan.run_host(bad, ok, ok.clone())
        with pytest.raises(ValueError):
            plan.run_host(ok, ok, bad)
    batched = Plan(64, 16, "BB", batch=3)
    with pytest.raises(ValueError, match="shape"):
        batched.run_host(ok, ok, ok.clone())
    strided = Plan(64, 16, "BB", lda=80)
    with pytest.raises(ValueError, match="raw pointers"):
        strided.run_host(ok, ok, ok.clone())
    with pytest.raises(ValueError, match="square"):
        matmul(torch.zeros((64, 32), dtype=torch.float64), torch.zeros((32, 64), dtype=torch.float64))
    plan.close()
    with pytest.raises(ValueError, match="closed"):
        plan.run_host(ok, ok, ok.clone())
    batched.close(); strided.close()

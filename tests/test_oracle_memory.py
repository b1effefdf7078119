"""Pins for the oracle's memory model against the closed forms of Sections 3.3.1 / 3.4.1
and against the outcomes the workload configurations state."""
import math

import pytest

import oracle

GB = 1e9


@pytest.mark.parametrize("n,k", [(64, 1), (256, 2), (4096, 3), (16384, 5)])
def test_all_bfs_matches_mem_um(n, k):
    cutoff = n >> k
    total = 3 * n * n + oracle.workspace_words(n, cutoff, "B" * k, accounting=21)
    assert math.isclose(total, oracle.mem_um_closed_form(n, k), rel_tol=1e-13)
    # the geometric series itself: 3 n^2 sum_{i=0..k} (7/4)^i
    assert math.isclose(total, 3 * n * n * sum(1.75 ** i for i in range(k + 1)), rel_tol=1e-13)
    # each BFS step needs 7/4 the extra space of the step above it
    per_level = [oracle.workspace_words(n, n >> j, "B" * j) - oracle.workspace_words(n, n >> (j - 1), "B" * (j - 1))
                 for j in range(2, k + 1)]
    first = oracle.workspace_words(n, n >> 1, "B")
    for j, w in enumerate(per_level):
        assert w * 4 ** (j + 1) == first * 7 ** (j + 1)


def test_all_bfs_4096_is_4_096_gb():
    assert oracle.workspace_words(4096, 512, "BBB") * 8 == 7 * 4096 ** 2 * (1.75 ** 3 - 1) * 8
    assert round(oracle.workspace_words(4096, 512, "BBB") * 8 / GB, 2) == 4.10


@pytest.mark.parametrize("n,ell,k", [(1024, 1, 2), (4096, 2, 1), (16384, 1, 4)])
def test_lm_scheme_matches_mem_lm(n, ell, k):
    cutoff = n >> (ell + k)
    total = 3 * n * n + oracle.workspace_words(n, cutoff, "D" * ell + "B" * k)
    m = n >> ell
    want = 3 * n * n * sum(0.25 ** i for i in range(ell)) + oracle.mem_um_closed_form(m, k)
    assert math.isclose(total, want, rel_tol=1e-13)
    # a DFS step adds one sub-problem: a quarter of the space of A, B, C
    assert oracle.workspace_words(n, n // 2, "D") * 4 == 3 * n * n


def test_dfs_first_shrinks_the_footprint():
    n, L = 16384, 5
    cutoff = n >> L
    w = [oracle.workspace_words(n, cutoff, "D" * ell + "B" * (L - ell)) for ell in range(L + 1)]
    assert all(a > b for a, b in zip(w, w[1:]))
    # the BFS part after ell DFS steps works on a matrix 4^ell smaller with ell fewer 7/4 factors
    for ell in range(1, L):
        bfs_part = w[ell] - sum(3 * (n >> i) ** 2 for i in range(1, ell + 1))
        assert bfs_part * 7 ** ell == pytest.approx(oracle.workspace_words(n >> ell, cutoff, "B" * (L - ell)) * 7 ** ell)
        assert bfs_part == oracle.workspace_words(n >> ell, cutoff, "B" * (L - ell))


def test_config_16384_outcome_under_40_gb():
    # the only schedule with four BFS steps that fits 40 GB is DFS at the top, then BFS
    n, cutoff, budget = 16384, 512, 40 * GB / 8
    fits = [s for s in ("".join(p) for p in __import__("itertools").product("BD", repeat=5))
            if s.count("B") == 4 and oracle.workspace_words(n, cutoff, s) <= budget]
    assert fits == ["DBBBB"]
    assert round(oracle.workspace_words(n, cutoff, "DBBBB") * 8 / GB, 1) == 33.1
    assert round(oracle.workspace_words(n, cutoff, "DBBBB", accounting=15) * 8 / GB, 1) == 24.1
    assert oracle.lm_schedule(n, cutoff, budget) == "DBBBB"
    assert oracle.workspace_words(n, cutoff, "BBBBB") * 8 > 180 * GB


def test_config_47040_choices_under_180_gb():
    n, cutoff = 47040, 2940
    room = (180 * GB - 3 * n * n * 8) / 8
    assert oracle.lm_schedule(n, cutoff, room, accounting=21) == "DDBB"
    assert oracle.lm_schedule(n, cutoff, room, accounting=15) == "DBBB"


def test_batch_multiplies_live_nodes():
    assert oracle.workspace_words(2048, 512, "BB", batch=32) == 32 * oracle.workspace_words(2048, 512, "BB")
    assert round(oracle.workspace_words(2048, 512, "BB", batch=32) * 8 / GB, 1) == 15.5


def test_bad_schedules_are_rejected():
    with pytest.raises(ValueError):
        oracle.workspace_words(4096, 512, "BB")
    with pytest.raises(ValueError):
        oracle.workspace_words(4096, 512, "BXB")
    with pytest.raises(ValueError):
        oracle.lm_schedule(4096, 512, 10)

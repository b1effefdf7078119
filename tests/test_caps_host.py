"""One BFS step of CAPS over seven ranks (Algorithm 2 with k = 1): the oracle's restatement pinned against the
definition, the partition and message arithmetic (Sections 3.2, 3.3), and the exchange code of the product
package run as seven gloo processes on CPU with the oracle standing in for the CUDA kernels."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
P = 7


def _ints(n, seed):
    rng = np.random.default_rng(seed)
    return rng.integers(-8, 9, (n, n)).astype(float), rng.integers(-8, 9, (n, n)).astype(float)


@pytest.mark.parametrize("n", [2, 6, 14, 28, 30, 100, 210])
def test_oracle_bfs_step_equals_the_definition(n):
    """All seven processors in numpy: shares -> operand blocks -> regroup by sub-problem -> classical products ->
    regroup by owner -> combine.  On integer data the result must equal the classical product exactly."""
    A, B = _ints(n, n)
    h = n // 2
    blocks = oracle.bfs_row_blocks(h)
    formed = [oracle.bfs_form_shares(oracle.bfs_share(A, r), oracle.bfs_share(B, r)) for r in range(P)]
    Q = []
    for j in range(P):                                  # processor j assembles T_j, S_j from the seven blocks
        Tj = np.vstack([formed[r][0][j] for r in range(P)])
        Sj = np.vstack([formed[r][1][j] for r in range(P)])
        assert Tj.shape == (h, h)
        Q.append(oracle.classical(Tj, Sj))
    shares = [oracle.bfs_combine_shares([Q[j][s:s + rows] for j in range(P)]) for s, rows in blocks]
    assert np.array_equal(oracle.bfs_unshare(shares, n), oracle.classical(A, B))
    # the shares partition the matrix: putting them back gives A again
    assert np.array_equal(oracle.bfs_unshare([oracle.bfs_share(A, r) for r in range(P)], n), A)


def test_partition_and_message_sizes():
    from paper_1202_3173_b200 import caps
    for h in (1, 5, 7, 8, 700, 23520):
        blocks = caps.row_blocks(h)
        assert blocks == oracle.bfs_row_blocks(h)
        assert sum(r for _, r in blocks) == h and [s for s, _ in blocks] == [sum(r for _, r in blocks[:i]) for i in range(P)]
        assert max(r for _, r in blocks) - min(r for _, r in blocks) <= 1            # load balance (Section 3.2)
    # Section 3.3: each of the three all-to-alls moves messages of n^2 / (4 P) words when 7 divides n / 2
    n = 1400
    st = caps.BfsStepRank(n, 3, _NumpyOps(n // 2))
    for peer, tag, t in st.sends_ts() + st.sends_q():
        assert t.numel() == n * n // (4 * P)
    assert len(st.sends_ts()) == 2 * P and len(st.sends_q()) == P and len(st.recvs_ts()) == 2 * P and len(st.recvs_q()) == P
    assert {tag for _, tag, _ in st.sends_ts()} == {caps.TAG_T, caps.TAG_S} and {tag for _, tag, _ in st.sends_q()} == {caps.TAG_Q}
    with pytest.raises(ValueError):
        caps.BfsStepRank(1401, 0, _NumpyOps(700))
    with pytest.raises(ValueError):
        caps.BfsStepRank(1400, 7, _NumpyOps(700))


class _NumpyOps:
    """Stand-in for the CUDA kernels on CPU tensors: the oracle's restatement of the three local steps."""

    def __init__(self, h):
        self.h = h

    def empty(self, *shape):
        import torch
        return torch.full(shape, float("nan"), dtype=torch.float64)

    def form(self, A_share, B_share, T_send, S_send):
        T, S = oracle.bfs_form_shares(A_share.numpy(), B_share.numpy())
        for j in range(P):
            T_send[j].numpy()[...] = T[j]
            S_send[j].numpy()[...] = S[j]

    def multiply(self, T_full, S_full, Q_full):
        Q_full.numpy()[...] = oracle.classical(T_full.numpy(), S_full.numpy())

    def combine(self, Q_recv, C_share):
        C_share.numpy()[...] = oracle.bfs_combine_shares([Q_recv[j].numpy() for j in range(P)])


@pytest.mark.parametrize("n", [28, 30, 6])
def test_in_process_exchange_runs_the_whole_step_on_cpu(n):
    import torch
    from paper_1202_3173_b200 import caps
    A, B = _ints(n, 3 * n)
    ranks = [caps.BfsStepRank(n, r, _NumpyOps(n // 2)) for r in range(P)]
    C = caps.bfs_step_in_process(ranks, torch.from_numpy(A), torch.from_numpy(B))
    assert np.array_equal(C.numpy(), oracle.classical(A, B))


WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import numpy as np, torch, torch.distributed as dist
import oracle
from paper_1202_3173_b200 import caps
from tests.test_caps_host import _NumpyOps, _ints
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, n = dist.get_rank(), int(os.environ["CAPS_N"])
A, B = _ints(n, 11)                                         # every rank draws the same matrices and keeps its share only
state = caps.BfsStepRank(n, rank, _NumpyOps(n // 2))
ex = caps.TorchDistExchange()
A_share, B_share = caps.take_share(torch.from_numpy(A), rank), caps.take_share(torch.from_numpy(B), rank)
C_share = caps.bfs_step(state, A_share, B_share, ex)
want = oracle.bfs_share(oracle.classical(A, B), rank)
print(json.dumps({"rank": rank, "ok": bool(np.array_equal(C_share.numpy(), want)), "log": ex.log}), flush=True)
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


@pytest.mark.parametrize("n", [42, 30])
def test_seven_gloo_ranks_exchange_and_agree_with_the_definition(n):
    port = _free_port()
    procs = []
    for rank in range(P):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(P), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   REPO_ROOT=ROOT, CAPS_N=str(n), OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-600:] for o in outs]
    h = n // 2
    blocks = oracle.bfs_row_blocks(h)
    for out, _ in outs:
        rec = json.loads(out.strip().splitlines()[-1])
        r = rec["rank"]
        assert rec["ok"], "rank %d's share of C differs from the definition" % r
        sends = [(peer, tag, count) for d, peer, tag, count in rec["log"] if d == "send"]
        recvs = [(peer, tag, count) for d, peer, tag, count in rec["log"] if d == "recv"]
        # three all-to-alls: to each of the six other ranks one T block, one S block, one Q block
        for tag in (1, 2):
            assert sorted((p_, c) for p_, t, c in sends if t == tag) == [(j, blocks[r][1] * h) for j in range(P) if j != r]
            assert sorted((p_, c) for p_, t, c in recvs if t == tag) == [(s, blocks[s][1] * h) for s in range(P) if s != r]
        assert sorted((p_, c) for p_, t, c in sends if t == 3) == [(j, blocks[j][1] * h) for j in range(P) if j != r]
        assert sorted((p_, c) for p_, t, c in recvs if t == 3) == [(j, blocks[r][1] * h) for j in range(P) if j != r]
        if h % P == 0:
            assert all(c == n * n // (4 * P) for _, _, c in sends + recvs)       # Section 3.3's message size

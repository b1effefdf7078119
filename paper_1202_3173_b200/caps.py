"""One BFS step of CAPS spread over seven GPUs (Algorithm 2, BFS(A, B, C, k) with k = 1, P = 7).

Each rank owns the same slice of every quadrant of A, B and C (Section 3.2), forms its blocks of the seven
operand pairs locally, the blocks are redistributed so that rank j holds T_j and S_j in full (two all-to-alls
among the seven ranks, messages of n^2 / (4 P) words, Section 3.3), rank j multiplies them with the single-GPU
path (`Plan`), the products are redistributed back (third all-to-all) and every rank combines its blocks of the
seven products into its slice of C.  The arithmetic runs in the library's kernels (strassen_bfs_form_shares,
strassen_dgemm, strassen_bfs_combine_shares); this module only owns buffers and moves blocks:

* `TorchDistExchange` posts the sends and receives of one all-to-all as torch.distributed point-to-point
  operations in one batch (NCCL groups them into one collective over NVLink; gloo serves the CPU tests).  Every
  block lands in the receiver's own memory before any kernel of that rank reads it; no kernel is ever given
  another GPU's memory.
* `InProcessExchange` delivers the same messages between seven rank objects that live in one process, so the
  whole code path can be checked on a single GPU.
* The direct form (`bfs_step_direct`, `DirectPeers`) has no messages at all: the formation kernel of rank r stores
  block r of T_j and S_j straight into rank j's operand matrices, and the combination kernel of rank r loads block r
  of Q_j straight from rank j's product -- plain stores and loads of the library's own kernels through peer
  pointers (over NVLink when the ranks are different GPUs), so the transfer is the kernel's own memory traffic and
  overlaps its arithmetic element by element.  Two barriers per step order writers before readers.  The peer
  pointers come from `InProcessPeers` (seven ranks of one process: the single-GPU check) or `SymmetricPeers`
  (torch symmetric memory on a group of seven GPUs; not exercised on hardware in this repository's tests).

Seven ranks take part; on an eight-GPU node one GPU stays idle (the paper itself leaves up to 6/7 of the
processors idle at P = c 7^k, Section 5.5).
"""
from __future__ import annotations

from . import binding

P = 7
TAG_T, TAG_S, TAG_Q = 1, 2, 3      # one tag per all-to-all of the step


def row_blocks(h: int):
    """[(first row, rows)] of the seven consecutive blocks the h rows of a quadrant are cut into."""
    base, extra = divmod(h, P)
    out, start = [], 0
    for r in range(P):
        rows = base + (1 if r < extra else 0)
        out.append((start, rows))
        start += rows
    return out


def take_share(X, r: int):
    """Rank r's share of an n x n matrix (n even): [X11_r | X12_r] above [X21_r | X22_r], a new (2 rows) x n tensor."""
    import torch
    n = X.shape[-1]
    if X.dim() != 2 or X.shape[0] != n or n % 2:
        raise ValueError("a square matrix of even size is expected, got %s" % (tuple(X.shape),))
    h = n // 2
    start, rows = row_blocks(h)[r]
    return torch.cat((X[start:start + rows], X[h + start:h + start + rows]), dim=0).contiguous()


def put_share(X, share, r: int) -> None:
    """Write rank r's share back into the n x n matrix X."""
    n = X.shape[-1]
    h = n // 2
    start, rows = row_blocks(h)[r]
    X[start:start + rows] = share[:rows]
    X[h + start:h + start + rows] = share[rows:]


class CudaOps:
    """The step's arithmetic through the C ABI (CUDA kernels).  `device` is a torch CUDA device."""

    def __init__(self, h: int, device, cutoff: int = 0, schedule=None, workspace_budget_bytes: int = 0):
        from . import Plan
        self.h, self.device = h, device
        self.plan = Plan(h, cutoff, schedule, workspace_budget_bytes=workspace_budget_bytes)

    def _stream(self):
        import torch
        return torch.cuda.current_stream(self.device).cuda_stream

    def empty(self, *shape):
        import torch
        return torch.empty(shape, dtype=torch.float64, device=self.device)

    def form(self, A_share, B_share, T_send, S_send):
        rows = A_share.shape[0] // 2
        if rows == 0:           # h < 7: this rank owns no rows (it still multiplies its sub-problem)
            return
        binding.strassen_bfs_form_shares(rows, self.h, A_share.data_ptr(), A_share.stride(0), B_share.data_ptr(),
                                         B_share.stride(0), [T_send[j].data_ptr() for j in range(P)],
                                         [S_send[j].data_ptr() for j in range(P)], self.h, self._stream())

    def form_into(self, A_share, B_share, T_addresses, S_addresses):
        """As `form`, the seven blocks of each side going to the given device addresses (rows x h, leading dimension h)."""
        rows = A_share.shape[0] // 2
        if rows == 0:
            return
        binding.strassen_bfs_form_shares(rows, self.h, A_share.data_ptr(), A_share.stride(0), B_share.data_ptr(),
                                         B_share.stride(0), T_addresses, S_addresses, self.h, self._stream())

    def combine_from(self, Q_addresses, C_share):
        """As `combine`, the seven blocks of products read from the given device addresses."""
        rows = C_share.shape[0] // 2
        if rows == 0:
            return
        binding.strassen_bfs_combine_shares(rows, self.h, Q_addresses, self.h, C_share.data_ptr(), C_share.stride(0),
                                            self._stream())

    def multiply(self, T_full, S_full, Q_full):
        self.plan(T_full, S_full, out=Q_full)

    def combine(self, Q_recv, C_share):
        rows = C_share.shape[0] // 2
        if rows == 0:
            return
        binding.strassen_bfs_combine_shares(rows, self.h, [Q_recv[j].data_ptr() for j in range(P)], self.h,
                                            C_share.data_ptr(), C_share.stride(0), self._stream())

    def close(self):
        self.plan.close()


class BfsStepRank:
    """What one of the seven ranks holds and does in the step.  `ops` supplies the arithmetic and the buffers
    (CudaOps on a GPU; the CPU tests of the exchange pass a stand-in of their own)."""

    def __init__(self, n: int, rank: int, ops):
        if n < 2 or n % 2:
            raise ValueError("the distributed step needs an even n >= 2 (its sub-problems may peel odd sizes below)")
        if not 0 <= rank < P:
            raise ValueError("rank must be 0..6")
        self.n, self.h, self.rank, self.ops = n, n // 2, rank, ops
        self.blocks = row_blocks(self.h)
        self.rows = self.blocks[rank][1]
        h, rows = self.h, self.rows
        self.T_send, self.S_send = ops.empty(P, rows, h), ops.empty(P, rows, h)      # block `rank` of T_j, S_j for j = 0..6
        self.T_full, self.S_full, self.Q_full = ops.empty(h, h), ops.empty(h, h), ops.empty(h, h)   # sub-problem `rank` in full
        self.Q_recv = ops.empty(P, rows, h)                                           # block `rank` of Q_j for j = 0..6
        self.C_share = ops.empty(2 * rows, 2 * h)

    # -- the three local steps (Algorithm 2: the lines "locally compute ...") ------------------------------
    def form(self, A_share, B_share):
        if tuple(A_share.shape) != (2 * self.rows, self.n) or tuple(B_share.shape) != (2 * self.rows, self.n):
            raise ValueError("rank %d expects shares of shape %s" % (self.rank, (2 * self.rows, self.n)))
        self.ops.form(A_share, B_share, self.T_send, self.S_send)

    def multiply(self):
        self.ops.multiply(self.T_full, self.S_full, self.Q_full)

    def combine(self):
        self.ops.combine(self.Q_recv, self.C_share)
        return self.C_share

    # -- the messages of the three all-to-alls: (peer, tag, tensor) ------------------------------------------
    def sends_ts(self):
        return ([(j, TAG_T, self.T_send[j]) for j in range(P)] + [(j, TAG_S, self.S_send[j]) for j in range(P)])

    def recvs_ts(self):
        out = []
        for tag, full in ((TAG_T, self.T_full), (TAG_S, self.S_full)):
            out += [(s, tag, full[start:start + rows]) for s, (start, rows) in enumerate(self.blocks)]
        return out

    def sends_q(self):
        return [(r, TAG_Q, self.Q_full[start:start + rows]) for r, (start, rows) in enumerate(self.blocks)]

    def recvs_q(self):
        return [(j, TAG_Q, self.Q_recv[j]) for j in range(P)]


class TorchDistExchange:
    """One all-to-all as a batch of point-to-point operations on a torch.distributed group of seven ranks.
    Blocks a rank keeps for itself are copied in place; empty blocks (h < 7) are not sent."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.rank = dist.get_rank(group)
        if dist.get_world_size(group) != P:
            raise ValueError("the BFS step runs on a group of exactly %d ranks" % P)
        self.log = []       # (direction, peer, tag, elements) of every message posted: what the tests inspect

    def _global(self, r):
        return self.dist.get_global_rank(self.group, r) if self.group is not None else r

    def exchange(self, sends, recvs):
        dist = self.dist
        mine = {tag: t for peer, tag, t in sends if peer == self.rank}
        ops = []
        for peer, tag, t in recvs:
            if peer == self.rank:
                t.copy_(mine[tag])
            elif t.numel():
                ops.append(dist.P2POp(dist.irecv, t, self._global(peer), self.group, tag))
                self.log.append(("recv", peer, tag, t.numel()))
        for peer, tag, t in sends:
            if peer != self.rank and t.numel():
                ops.append(dist.P2POp(dist.isend, t, self._global(peer), self.group, tag))
                self.log.append(("send", peer, tag, t.numel()))
        if ops:
            for req in dist.batch_isend_irecv(ops):
                req.wait()


class InProcessExchange:
    """The same all-to-all between seven BfsStepRank objects of one process: every (peer, tag) message a rank
    sends is copied into the matching receive buffer of that peer."""

    def exchange_all(self, sends_by_rank, recvs_by_rank):
        for dst, recvs in enumerate(recvs_by_rank):
            for src, tag, buf in recvs:
                msg = [t for peer, tg, t in sends_by_rank[src] if peer == dst and tg == tag]
                if len(msg) != 1 or msg[0].shape != buf.shape:
                    raise RuntimeError("rank %d expects one message with tag %d from rank %d" % (dst, tag, src))
                buf.copy_(msg[0])


def bfs_step(rank_state: BfsStepRank, A_share, B_share, exchange: TorchDistExchange):
    """The whole step on one rank of a seven-rank group; returns the rank's share of C."""
    rank_state.form(A_share, B_share)
    exchange.exchange(rank_state.sends_ts(), rank_state.recvs_ts())
    rank_state.multiply()
    exchange.exchange(rank_state.sends_q(), rank_state.recvs_q())
    return rank_state.combine()


def bfs_step_in_process(ranks, A, B):
    """All seven ranks one after another in this process (on one device): C = A @ B assembled from their shares."""
    import torch
    if len(ranks) != P:
        raise ValueError("seven ranks expected")
    ex = InProcessExchange()
    for st in ranks:
        st.form(take_share(A, st.rank), take_share(B, st.rank))
    ex.exchange_all([st.sends_ts() for st in ranks], [st.recvs_ts() for st in ranks])
    for st in ranks:
        st.multiply()
    ex.exchange_all([st.sends_q() for st in ranks], [st.recvs_q() for st in ranks])
    C = torch.empty_like(A)
    for st in ranks:
        put_share(C, st.combine(), st.rank)
    return C


# ---- the direct form: no messages, the kernels store to and load from the peers' matrices -------------------

class InProcessPeers:
    """Peer addresses for seven ranks that live in this process (on one device): the operand and product matrices
    of the BfsStepRank objects themselves.  `barrier` has nothing to wait for: the ranks run one after another on
    one stream."""

    def __init__(self, ranks):
        if len(ranks) != P:
            raise ValueError("seven ranks expected")
        self.T = [st.T_full.data_ptr() for st in ranks]
        self.S = [st.S_full.data_ptr() for st in ranks]
        self.Q = [st.Q_full.data_ptr() for st in ranks]

    def barrier(self):
        pass


class SymmetricPeers:
    """Peer addresses on a group of seven GPUs: each rank's T, S and Q matrices are allocated in torch symmetric
    memory, whose rendezvous maps every rank's buffer into every process.  `adopt` replaces the rank's three
    matrices by views of its own symmetric buffer; `barrier` orders all ranks (and their streams).  This class is
    glue around torch's symmetric-memory module and is not exercised by the tests here (it needs seven GPUs)."""

    def __init__(self, rank_state, group=None):
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm
        h = rank_state.h
        self._dist, self._torch = dist, torch
        buf = symm.empty(3 * h * h, dtype=torch.float64, device=rank_state.T_full.device)
        self._handle = symm.rendezvous(buf, group if group is not None else dist.group.WORLD)
        self._buf = buf
        bases = [int(p) for p in self._handle.buffer_ptrs]
        if len(bases) != P:
            raise ValueError("the BFS step runs on a group of exactly %d ranks" % P)
        words = h * h * 8
        self.T = bases
        self.S = [b + words for b in bases]
        self.Q = [b + 2 * words for b in bases]
        rank_state.T_full = buf[:h * h].view(h, h)
        rank_state.S_full = buf[h * h:2 * h * h].view(h, h)
        rank_state.Q_full = buf[2 * h * h:].view(h, h)

    def barrier(self):
        self._torch.cuda.current_stream().synchronize()      # this rank's stores and loads have completed ...
        self._dist.barrier()                                  # ... and so have every other rank's


def form_direct(st: BfsStepRank, A_share, B_share, peers) -> None:
    """Rank st.rank forms its blocks and stores block `rank` of T_j, S_j into rank j's matrices (rows of rank j's
    h x h operands that belong to this rank)."""
    off = st.blocks[st.rank][0] * st.h * 8
    st.ops.form_into(A_share, B_share, [peers.T[j] + off for j in range(P)], [peers.S[j] + off for j in range(P)])


def combine_direct(st: BfsStepRank, peers):
    """Rank st.rank loads block `rank` of every Q_j from rank j's product and combines them into its share of C."""
    off = st.blocks[st.rank][0] * st.h * 8
    st.ops.combine_from([peers.Q[j] + off for j in range(P)], st.C_share)
    return st.C_share


def bfs_step_direct(st: BfsStepRank, A_share, B_share, peers):
    """The whole step on one rank without messages.  A barrier before the products (all blocks of T_rank, S_rank
    have been stored by their owners) and one before the combination (all products are complete)."""
    form_direct(st, A_share, B_share, peers)
    peers.barrier()
    st.multiply()
    peers.barrier()
    out = combine_direct(st, peers)
    peers.barrier()          # nobody overwrites its operands or product while a peer may still read or write them
    return out


def bfs_step_direct_in_process(ranks, A, B):
    """All seven ranks one after another in this process with the direct form: C = A @ B."""
    import torch
    peers = InProcessPeers(ranks)
    for st in ranks:
        form_direct(st, take_share(A, st.rank), take_share(B, st.rank), peers)
    for st in ranks:
        st.multiply()
    C = torch.empty_like(A)
    for st in ranks:
        put_share(C, combine_direct(st, peers), st.rank)
    return C

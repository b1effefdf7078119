"""The two kernels of the seven-rank BFS step against the oracle's restatement, and the whole step with the seven
ranks run one after another on one GPU through the same code as the distributed path (Algorithm 2 with k = 1)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1202_3173_b200 import StrassenError, binding, caps, inputs

pytestmark = pytest.mark.gpu
P = 7


@pytest.mark.parametrize("rows,h,offset", [(100, 700, 0), (74, 515, 0), (73, 515, 1), (1, 6, 0), (3, 20, 1), (300, 2048, 0)])
def test_share_kernels_give_the_bits_of_the_oracle_restatement(rows, h, offset):
    g = torch.Generator("cuda").manual_seed(rows + h)
    def mat(r, c):      # optionally start 8 bytes off a 16-byte boundary
        buf = torch.rand(r * c + offset, generator=g, device="cuda", dtype=torch.float64) * 2 - 1
        return buf[offset:].view(r, c)
    A, B = mat(2 * rows, 2 * h), mat(2 * rows, 2 * h)
    T, S = [mat(rows, h) for _ in range(P)], [mat(rows, h) for _ in range(P)]
    stream = torch.cuda.current_stream().cuda_stream
    binding.strassen_bfs_form_shares(rows, h, A.data_ptr(), 2 * h, B.data_ptr(), 2 * h, [t.data_ptr() for t in T],
                                     [s.data_ptr() for s in S], h, stream)
    torch.cuda.synchronize()
    Tw, Sw = oracle.bfs_form_shares(A.cpu().numpy(), B.cpu().numpy())
    for j in range(P):
        assert np.array_equal(T[j].cpu().numpy(), Tw[j]) and np.array_equal(S[j].cpu().numpy(), Sw[j]), j
    C = mat(2 * rows, 2 * h)
    C.fill_(float("nan"))
    binding.strassen_bfs_combine_shares(rows, h, [t.data_ptr() for t in T], h, C.data_ptr(), 2 * h, stream)
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy(), oracle.bfs_combine_shares([t.cpu().numpy() for t in T]))


@pytest.mark.parametrize("n,cutoff,sched,dist", [(1400, 350, "B", "int8"), (1400, 175, "BB", "uniform"), (1030, 515, "", "int8"),
                                                 (1030, 129, "DB", "normal"), (12, 3, "B", "int8"), (4, 2, "", "int8")])
def test_seven_ranks_in_turn_on_one_gpu_give_the_product(n, cutoff, sched, dist):
    A, B = inputs.pair(n, dist, 800 + n, device="cuda")
    dev = A.device
    ranks = [caps.BfsStepRank(n, r, caps.CudaOps(n // 2, dev, cutoff, sched)) for r in range(P)]
    C = caps.bfs_step_in_process(ranks, A, B)
    torch.cuda.synchronize()
    for st in ranks:
        st.ops.close()
    ref = oracle.classical(A.cpu().numpy(), B.cpu().numpy())
    if dist == "int8":
        assert np.array_equal(C.cpu().numpy(), ref)
    else:
        err = float(np.abs(C.cpu().numpy() - ref).max())
        lim = 1e-11 * n * float(A.abs().max()) * float(B.abs().max())
        assert err <= 0.02 * lim, (err, lim)
    # the messages of the exchange: n^2 / (4 P) words each when 7 divides n / 2 (Section 3.3)
    if (n // 2) % P == 0:
        assert all(t.numel() == n * n // (4 * P) for _, _, t in ranks[0].sends_ts() + ranks[0].sends_q())


@pytest.mark.parametrize("n,cutoff,sched,dist", [(1400, 350, "B", "uniform"), (1030, 129, "BB", "int8"), (12, 3, "B", "int8")])
def test_direct_form_without_messages_gives_the_same_bits(n, cutoff, sched, dist):
    """The formation kernels store straight into the other ranks' operand matrices and the combination kernels load
    straight from their products (peer addresses; here all seven ranks share one device)."""
    A, B = inputs.pair(n, dist, 820 + n, device="cuda")
    dev = A.device
    def ranks():
        return [caps.BfsStepRank(n, r, caps.CudaOps(n // 2, dev, cutoff, sched)) for r in range(P)]
    a, b = ranks(), ranks()
    C_msg = caps.bfs_step_in_process(a, A, B)
    C_dir = caps.bfs_step_direct_in_process(b, A, B)
    torch.cuda.synchronize()
    assert torch.equal(C_msg, C_dir)
    for st in a + b:
        st.ops.close()
    ref = oracle.classical(A.cpu().numpy(), B.cpu().numpy())
    if dist == "int8":
        assert np.array_equal(C_dir.cpu().numpy(), ref)
    else:
        assert float(np.abs(C_dir.cpu().numpy() - ref).max()) <= 0.02 * 1e-11 * n * float(A.abs().max()) * float(B.abs().max())


def test_share_entry_points_reject_bad_arguments():
    x = torch.zeros(64, dtype=torch.float64, device="cuda")
    seven = [x.data_ptr()] * P
    with pytest.raises(StrassenError) as e:
        binding.strassen_bfs_form_shares(2, 4, x.data_ptr(), 7, x.data_ptr(), 8, seven, seven, 4, 0)     # lda < 2 h
    assert e.value.status == -1
    with pytest.raises(StrassenError) as e:
        binding.strassen_bfs_form_shares(5, 4, x.data_ptr(), 8, x.data_ptr(), 8, seven, seven, 4, 0)     # rows > h
    assert e.value.status == -1
    with pytest.raises(StrassenError) as e:
        binding.strassen_bfs_combine_shares(2, 4, seven[:6] + [0], 4, x.data_ptr(), 8, 0)                # a NULL block
    assert e.value.status == -1
    with pytest.raises(StrassenError) as e:
        binding.strassen_bfs_combine_shares(2, 4, seven, 4, x.data_ptr() + 4, 8, 0)                      # misaligned share
    assert e.value.status == -5
    binding.strassen_bfs_combine_shares(0, 4, seven, 4, x.data_ptr(), 8, 0)                              # an empty block is fine

"""Host-side pieces of bench.py: the N > 1 (replicas) reduction over a world-size-2 gloo group on
CPU, the algorithmic-work arithmetic, and the reference arm's JSON line."""
import json
import os
import socket
import subprocess
import sys

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
ms = bench.reduce_max(3.0 + rank, torch.device("cpu"))          # ranks report 3.0 and 4.0 ms
value = bench.whole_job_value(4096, 1, ms, dist.get_world_size())
dist.barrier()
if rank == 0:
    print(json.dumps({"ms": ms, "value": value}))
dist.destroy_process_group()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_replica_timing_is_the_max_over_ranks_gloo_world_2():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   REPO_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["ms"] == 4.0                                   # the slower rank decides
    assert line["value"] == pytest.approx(2 * 2 * 4096 ** 3 / 4.0e-3 / 1e9)   # both replicas' work / max time


def test_single_process_reduce_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(1.25, "cpu") == 1.25


def test_algorithmic_work_matches_the_oracle_counts():
    sys.path.insert(0, ROOT)
    import bench
    f_base, b_alg = bench.algorithmic_work(4096, 512, 1)
    assert f_base == 343 * 2 * 512 ** 3
    assert b_alg == 8 * 27 * (2048 ** 2 + 7 * 1024 ** 2 + 49 * 512 ** 2)
    # base flops + 15 quadrant additions per node = the flop recurrence of Appendix A (+ n0^2 per leaf:
    # the recurrence counts n0 - 1 additions per entry, the GEMM does n0 fused multiply-adds)
    adds = 15 * b_alg / (27 * 8)
    assert f_base - 343 * 512 ** 2 + adds == oracle.flops_recurrence(4096, 512)
    assert bench.level_sizes(12345, 771) == oracle.level_sizes(12345, 771)


def test_reference_arm_prints_the_contract_line():
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                                   "n512", "--steps", "1", "--warmup", "1"], cwd=ROOT, text=True, timeout=300)
    line = json.loads(out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GFLOP/s" and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"] > 0


def test_gpus_n_without_a_launcher_starts_n_ranks():
    """`python bench.py --gpus 2` started plainly must become two ranks by itself; the stand-in mode runs the same
    launch path and the same max-over-ranks reduction over gloo, with no GPU work."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--check-launch"],
                                  cwd=ROOT, text=True, timeout=300, env=env, stderr=subprocess.DEVNULL)
    line = json.loads([l for l in out.strip().splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["scaling"] == "weak"
    assert line["ms_per_step"] == 4.0                                    # the slower of the ranks' 3 and 4 ms
    assert line["value"] == pytest.approx(2 * 2 * 4096 ** 3 / 4.0e-3 / 1e9)
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.self_launch_command(8, ["--gpus", "8", "--steps", "5"])
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd and cmd[cmd.index("--nproc-per-node") + 1] == "8"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "8", "--steps", "5"]

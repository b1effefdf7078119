#!/usr/bin/env python
"""Benchmark of the Strassen-Winograd hot path on B200: effective FP64 GFLOP/s (2 n^3 / t).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one whole product C = A.B (operand formation, the batched base products,
recombination) on one batch of seeded synthetic input.  With N > 1 every rank (one per GPU)
runs an independent replica of the same product; there is no data-path collective.  Started
without torchrun, `--gpus N` launches its own N ranks.  Rank 0 prints ONE JSON line; besides the
headline workload it carries `per_config`, a short measurement of every configuration the
metric is defined on.  `--impl reference` times the CPU oracle on the host cores instead (a
reported baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# name -> (n, cutoff, schedule, batch, distribution, seed, workspace budget in bytes or 0)
WORKLOADS = {
    "n512": (512, 256, "B", 1, "uniform", 1001, 0),
    "n4096": (4096, 512, "BBB", 1, "uniform", 2001, 0),
    "n16384": (16384, 512, "auto", 1, "uniform", 3001, int(40e9)),
    "n47040": (47040, 2940, "auto", 1, "normal", 4001, -1),   # -1: what 180 GB leaves after A, B, C
    "n12345": (12345, 771, "DBBB", 1, "uniform", 5001, 0),
    "b32n2048": (2048, 512, "BB", 32, "uniform", 5002, 0),
    # the base-product step alone: the 343 leaves of the n=4096 tree as a batch with zero levels
    "gemm512x343": (512, 512, "", 343, "uniform", 6001, 0),
    "gemm2940x2": (2940, 2940, "", 2, "uniform", 6002, 0),
    "gemm771x49": (771, 771, "", 49, "uniform", 6003, 0),
}
DEFAULT_WORKLOAD = "n4096"   # the configuration the headline metric is quoted on
# the configurations of the metric, in the order they are reported in `per_config`, with their timed steps
PER_CONFIG = (("n512", 200), ("n4096", 20), ("b32n2048", 10), ("n12345", 5), ("n16384", 5), ("n47040", 2))
METRIC = "effective FP64 GFLOP/s (2n^3/t)"
UNIT = "GFLOP/s"

# DRAM bytes (read + write) of the dominant kernel's launches per step, from ncu captures of that workload
# (profiles/launch_list_bench_n4096.md: 1.446 GB read + 0.682 GB written; profiles/gemm_f64_kernel_343x512.md);
# None where no capture of that exact launch exists.
GEMM_DRAM_TRAFFIC_BYTES = {"n4096": 2.13e9, "gemm512x343": 2.125e9}

# FP64 arithmetic peak from unit counts and clocks: 148 SMs x 64 FP64 FMA lanes x 2 flop x 1.965 GHz
FP64_PEAK_NOMINAL_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12
HBM_NOMINAL_GBS = 8000.0     # the figure the metric's definition names; the measured copy rate is the denominator used


def describe(name):
    n, cutoff, sched, batch, dist, seed, _ = WORKLOADS[name]
    return ("%s: %sn=%d FP64 C=A.B, Strassen-Winograd to base <= %d, schedule %s, %s entries, seed %d"
            % (name, "%d x " % batch if batch > 1 else "", n, cutoff, sched, dist, seed))


def level_sizes(n, cutoff):
    m = [n]
    while m[-1] > cutoff:
        m.append(m[-1] // 2)
    return m


def algorithmic_work(n, cutoff, batch):
    """(base-product flops, sum/recombine bytes) of one product with one streaming pass per level: 7^L
    products of 2 m_L^3 flops; per node per level 16 h^2 words to form the sums + 11 h^2 to recombine."""
    m = level_sizes(n, cutoff)
    L = len(m) - 1
    f_base = batch * 7 ** L * 2.0 * m[-1] ** 3
    b_alg = batch * 8.0 * sum(7 ** i * 27 * m[i + 1] ** 2 for i in range(L))
    return f_base, b_alg


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock, power and throttle reasons while the timed region runs (NVML from a thread,
    every few milliseconds; read-only queries)."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, index):
        self.rows, self.stop_flag, self.thread, self.err = [], False, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:                                   # the CUDA ordinal need not be the NVML index: go by PCI address
                import torch
                pr = torch.cuda.get_device_properties(index)
                self.h = pynvml.nvmlDeviceGetHandleByPciBusId(
                    ("%08x:%02x:%02x.0" % (pr.pci_domain_id, pr.pci_bus_id, pr.pci_device_id)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
        except Exception as exc:
            self.err = str(exc)

    def _poll(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                try:
                    rs = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    rs = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.rows.append((time.time(), float(sm), pw, int(rs)))
            except Exception as exc:
                self.err = str(exc)
                return
            time.sleep(0.004)

    def stop(self, t0, t1):
        self.stop_flag = True
        if self.thread:
            self.thread.join(timeout=2)
        rows = [r for r in self.rows if t0 <= r[0] <= t1] or self.rows
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples: %s" % self.err]}
        bits = 0
        for r in rows:
            bits |= r[3]
        return {"sm_mhz": statistics.median(r[1] for r in rows), "sm_max_mhz": self.max_sm,
                "reasons": [name for name, bit in self.REASONS if bits & bit],
                "power_w_max": max(r[2] for r in rows), "samples": len(rows)}


def reduce_max(value: float, device) -> float:
    """Max over ranks of a per-rank time (the only cross-rank exchange: a scalar)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(n, batch, ms_per_step, world):
    """Effective GFLOP/s of all replicas together: world x 2 n^3 x batch / t."""
    return world * 2.0 * n ** 3 * batch / (ms_per_step * 1e-3) / 1e9


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def self_launch_command(gpus, argv):
    """The command that runs this script as `gpus` ranks on this node (used when --gpus N > 1 is given
    without a launcher): torch.distributed.run with a rendezvous on 127.0.0.1."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)


def time_oracle_slab(n, A_host, B_host, target_seconds=12.0):
    """Time the classical oracle on a slab of rows of the same product; the slab is grown until it
    costs about target_seconds.  Returns (GFLOP/s, rows, seconds, the slab of C)."""
    import oracle
    rows, t = min(n, 32), 0.0
    while True:
        t0 = time.perf_counter()
        slab = oracle.classical(A_host[:rows], B_host)
        t = time.perf_counter() - t0
        if rows >= n or t >= target_seconds / 3:
            break
        rows = min(n, max(rows * 2, int(rows * 0.6 * target_seconds / max(t, 1e-3))))
    return 2.0 * rows * n * n / t / 1e9, rows, t, slab


def sample_indices(sizes, extra, seed):
    """Row / column indices that touch every recursion boundary (first and last row of each quadrant at every
    level, the peeled last row) plus seeded random ones."""
    import numpy as np
    n = sizes[0]
    idx, starts = {0, n - 1}, [0]
    for m, h in zip(sizes[:-1], sizes[1:]):
        new = []
        for s in starts[:32]:
            for q in (0, 1):
                o = s + q * h
                new.append(o)
                idx.update(i for i in (o, o + h - 1, o + h, s + m - 1) if 0 <= i < n)
        starts = new
    rng = np.random.default_rng(seed)
    idx.update(int(i) for i in rng.integers(0, n, extra))
    return np.array(sorted(idx), dtype=np.int64)


def oracle_block_check(A, B, C, sizes, seed, exact):
    """Part of the CPU-oracle leg: the block C[R, S] of the definition, computed by the classical oracle from
    the sampled rows of A and columns of B, against the same block of the device result."""
    import numpy as np
    import torch
    import oracle
    R, S = sample_indices(sizes, 64, seed + 17), sample_indices(sizes, 64, seed + 29)
    Rt, St = torch.from_numpy(R).to(A.device), torch.from_numpy(S).to(A.device)
    rows = A.index_select(0, Rt).cpu().numpy()
    cols = B.index_select(1, St).cpu().numpy()
    got = C.index_select(0, Rt).index_select(1, St).cpu().numpy()
    ref = oracle.classical(rows, cols)
    if exact:
        return bool(np.array_equal(got, ref))
    return float(np.abs(got - ref).max())


def absmax(X):
    import torch
    lo, hi = torch.aminmax(X)
    return max(abs(float(lo)), abs(float(hi)))


def timed_steps(fn, steps, stream, barrier=None, stride=1):
    """K steps in one timed region with a CUDA event after every `stride` steps (no host synchronisation inside):
    returns the per-step times of the intervals in ms, the mean over the whole region, and its wall-clock bracket.
    A stride above 1 is for steps of a few microseconds, where an event after each would be a good part of it."""
    import torch
    marks = list(range(stride, steps, stride)) + [steps]
    events = [torch.cuda.Event(enable_timing=True) for _ in range(len(marks) + 1)]
    w0 = time.time()
    events[0].record(stream)
    k = 0
    for i in range(steps):
        fn()
        if i + 1 == marks[k]:
            k += 1
            events[k].record(stream)
    if barrier:
        barrier()
    else:
        torch.cuda.synchronize()
    w1 = time.time()
    spans = [marks[0]] + [marks[i] - marks[i - 1] for i in range(1, len(marks))]
    per_step = [events[i].elapsed_time(events[i + 1]) / spans[i] for i in range(len(marks))]
    return per_step, events[0].elapsed_time(events[-1]) / steps, w0, w1


def measure(name, steps, warmup, rank, world, dev, sampler_factory=None, want_cublas=True, want_oracle=True):
    """One configuration on this rank's GPU: the timed region (K steps, one CUDA event between steps, barrier and
    synchronize on both sides), a second pass with per-kernel-family events, cuBLAS DGEMM on the same buffers,
    and -- in the CPU-oracle leg -- a sampled block of the definition on the float and the integer variant."""
    import torch
    import torch.distributed as dist
    from paper_1202_3173_b200 import Plan, inputs

    n, cutoff, sched, batch, dist_name, seed, budget = WORKLOADS[name]
    if budget < 0:
        budget = int(min(180e9, torch.cuda.mem_get_info()[0] - 4e9) - 3 * n * n * 8)
    A, B = inputs.pair(n, dist_name, seed + 1000 * rank, device=dev, batch=None if batch == 1 else batch)
    C = torch.empty_like(A)
    plan = Plan(n, cutoff, sched, batch=batch, workspace_budget_bytes=budget)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        plan(A, B, out=C)
    barrier()
    # steps of a few microseconds: one event per ~20 steps instead of one per step
    t0 = time.perf_counter()
    for _ in range(3):
        plan(A, B, out=C)
    torch.cuda.synchronize()
    stride = 1 if (time.perf_counter() - t0) / 3 > 200e-6 else max(1, min(20, steps // 10))
    sampler = sampler_factory() if sampler_factory else None
    per_step, ms_mean_local, w0, w1 = timed_steps(lambda: plan(A, B, out=C), steps, stream, barrier, stride)
    clocks = sampler.stop(w0, w1) if sampler else None
    ms_median_local = statistics.median(per_step)
    ms = reduce_max(ms_median_local, dev)
    ms_mean = reduce_max(ms_mean_local, dev)

    # per-kernel-family split: a separate, shorter pass with two events around every launch
    split_steps = max(1, min(steps, 5))
    plan.set_timing(True)
    for _ in range(split_steps):
        plan(A, B, out=C)
    kinds = {k: v / split_steps for k, v in plan.timings_ms().items()}
    plan.set_timing(False)

    sizes = plan.level_sizes
    f_base, b_27 = algorithmic_work(n, sizes[-1], batch)
    pass_bytes = plan.pass_bytes
    hbm_gbs, hbm_src = hbm_peak()
    product_kind = "fused_step" if kinds.get("fused_step", 0.0) > 0 else "gemm"
    product_ms = kinds[product_kind]
    add_ms = sum(v for k, v in kinds.items() if k not in ("gemm", "fused_step", "scale"))
    out = {
        "workload": name, "n": n, "batch": batch, "schedule": plan.schedule, "levels": sizes,
        "workspace_bytes": plan.workspace_bytes, "steps": steps, "steps_per_event": stride, "launches_per_step": plan.launch_count,
        "launches_by_kind": {k: v for k, v in plan.launches_by_kind().items() if v},
        "ms_per_step": ms, "ms_per_step_mean": ms_mean, "ms_per_step_min": min(per_step), "ms_per_step_max": max(per_step),
        "effective_gflops": whole_job_value(n, batch, ms, 1),
        "actual_gflops": (f_base + 15 * b_27 / (27 * 8)) / (ms * 1e-3) / 1e9,
        "kernel_ms_per_step": {k: round(v, 6) for k, v in kinds.items() if v},
        "product_kernel": product_kind,
        "product_tflops": f_base / (product_ms * 1e-3) / 1e12 if product_ms > 0 else None,
        "product_frac_of_fp64_peak": f_base / (product_ms * 1e-3) / 1e12 / FP64_PEAK_NOMINAL_TFLOPS if product_ms > 0 else None,
        "add_bytes_scheduled": pass_bytes, "add_bytes_27h2": b_27,
        "add_gbs": pass_bytes / (add_ms * 1e-3) / 1e9 if add_ms > 0 else None,
        "add_frac_of_measured_hbm": pass_bytes / (add_ms * 1e-3) / 1e9 / hbm_gbs if add_ms > 0 else None,
        "add_frac_of_nominal_8000": pass_bytes / (add_ms * 1e-3) / 1e9 / HBM_NOMINAL_GBS if add_ms > 0 else None,
        "l2": "inputs larger than L2 (A+B+C %.0f MB + workspace): no flush" % (3 * batch * n * n * 8 / 1e6)
              if 3 * batch * n * n * 8 > 126e6 else
              "L2-resident by nature (A+B+C %.1f MB): launch-bound, no flush between steps" % (3 * batch * n * n * 8 / 1e6),
    }
    # roofline of the whole product: base products at the FP64 peak + the scheduled passes at the HBM rate; and the
    # floor no fusion can beat (products at peak + A and B read, C written once)
    t_roof = (f_base / (FP64_PEAK_NOMINAL_TFLOPS * 1e12) + pass_bytes / (hbm_gbs * 1e9)) * 1e3
    t_floor = (f_base / (FP64_PEAK_NOMINAL_TFLOPS * 1e12) + 3.0 * batch * n * n * 8 / (hbm_gbs * 1e9)) * 1e3
    t_27 = (f_base / (FP64_PEAK_NOMINAL_TFLOPS * 1e12) + b_27 / (hbm_gbs * 1e9)) * 1e3
    out["path_roofline"] = {"t_roof_ms": t_roof, "frac": t_roof / ms_median_local,
                            "bytes": "the passes as scheduled (strassen_plan_pass_bytes): multi-level passes, DFS surcharge and peeling included",
                            "floor_ms": t_floor, "frac_of_floor": t_floor / ms_median_local,
                            "floor": "base products at the FP64 peak + 3 n^2 words over HBM: what no fusion of the passes can beat",
                            "t_one_pass_per_level_ms": t_27, "ratio_to_one_pass_per_level": t_27 / ms_median_local,
                            "one_pass_per_level": "27 h^2 words per node per level; NOT a lower bound: multi-level passes move less, "
                                                  "so this ratio may exceed 1",
                            "base_flops": f_base, "hbm_gbs": hbm_gbs, "hbm_source": hbm_src}

    if want_cublas:
        Cc = C if 3 * batch * n * n * 8 > 40e9 else torch.empty_like(A)      # no room for a fourth matrix at the largest size
        reps = max(2, min(steps, 200 if n <= 512 else 20 if n <= 4096 else 5))
        try:
            for _ in range(3 if n <= 16384 else 1):
                torch.matmul(A, B, out=Cc)
            torch.cuda.synchronize()
            c_steps, c_mean, _, _ = timed_steps(lambda: torch.matmul(A, B, out=Cc), reps, stream, None, stride)     # same protocol as ours
            cms = statistics.median(c_steps)
            out["cublas_dgemm"] = {"ms": cms, "ms_mean": c_mean, "steps": reps, "gflops": 2.0 * n ** 3 * batch / (cms * 1e-3) / 1e9}
            out["vs_cublas"] = cms / ms_median_local
        except Exception as exc:
            out["cublas_dgemm"] = {"error": str(exc)[:200]}
        if Cc is C:
            plan(A, B, out=C)               # C holds our product again
            torch.cuda.synchronize()
        del Cc

    if want_oracle and rank == 0:
        # CPU-oracle leg, parity part: a block of the definition that contains every recursion boundary
        try:
            a0, b0, c0 = (A, B, C) if batch == 1 else (A[0], B[0], C[0])
            lim = 1e-11 * n * absmax(A) * absmax(B)
            err = oracle_block_check(a0, b0, c0, sizes, seed, exact=False)
            out["max_err"], out["bound"], out["err_over_bound"] = err, lim, err / lim
            del A, B, a0, b0, c0
            A, B = inputs.pair(n, "int8", seed + 500, device=dev, batch=None if batch == 1 else batch)
            plan(A, B, out=C)
            torch.cuda.synchronize()
            a0, b0, c0 = (A, B, C) if batch == 1 else (A[0], B[0], C[0])
            out["int_equal"] = oracle_block_check(a0, b0, c0, sizes, seed + 500, exact=True)
            del a0, b0, c0
        except Exception as exc:
            out["oracle_check_error"] = str(exc)[:200]
    return out, clocks, plan, (A, B, C)


def run_bfs_step(args, rank, world, dev):
    """One product over seven GPUs (strong scaling): every rank draws the same seeded A and B, keeps its share,
    and the K timed steps are K whole distributed products; time = max over ranks."""
    import torch
    import torch.distributed as dist
    from paper_1202_3173_b200 import caps, inputs
    if world != caps.P:
        raise SystemExit("--bfs-step needs exactly %d ranks (--gpus %d)" % (caps.P, caps.P))
    n, cutoff, sched, batch, dist_name, seed, _ = WORKLOADS[args.workload]
    if batch != 1 or n % 2:
        raise SystemExit("--bfs-step takes a single product of even size")
    A, B = inputs.pair(n, dist_name, seed, device=dev)
    A_share, B_share = caps.take_share(A, rank), caps.take_share(B, rank)
    del A, B
    # the workload's top level is the distributed step; the levels below it run on each GPU
    ops = caps.CudaOps(n // 2, dev, cutoff, None if sched == "auto" else sched[1:])
    state = caps.BfsStepRank(n, rank, ops)
    if args.bfs_direct:
        peers = caps.SymmetricPeers(state)
        step = lambda: caps.bfs_step_direct(state, A_share, B_share, peers)
    else:
        ex = caps.TorchDistExchange()
        step = lambda: caps.bfs_step(state, A_share, B_share, ex)
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        step()
    dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    dist.barrier()
    torch.cuda.synchronize()
    ms = reduce_max(e0.elapsed_time(e1) / args.steps, dev)
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": 2.0 * n ** 3 / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(args.workload), "parallelism": "one BFS step over 7 GPUs (Algorithm 2, k = 1), "
                                      + ("direct peer stores and loads" if args.bfs_direct else "three NCCL all-to-alls"),
                       "sub_problem": {"n": n // 2, "schedule": ops.plan.schedule, "levels": ops.plan.level_sizes},
                       "message_words": n * n // (4 * caps.P), "all_to_alls_per_step": 3},
            "gpu_launches": args.steps * (ops.plan.launch_count + 2)}), flush=True)
    ops.close()


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle as it stands, on the host cores, rank 0 only."""
    if rank != 0:
        return
    import oracle
    from paper_1202_3173_b200 import inputs
    n, cutoff, sched, batch, dist_name, seed, _ = WORKLOADS[args.workload]
    A, B = inputs.pair(n, dist_name, seed, device="cpu")
    A, B = A.numpy(), B.numpy()
    rows = min(n, max(16, int(2.0e9 / (2.0 * n * n)) * 8))     # about 16 GFLOP per step
    for _ in range(args.warmup):
        oracle.classical(A[: max(8, rows // 8)], B)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.classical(A[:rows], B)
    dt = (time.perf_counter() - t0) / args.steps
    gflops = 2.0 * rows * n * n / dt / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": gflops, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(args.workload)},
            "cpu_baseline": {"value": gflops, "unit": UNIT, "cores": oracle.cores(), "kind": "oracle",
                             "sample": "classical oracle on the first %d of %d rows of C per step "
                                       "(classical flops = effective flops, so the rate stands for the full product)" % (rows, n)},
            "e2e": {"value": gflops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the timed CPU oracle leg (and its parity samples)")
    ap.add_argument("--no-cublas", action="store_true", help="skip the cuBLAS DGEMM comparator")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-probes", action="store_true", help="skip the FP64 rate probes")
    ap.add_argument("--no-autotune", action="store_true", help="skip the measured choice of steps and interleaving")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short measurement of the other configurations")
    ap.add_argument("--graph", action="store_true", help="also time the plan replayed as one CUDA graph")
    ap.add_argument("--bfs-step", action="store_true",
                    help="with --gpus 7: time ONE product spread over the seven GPUs as a BFS step of CAPS (Algorithm 2, "
                         "k = 1: local sums, three all-to-alls over NCCL, the n/2 sub-products on the single-GPU path, local "
                         "combine) instead of seven independent replicas")
    ap.add_argument("--bfs-direct", action="store_true",
                    help="with --bfs-step: no messages -- the kernels store to and load from the peers' matrices through "
                         "symmetric-memory peer pointers")
    ap.add_argument("--check-launch", action="store_true",
                    help="no GPU work: every rank joins a gloo group and exchanges a stand-in time through the same reduction "
                         "(checks the launcher plumbing of --gpus N on a machine without GPUs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher around us: build first (no rank may find a half-linked library), then become N ranks
        if args.impl == "ours" and not args.check_launch:
            from paper_1202_3173_b200 import build as _build
            _build.ensure_built()
        cmd = self_launch_command(args.gpus, sys.argv[1:])
        os.execvp(cmd[0], cmd)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.check_launch:
        import torch
        import torch.distributed as dist
        if world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group("gloo")
        ms = reduce_max(3.0 + rank, torch.device("cpu"))       # stand-in per-rank times 3, 4, ... ms
        if rank == 0:
            print(json.dumps({"check_launch": True, "n_gpus": world, "ms_per_step": ms, "scaling": "weak",
                              "value": whole_job_value(*WORKLOADS[args.workload][:1], WORKLOADS[args.workload][3], ms, world)}),
                  flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("NCCL_DEBUG", "INFO")          # the communicator log shows every rank that joined
        dist.init_process_group("nccl", device_id=dev)
    from paper_1202_3173_b200 import build as _build
    if local_rank == 0:
        _build.ensure_built()                                 # one rank (re)builds; the others wait, then load
    if world > 1:
        dist.barrier()
    from paper_1202_3173_b200 import Plan, binding

    if args.bfs_step:
        run_bfs_step(args, rank, world, dev)
        if world > 1:
            dist.destroy_process_group()
        return

    n, cutoff, sched, batch, dist_name, seed, _ = WORKLOADS[args.workload]
    head, clocks, plan, (A, B, C) = measure(args.workload, args.steps, args.warmup, rank, world, dev,
                                            sampler_factory=(lambda: ClockSampler(local_rank)) if rank == 0 else None,
                                            want_cublas=rank == 0 and not args.no_cublas,
                                            want_oracle=rank == 0 and not args.no_cpu_baseline)
    stream = torch.cuda.current_stream()
    ms = head["ms_per_step"]
    sched_resolved = plan.schedule

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    del A, B
    from paper_1202_3173_b200 import inputs
    A, B = inputs.pair(n, dist_name, seed + 1000 * rank, device=dev, batch=None if batch == 1 else batch)
    hA = hB = None
    if not args.no_e2e or (rank == 0 and not args.no_cpu_baseline):
        hA, hB = A.cpu().pin_memory(), B.cpu().pin_memory()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def run_e2e():
        """Host buffers, copies inside the timed region.  Runs last: the device copies of A, B, C are freed
        first so that the library's staging buffers fit beside the workspace at the largest size."""
        nonlocal A, B, C
        if args.no_e2e:
            return [None, None], None
        try:
            del A, B, C
            torch.cuda.empty_cache()
            hC = torch.empty_like(hA).pin_memory()
            e2e_steps = max(3, min(args.steps, 10))
            out = []
            for flags in (0, binding.STRASSEN_FLAG_HOST_PIPELINE):     # strictly in stream order, then pipelined
                hplan = plan if flags == 0 else Plan(n, cutoff, sched_resolved, batch=batch, flags=flags)
                if flags and 3 * batch * n * n * 8 * 2 > 60e9:
                    out.append(None)                                  # two sets of device copies would not fit
                    continue
                for _ in range(2):
                    hplan.run_host(hA, hB, hC)
                barrier()
                ev0.record(stream)
                for _ in range(e2e_steps):
                    hplan.run_host(hA, hB, hC)
                ev1.record(stream)
                barrier()
                out.append(reduce_max(ev0.elapsed_time(ev1) / e2e_steps, dev))
                if flags:
                    hplan.close()
            return out, None
        except Exception as exc:           # out of device or pinned memory at the largest sizes
            return [None, None], str(exc)

    if rank != 0:
        run_e2e()
        plan.close()
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- rank 0: probes, tuner, CPU oracle, the other configurations, report --------------------
    f_base, _ = algorithmic_work(n, head["levels"][-1], batch)
    probes = {}
    for kind, pname in enumerate(("dfma", "dmma_m8n8k4", "dmma_m16n8k4", "dmma_m16n8k8", "dmma_m16n8k16")):
        if args.no_probes:
            break
        try:
            probes[pname] = round(binding.strassen_probe_fp64(kind, 20000, stream.cuda_stream), 2)
        except Exception as exc:   # a probe is context, never fatal
            probes[pname] = str(exc)
    measured = [v for v in probes.values() if isinstance(v, float)]
    fp64_peak, peak_source = ((max(measured), "strassen_probe_fp64 in this run: register-resident mma.sync f64 loop on every SM")
                              if measured else
                              (FP64_PEAK_NOMINAL_TFLOPS, "148 SMs x 64 FP64 FMA/clk x 2 x 1.965 GHz (unit counts and max clock)"))

    tuned = None
    if not args.no_autotune:
        # the paper tunes every point to the best interleaving and number of Strassen steps (Section 5.4);
        # reported beside the prescribed configuration, never instead of it
        try:
            if batch * n * n * 8 * 3 < 20e9:
                ws_budget = max(plan.workspace_bytes, int(min(40e9, torch.cuda.mem_get_info()[0] - 2e9)))
                ws = torch.empty(ws_budget, dtype=torch.uint8, device=dev)
                Ct = torch.empty_like(A)
            else:       # no room for a second workspace and result: the plan's own workspace and C serve the search
                ws_budget, ws, Ct = plan.workspace_bytes, plan.workspace, C
            best, log = binding.strassen_autotune(n, A.data_ptr(), B.data_ptr(), Ct.data_ptr(),
                                                  ws.data_ptr() if ws is not None else 0, ws_budget,
                                                  stream.cuda_stream, batch, 256, 3 if n < 20000 else 1, 60.0)
            tuned = dict(best, candidates=len(log), gflops=2.0 * n ** 3 * batch / (best["ms"] * 1e-3) / 1e9,
                         workspace_budget_bytes=ws_budget)
            del ws, Ct
        except Exception as exc:
            tuned = {"error": str(exc)}

    graph_ms = None
    if args.graph:
        gplan = Plan(n, cutoff, plan.schedule, batch=batch, flags=binding.STRASSEN_FLAG_CUDA_GRAPH)
        Cg = torch.empty_like(A)
        for _ in range(3):
            gplan(A, B, out=Cg)
        torch.cuda.synchronize()
        ev0.record(stream)
        for _ in range(args.steps):
            gplan(A, B, out=Cg)
        ev1.record(stream)
        torch.cuda.synchronize()
        graph_ms = ev0.elapsed_time(ev1) / args.steps
        gplan.close()
        del Cg

    cpu = None
    if not args.no_cpu_baseline:
        import numpy as np
        import oracle
        a_h = (hA if batch == 1 else hA[0]).numpy()
        b_h = (hB if batch == 1 else hB[0]).numpy()
        g, rows, secs, slab = time_oracle_slab(n, a_h, b_h)
        plan(A, B, out=C)
        torch.cuda.synchronize()
        ours = (C if batch == 1 else C[0])[:rows].cpu().numpy()
        slab_err = float(np.abs(ours - slab).max())
        cpu = {"value": g, "unit": UNIT, "cores": oracle.cores(), "kind": "oracle",
               "sample": "classical oracle (the definition, Oracle A) on the first %d of %d rows of one product (%.1f s); "
                         "classical flops equal effective flops, so the rate stands for the whole product" % (rows, n, secs),
               "max_err_on_sample": slab_err, "bound": head.get("bound")}
        # Oracle B, the CPU Strassen-Winograd with the same cutoff, timed once on a leading block it finishes in seconds
        try:
            nb = n if n <= 4096 else 4096
            t0 = time.perf_counter()
            cb, counters = oracle.strassen_winograd(np.ascontiguousarray(a_h[:nb, :nb]), np.ascontiguousarray(b_h[:nb, :nb]),
                                                    head["levels"][-1])
            tb = time.perf_counter() - t0
            cpu["strassen_winograd_oracle"] = {
                "value": 2.0 * nb ** 3 / tb / 1e9, "unit": "effective " + UNIT, "seconds": tb, "n": nb,
                "cutoff": head["levels"][-1], "base_products": int(counters["base_calls"]),
                "sample": "Oracle B on the leading %d x %d blocks of A and B, once" % (nb, nb)}
        except Exception as exc:
            cpu["strassen_winograd_oracle"] = {"error": str(exc)[:200]}

    launch_count = plan.launch_count
    (e2e_ms, e2e_pipe_ms), e2e_error = run_e2e()
    plan.close()
    del plan
    torch.cuda.empty_cache()

    per_config = []
    if not args.no_per_config and args.workload == DEFAULT_WORKLOAD and world == 1:
        for cname, csteps in PER_CONFIG:
            if cname == args.workload:
                per_config.append(dict(head, note="the headline run above"))
                continue
            cn, _, _, cb, _, _, cbudget = WORKLOADS[cname]
            need = 3 * cb * cn * cn * 8 + (110e9 if cbudget < 0 else 45e9 if cbudget else 16e9)
            torch.cuda.empty_cache()
            if torch.cuda.mem_get_info()[0] < need:
                per_config.append({"workload": cname, "skipped": "needs about %.0f GB of free device memory" % (need / 1e9)})
                continue
            try:
                res, _, cplan, bufs = measure(cname, csteps, 3, 0, 1, dev, want_cublas=not args.no_cublas,
                                              want_oracle=not args.no_cpu_baseline)
                cplan.close()
                del cplan, bufs
                per_config.append(res)
            except Exception as exc:
                per_config.append({"workload": cname, "error": str(exc)[:300]})
            torch.cuda.empty_cache()

    product_kind = head["product_kernel"]
    product_ms = head["kernel_ms_per_step"].get(product_kind)
    achieved = head["product_tflops"]
    ours_gflops = whole_job_value(n, batch, ms, world)
    line = {
        "metric": METRIC, "value": ours_gflops, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "ms_per_step_mean": head["ms_per_step_mean"],
        "timing": "median over the CUDA-event intervals (one event per %d step(s)) of one timed region of %d steps (barrier + "
                  "synchronize on both sides, no per-launch events inside); max over ranks" % (head["steps_per_event"], args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": describe(args.workload), "schedule": sched_resolved, "levels": head["levels"],
                   "workspace_bytes": head["workspace_bytes"], "l2": head["l2"],
                   "parallelism": "replicas only (no collective)" if world > 1 else "single GPU"},
        "clocks": clocks,
        "e2e_error": e2e_error,
        "e2e": None if e2e_ms is None else
               {"value": whole_job_value(n, batch, e2e_pipe_ms or e2e_ms, world), "unit": UNIT,
                "ms_per_step": e2e_pipe_ms or e2e_ms,
                "mode": "strassen_dgemm_host, consecutive calls pipelined over plan-owned streams (STRASSEN_FLAG_HOST_PIPELINE)"
                        if e2e_pipe_ms else "strassen_dgemm_host, everything in stream order",
                "h2d_bytes_per_step": 2 * batch * n * n * 8, "d2h_bytes_per_step": batch * n * n * 8,
                "in_order_ms_per_step": e2e_ms, "pipelined_ms_per_step": e2e_pipe_ms},
        "gpu_launches": args.steps * launch_count,
        "roofline": {"bound": "alu",
                     "kernel": "gemm_f64_kernel (batched base products)" if product_kind == "gemm"
                               else "fused_step_kernel (sums, seven products and U-chain of the deepest step)",
                     "achieved": achieved, "peak": fp64_peak, "unit": "TFLOP/s", "frac": achieved / fp64_peak if achieved else None,
                     "peak_source": peak_source,
                     "peak_nominal": FP64_PEAK_NOMINAL_TFLOPS, "frac_of_nominal": achieved / FP64_PEAK_NOMINAL_TFLOPS if achieved else None,
                     "fp64_probe_tflops": probes,
                     "flops_per_step": f_base, "kernel_ms_per_step": product_ms,
                     "launches_per_step": head["launches_by_kind"].get(product_kind),
                     "launches": "the family's launches of one step are timed together (two CUDA events around each, a separate "
                                 "pass from the timed region); at n=4096 they are 342 leaves on 128 x 128 tiles and 1 leaf on "
                                 "32 x 64 tiles",
                     "traffic": GEMM_DRAM_TRAFFIC_BYTES.get(args.workload),
                     "traffic_source": "one ncu capture of this launch (profiles/), per step; not measured in this run"
                                       if GEMM_DRAM_TRAFFIC_BYTES.get(args.workload) else None},
        "path_roofline": dict(head["path_roofline"], kernel_ms_per_step=head["kernel_ms_per_step"]),
        "add_kernels": {k: head[k] for k in ("add_bytes_scheduled", "add_bytes_27h2", "add_gbs", "add_frac_of_measured_hbm",
                                             "add_frac_of_nominal_8000")},
        "actual_gflops": head["actual_gflops"] * world,
        "parity": {k: head.get(k) for k in ("max_err", "bound", "err_over_bound", "int_equal")},
        "autotuned": tuned,
        "cuda_graph_ms_per_step": graph_ms,
        "cublas_dgemm": head.get("cublas_dgemm"),
        "vs_cublas": head.get("vs_cublas"),
        "cpu_baseline": cpu,
        "per_config": per_config,
    }
    if world > 1:
        dist.destroy_process_group()         # first: whatever the communicator logs on its way out stays above the line
    sys.stdout.flush()
    print(json.dumps(line), flush=True)      # the last line of stdout


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the Strassen-Winograd hot path on B200: effective FP64 GFLOP/s (2 n^3 / t).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one whole product C = A.B (operand formation, the batched base products,
recombination) on one batch of seeded synthetic input.  With N > 1 (torchrun, one rank per
GPU) every rank runs an independent replica of the same product; there is no data-path
collective.  Rank 0 prints ONE JSON line.  `--impl reference` times the CPU oracle on the
host cores instead (a reported baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
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
METRIC = "effective FP64 GFLOP/s (2n^3/t)"
UNIT = "GFLOP/s"

# DRAM bytes (read + write) of the dominant kernel's launch from one ncu capture, per workload
# (profiles/gemm_f64_kernel_343x512.md); None where no capture of that exact launch exists.
GEMM_DRAM_TRAFFIC_BYTES = {"n4096": 2.125e9, "gemm512x343": 2.125e9}

# FP64 arithmetic peak from unit counts and clocks: 148 SMs x 64 FP64 FMA lanes x 2 flop x 1.965 GHz
FP64_PEAK_NOMINAL_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12


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
    """(base-product flops, sum/recombine bytes) one product must move: 7^L products of 2 m_L^3
    flops; per node per level 16 h^2 words to form the sums + 11 h^2 to recombine."""
    m = level_sizes(n, cutoff)
    L = len(m) - 1
    f_base = batch * 7 ** L * 2.0 * m[-1] ** 3
    b_alg = batch * 8.0 * sum(7 ** i * 27 * m[i + 1] ** 2 for i in range(L))
    return f_base, b_alg


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


def time_oracle_slab(n, A_host, B_host, target_seconds=12.0):
    """Time the classical oracle on a slab of rows of the same product; the slab is grown until it
    costs about target_seconds.  Returns (GFLOP/s, rows, seconds)."""
    import oracle
    rows, t = min(n, 32), 0.0
    while True:
        t0 = time.perf_counter()
        oracle.classical(A_host[:rows], B_host)
        t = time.perf_counter() - t0
        if rows >= n or t >= target_seconds / 3:
            break
        rows = min(n, max(rows * 2, int(rows * 0.6 * target_seconds / max(t, 1e-3))))
    return 2.0 * rows * n * n / t / 1e9, rows, t


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle as it stands, on the host cores, rank 0 only."""
    if rank != 0:
        return
    import numpy as np
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
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the timed CPU oracle leg")
    ap.add_argument("--no-cublas", action="store_true", help="skip the cuBLAS DGEMM comparator")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-probes", action="store_true", help="skip the FP64 rate probes")
    ap.add_argument("--no-autotune", action="store_true", help="skip the measured choice of steps and interleaving")
    ap.add_argument("--graph", action="store_true", help="also time the plan replayed as one CUDA graph")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_1202_3173_b200 import build as _build
    if local_rank == 0:
        _build.ensure_built()
    from paper_1202_3173_b200 import Plan, binding, inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    n, cutoff, sched, batch, dist_name, seed, budget = WORKLOADS[args.workload]
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

    # ---- device-resident timing -----------------------------------------------------------
    for _ in range(args.warmup):
        plan(A, B, out=C)
    barrier()
    plan.set_timing(True)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        plan(A, B, out=C)
    ev1.record(stream)
    barrier()
    w1 = time.time()
    clocks = sampler.stop(w0, w1) if sampler else None
    ms_local = ev0.elapsed_time(ev1) / args.steps
    kinds = plan.timings_ms()
    plan.set_timing(False)
    ms = reduce_max(ms_local, dev)

    sched_resolved = plan.schedule
    hA = hB = None
    if not args.no_e2e or (rank == 0 and not args.no_cpu_baseline):
        hA, hB = A.cpu().pin_memory(), B.cpu().pin_memory()

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

    # ---- rank 0: comparator, probes, CPU oracle, report ----------------------------------------
    f_base, b_alg = algorithmic_work(n, cutoff, batch)
    gemm_launches = plan.launches_by_kind()["gemm"]
    gemm_ms = kinds["gemm"] / (args.steps * gemm_launches)
    achieved_tflops = f_base / gemm_launches / (gemm_ms * 1e-3) / 1e12

    probes = {}
    for kind, name in enumerate(("dfma", "dmma_m8n8k4", "dmma_m16n8k4", "dmma_m16n8k8", "dmma_m16n8k16")):
        if args.no_probes:
            break
        try:
            probes[name] = round(binding.strassen_probe_fp64(kind, 20000, stream.cuda_stream), 2)
        except Exception as exc:   # a probe is context, never fatal
            probes[name] = str(exc)
    fp64_measured = max([v for v in probes.values() if isinstance(v, float)] or [FP64_PEAK_NOMINAL_TFLOPS])

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        hbm_gbs, hbm_src = json.load(open(peaks_path))["hbm_gbs"], "measured"
    else:
        hbm_gbs, hbm_src = 6650.0, "fallback"
    t_roof_ms = (f_base / (FP64_PEAK_NOMINAL_TFLOPS * 1e12) + b_alg / (hbm_gbs * 1e9)) * 1e3

    cublas = None
    if not args.no_cublas:
        Cc = torch.empty_like(A)
        for _ in range(3):
            torch.matmul(A, B, out=Cc)
        torch.cuda.synchronize()
        reps = max(3, min(args.steps, 10))
        ev0.record(stream)
        for _ in range(reps):
            torch.matmul(A, B, out=Cc)
        ev1.record(stream)
        torch.cuda.synchronize()
        cms = ev0.elapsed_time(ev1) / reps
        cublas = {"ms": cms, "gflops": 2.0 * n ** 3 * batch / (cms * 1e-3) / 1e9,
                  "max_abs_diff_vs_ours": float((Cc - C).abs().max()) if n <= 16384 else None}
        del Cc

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
        import oracle
        a_h = (hA if batch == 1 else hA[0]).numpy()
        b_h = (hB if batch == 1 else hB[0]).numpy()
        g, rows, secs = time_oracle_slab(n, a_h, b_h)
        cpu = {"value": g, "unit": UNIT, "cores": oracle.cores(), "kind": "oracle",
               "sample": "classical oracle on the first %d of %d rows of one product (%.1f s); classical flops "
                         "equal effective flops, so the rate stands for the whole product" % (rows, n, secs)}

    launches_by_kind, launch_count, level_list, ws_bytes = (plan.launches_by_kind(), plan.launch_count, plan.level_sizes,
                                                        plan.workspace_bytes)
    (e2e_ms, e2e_pipe_ms), e2e_error = run_e2e()
    ours_gflops = whole_job_value(n, batch, ms, world)
    line = {
        "metric": METRIC, "value": ours_gflops, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": describe(args.workload), "schedule": sched_resolved, "levels": level_list,
                   "workspace_bytes": ws_bytes,
                   "l2": "inputs larger than L2 (A+B+C %.0f MB + workspace)" % (3 * batch * n * n * 8 / 1e6)
                         if 3 * batch * n * n * 8 > 126e6 else "L2-resident problem (A+B+C %.1f MB): launch-bound"
                         % (3 * batch * n * n * 8 / 1e6),
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
        "roofline": {"bound": "alu", "kernel": "gemm_f64_kernel (batched base products)", "achieved": achieved_tflops,
                     "peak": FP64_PEAK_NOMINAL_TFLOPS, "unit": "TFLOP/s", "frac": achieved_tflops / FP64_PEAK_NOMINAL_TFLOPS,
                     "peak_source": "148 SMs x 64 FP64 FMA/clk x 2 x 1.965 GHz (unit counts and max clock)",
                     "fp64_probe_tflops": probes, "frac_of_probe": achieved_tflops / fp64_measured,
                     "ms_per_launch": gemm_ms, "flops_per_launch": f_base / gemm_launches,
                     "traffic": GEMM_DRAM_TRAFFIC_BYTES.get(args.workload)},
        "path_roofline": {"t_roof_ms": t_roof_ms, "frac": t_roof_ms / ms_local, "base_flops": f_base, "add_bytes": b_alg,
                          "hbm_gbs": hbm_gbs, "hbm_source": hbm_src,
                          "kernel_ms_per_step": {k: v / args.steps for k, v in kinds.items()}},
        "actual_gflops": (f_base + 15 * b_alg / (27 * 8)) / (ms * 1e-3) / 1e9 * world,
        "autotuned": tuned,
        "cuda_graph_ms_per_step": graph_ms,
        "cublas_dgemm": cublas,
        "vs_cublas": (cublas["ms"] / ms_local) if cublas else None,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    plan.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Seeded synthetic input generators shared by the tests and the benchmark.

This module holds none of the method's arithmetic: it only draws matrices.  The
paper's workload is a pair of dense square FP64 matrices (Section 5.1) whose
values are not described, so three value distributions are offered:

* ``"uniform"`` -- uniform in [-1, 1)
* ``"normal"``  -- standard normal
* ``"int8"``    -- integers uniform in [-8, 8] stored as FP64; with these every
  intermediate of the Strassen-Winograd recursion is an exactly representable
  integer, so any correct implementation returns the same values.

Matrices are drawn with a ``torch.Generator`` on the requested device (the CPU and
CUDA generators are different streams; a test draws once and hands the same bits
to both sides).
"""
from __future__ import annotations

import torch

DISTRIBUTIONS = ("uniform", "normal", "int8")


def matrix(shape, dist: str = "uniform", seed: int = 0, device="cpu") -> torch.Tensor:
    """A contiguous float64 tensor of ``shape`` drawn from ``dist`` with ``seed``."""
    if isinstance(shape, int):
        shape = (shape, shape)
    shape = tuple(int(s) for s in shape)
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    if dist == "uniform":
        x = torch.rand(shape, dtype=torch.float64, device=device, generator=g)
        return x.mul_(2.0).sub_(1.0)
    if dist == "normal":
        return torch.randn(shape, dtype=torch.float64, device=device, generator=g)
    if dist == "int8":
        x = torch.randint(-8, 9, shape, dtype=torch.int32, device=device, generator=g)
        return x.to(torch.float64)
    raise ValueError("dist must be one of %s" % (DISTRIBUTIONS,))


def pair(n: int, dist: str = "uniform", seed: int = 0, device="cpu", batch: int | None = None):
    """(A, B): two n x n matrices (or batch x n x n) with seeds ``seed`` and ``seed + 1``."""
    shape = (n, n) if batch is None else (batch, n, n)
    return matrix(shape, dist, seed, device), matrix(shape, dist, seed + 1, device)

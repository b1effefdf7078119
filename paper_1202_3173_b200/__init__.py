"""B200-native Strassen-Winograd product C = A.B (the single-GPU hot path of CAPS).

The work is done by ``libstrassen_b200.so`` (CUDA, sm_100a; C ABI in
``include/strassen_b200.h``).  ``binding`` mirrors that ABI one to one; ``Plan`` adds
only what PyTorch is used for here: device memory for C and the workspace, and the
current CUDA stream.  Nothing in this package computes on the CPU.
"""
from __future__ import annotations

from . import binding
from .binding import StrassenError  # noqa: F401

__all__ = ["Plan", "matmul", "autotune", "binding", "StrassenError"]


class Plan:
    """A planned product for n x n FP64 matrices (optionally a batch of them).

    ``schedule`` is one 'B' (breadth-first step) or 'D' (depth-first step) per recursion
    level, or None / "auto" for the Limited-Memory rule against ``workspace_budget_bytes``.
    ``cutoff`` 0 lets the library choose the number of steps (and, with schedule None, the
    interleaving) by its cost model.
    """

    def __init__(self, n, cutoff=0, schedule=None, batch=1, workspace_budget_bytes=0, lda=0, ldb=0, ldc=0,
                 stride_a=0, stride_b=0, stride_c=0, flags=0, scheme=None):
        """``scheme``: None for the Strassen-Winograd step of the paper's Appendix A; the name of a built-in
        bilinear scheme ("classical", "strassen", "winograd"); or a tuple (n0, q, u, v, w) of coefficient tables
        for any <n0, n0, n0; q> scheme (Section 6.6) -- sizes must then divide by n0 at every level."""
        self.n, self.cutoff, self.batch = int(n), int(cutoff), int(batch)
        if scheme is None:
            self._h = binding.strassen_plan_create_ex(n, cutoff, schedule, batch, lda, ldb, ldc, stride_a, stride_b,
                                                      stride_c, workspace_budget_bytes, flags)
        else:
            if lda or ldb or ldc or stride_a or stride_b or stride_c:
                raise ValueError("plans for a generic scheme take packed matrices")
            if isinstance(scheme, str):
                self._h = binding.strassen_plan_create_named_scheme(n, cutoff, schedule, scheme, batch,
                                                                    workspace_budget_bytes, flags)
            else:
                n0, q, u, v, w = scheme
                self._h = binding.strassen_plan_create_scheme(n, cutoff, schedule, n0, q, u, v, w, batch,
                                                              workspace_budget_bytes, flags)
        self._ws = None
        self._packed = not (lda or ldb or ldc or stride_a or stride_b or stride_c)
        self._want = (self.n, self.n) if self.batch == 1 else (self.batch, self.n, self.n)

    # -- introspection -------------------------------------------------------------
    @property
    def handle(self):
        return self._h

    @property
    def schedule(self):
        return binding.strassen_plan_schedule(self._h)

    @property
    def levels(self):
        return binding.strassen_plan_levels(self._h)

    @property
    def level_sizes(self):
        return [binding.strassen_plan_level_size(self._h, i) for i in range(self.levels + 1)]

    @property
    def base_size(self):
        return binding.strassen_plan_base_size(self._h)

    @property
    def base_products(self):
        return binding.strassen_plan_base_products(self._h)

    @property
    def workspace_bytes(self):
        return binding.strassen_plan_workspace_bytes(self._h)

    @property
    def workspace(self):
        """The torch tensor holding the workspace (None before the first call or for plans without one)."""
        return self._ws

    @property
    def pass_bytes(self):
        """HBM bytes the streaming passes (sums, recombination, DFS folds, peeling) move per product as scheduled."""
        return binding.strassen_plan_pass_bytes(self._h)

    @property
    def model_ms(self):
        return binding.strassen_plan_model_ms(self._h)

    @property
    def launch_count(self):
        return binding.strassen_plan_launch_count(self._h)

    def launches_by_kind(self):
        return {k: binding.strassen_plan_launches_of(self._h, i) for i, k in enumerate(binding.KERNEL_KINDS)}

    # -- execution -----------------------------------------------------------------
    def _ensure_workspace(self, device):
        import torch
        need = self.workspace_bytes
        if need and self._ws is None:
            self._ws = torch.empty(need, dtype=torch.uint8, device=device)
            binding.strassen_plan_set_workspace(self._h, self._ws.data_ptr(), need)

    def _check(self, what, cuda, *tensors):
        """The kernels index the tensors by the plan's n and batch alone: anything smaller than that would be
        read or written out of bounds on the device, so shapes are checked here and not left to the library."""
        import torch
        if not self._h:
            raise ValueError("the plan has been closed")
        if not self._packed:
            raise ValueError("plans with leading dimensions or strides take raw pointers (binding.strassen_dgemm)")
        want, f64, dev0 = self._want, torch.float64, tensors[0].device
        for name, t in zip(what, tensors):
            if t.shape == want and t.dtype is f64 and t.is_cuda is cuda and t.is_contiguous() and t.device == dev0:
                continue
            if t.dtype != f64:
                raise ValueError("%s must be float64, not %s" % (name, t.dtype))
            if tuple(t.shape) != want:
                raise ValueError("%s has shape %s; the plan is for %s" % (name, tuple(t.shape), want))
            if not t.is_contiguous():
                raise ValueError("%s must be contiguous" % name)
            if t.is_cuda != cuda:
                raise ValueError("%s must be a %s tensor" % (name, "CUDA" if cuda else "host"))
            raise ValueError("%s is on %s, A on %s" % (name, t.device, dev0))

    def __call__(self, A, B, out=None):
        """C = A @ B for CUDA float64 tensors of the plan's shape, enqueued on the current stream."""
        import torch
        if out is None:
            self._check("AB", True, A, B)
            out = torch.empty_like(A)
        else:
            self._check(("A", "B", "out"), True, A, B, out)
        if self._ws is None:
            self._ensure_workspace(A.device)
        index = A.device.index
        if index == torch.cuda.current_device():
            binding.strassen_dgemm(self._h, A.data_ptr(), B.data_ptr(), out.data_ptr(), torch.cuda.current_stream().cuda_stream)
        else:
            with torch.cuda.device(index):
                binding.strassen_dgemm(self._h, A.data_ptr(), B.data_ptr(), out.data_ptr(),
                                       torch.cuda.current_stream().cuda_stream)
        return out

    def run_host(self, A, B, out):
        """The same product for host (ideally pinned) tensors, copies included, on the current stream."""
        import torch
        self._check(("A", "B", "out"), False, A, B, out)
        self._ensure_workspace(torch.device("cuda", torch.cuda.current_device()))
        stream = torch.cuda.current_stream().cuda_stream
        binding.strassen_dgemm_host(self._h, A.data_ptr(), B.data_ptr(), out.data_ptr(), stream)
        return out

    def set_timing(self, enabled=True):
        binding.strassen_plan_set_timing(self._h, enabled)

    def timings_ms(self):
        return binding.strassen_plan_get_timings(self._h)

    def close(self):
        """Destroy the plan.  Launches that still use its workspace may be in flight on any stream, so the device
        the workspace lives on is synchronised before the memory goes back to torch's allocator."""
        if self._h:
            if self._ws is not None:
                import torch
                torch.cuda.synchronize(self._ws.device)
            binding.strassen_plan_destroy(self._h)
            self._h = None
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def matmul(A, B, cutoff=0, schedule=None, workspace_budget_bytes=0):
    """One-shot C = A @ B for square CUDA float64 tensors (2-D, or 3-D for a batch)."""
    import torch
    if A.dim() not in (2, 3) or A.shape != B.shape or A.shape[-1] != A.shape[-2]:
        raise ValueError("A and B must be square matrices (or batches of them) of equal shape, got %s and %s"
                         % (tuple(A.shape), tuple(B.shape)))
    batch = 1 if A.dim() == 2 else A.shape[0]
    n = A.shape[-1]
    plan = Plan(n, cutoff, schedule, batch=batch, workspace_budget_bytes=workspace_budget_bytes)
    try:
        C = plan(A, B)
        torch.cuda.current_stream().synchronize()
    finally:
        plan.close()
    return C


def autotune(A, B, workspace_budget_bytes, min_base=0, repetitions=0, max_seconds=0.0):
    """Measure every (number of Strassen steps, BFS/DFS string) candidate that fits the budget on
    A @ B and return (best, log, C): dicts with cutoff / levels / schedule / ms, and the product
    computed with the winning plan.  torch supplies C and the workspace; the search itself runs
    inside the library (strassen_autotune)."""
    import torch
    if (A.dim() not in (2, 3) or A.shape != B.shape or A.shape[-1] != A.shape[-2] or not (A.is_cuda and B.is_cuda)
            or A.dtype != torch.float64 or B.dtype != torch.float64 or not (A.is_contiguous() and B.is_contiguous())):
        raise ValueError("A and B must be contiguous square CUDA float64 matrices (or batches) of equal shape")
    batch = 1 if A.dim() == 2 else A.shape[0]
    n = A.shape[-1]
    C = torch.empty_like(A)
    ws = torch.empty(max(int(workspace_budget_bytes), 256), dtype=torch.uint8, device=A.device)
    with torch.cuda.device(A.device):
        stream = torch.cuda.current_stream().cuda_stream
        best, log = binding.strassen_autotune(n, A.data_ptr(), B.data_ptr(), C.data_ptr(), ws.data_ptr(),
                                              int(workspace_budget_bytes), stream, batch, min_base, repetitions, max_seconds)
    return best, log, C

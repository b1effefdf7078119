"""Thin ctypes binding of libstrassen_b200.so -- argument marshalling only.

Every function here has the name of the C entry point it calls (include/strassen_b200.h)
and does no arithmetic of the method: all steps run in the library's CUDA kernels.
There is no fallback: if the shared library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstrassen_b200.so")

STRASSEN_OK = 0
STRASSEN_FLAG_SINGLE_LEVEL_PASSES = 1
STRASSEN_FLAG_CUDA_GRAPH = 2
STRASSEN_FLAG_HOST_PIPELINE = 4
STRASSEN_FLAG_SCALE_OUTSIDE = 8
STRASSEN_FLAG_SCALE_INSIDE = 16
STRASSEN_FLAG_TWO_LEVEL_PASSES = 32
STRASSEN_FLAG_FUSED_STEP = 64
STRASSEN_FLAG_NO_FUSED_STEP = 128
STRASSEN_FLAG_NO_DFS_FOLD = 256
STATUS_NAMES = {0: "OK", -1: "INVALID_ARG", -2: "BAD_SCHEDULE", -3: "WORKSPACE_TOO_SMALL", -4: "ALIAS",
                -5: "MISALIGNED", -6: "CUDA_ERROR", -7: "OUT_OF_MEMORY"}
K_FORM, K_GEMM, K_RECOMBINE, K_FORM_ONE, K_ACCUMULATE, K_PEEL, K_SCALE, K_FUSED_STEP, K_LINCOMB, K_COUNT = range(10)
KERNEL_KINDS = ("form", "gemm", "recombine", "form_one", "accumulate", "peel", "scale", "fused_step", "lincomb")

# every symbol the header declares: (name, restype, argtypes)
_vp, _i64, _sz, _cp, _int = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_char_p, ctypes.c_int
_dp = ctypes.POINTER(ctypes.c_double)


class strassen_options(ctypes.Structure):
    _fields_ = [("n", _i64), ("cutoff", _i64), ("schedule", _cp), ("batch", _i64),
                ("lda", _i64), ("ldb", _i64), ("ldc", _i64),
                ("stride_a", _i64), ("stride_b", _i64), ("stride_c", _i64),
                ("workspace_budget_bytes", _sz), ("flags", _i64)]


class strassen_scheme(ctypes.Structure):
    _fields_ = [("n0", _int), ("q", _int), ("u", ctypes.POINTER(ctypes.c_int8)), ("v", ctypes.POINTER(ctypes.c_int8)),
                ("w", ctypes.POINTER(ctypes.c_int8))]


class strassen_tune_request(ctypes.Structure):
    _fields_ = [("n", _i64), ("batch", _i64), ("min_base", _i64), ("repetitions", _int), ("max_seconds", ctypes.c_double),
                ("A", _vp), ("B", _vp), ("C", _vp), ("workspace", _vp), ("workspace_bytes", _sz), ("stream", _vp)]


class strassen_tune_entry(ctypes.Structure):
    _fields_ = [("cutoff", _i64), ("levels", _int), ("schedule", ctypes.c_char * 36), ("ms", ctypes.c_double),
                ("model_ms", ctypes.c_double)]

    def as_dict(self):
        return {"cutoff": int(self.cutoff), "levels": int(self.levels), "schedule": self.schedule.decode(), "ms": float(self.ms),
                "model_ms": float(self.model_ms)}


SYMBOLS = [
    ("strassen_plan_create", _vp, [_i64, _i64, _cp]),
    ("strassen_plan_create_ex", _vp, [ctypes.POINTER(strassen_options)]),
    ("strassen_dgemm", _int, [_vp, _vp, _vp, _vp, _vp]),
    ("strassen_dgemm_host", _int, [_vp, _vp, _vp, _vp, _vp]),
    ("strassen_plan_destroy", None, [_vp]),
    ("strassen_plan_workspace_bytes", _sz, [_vp]),
    ("strassen_plan_set_workspace", _int, [_vp, _vp, _sz]),
    ("strassen_plan_schedule", _cp, [_vp]),
    ("strassen_plan_levels", _int, [_vp]),
    ("strassen_plan_level_size", _i64, [_vp, _int]),
    ("strassen_plan_base_size", _i64, [_vp]),
    ("strassen_plan_base_products", _i64, [_vp]),
    ("strassen_plan_launch_count", _i64, [_vp]),
    ("strassen_plan_launches_of", _i64, [_vp, _int]),
    ("strassen_plan_pass_bytes", ctypes.c_double, [_vp]),
    ("strassen_plan_model_ms", ctypes.c_double, [_vp]),
    ("strassen_schedule_model_bytes", _sz, [_i64, _i64, _i64, _cp, _int]),
    ("strassen_plan_set_timing", _int, [_vp, _int]),
    ("strassen_plan_get_timings", _int, [_vp, _dp]),
    ("strassen_autotune", _int, [ctypes.POINTER(strassen_tune_request), ctypes.POINTER(strassen_tune_entry),
                                 ctypes.POINTER(strassen_tune_entry), _int, ctypes.POINTER(_int)]),
    ("strassen_probe_fp64", _int, [_int, _i64, _vp, _dp]),
    ("strassen_scheme_check", _int, [ctypes.POINTER(strassen_scheme)]),
    ("strassen_plan_create_scheme", _vp, [ctypes.POINTER(strassen_options), ctypes.POINTER(strassen_scheme)]),
    ("strassen_plan_create_named_scheme", _vp, [ctypes.POINTER(strassen_options), _cp]),
    ("strassen_bfs_form_shares", _int, [_i64, _i64, _vp, _i64, _vp, _i64, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _i64, _vp]),
    ("strassen_bfs_combine_shares", _int, [_i64, _i64, ctypes.POINTER(_vp), _i64, _vp, _i64, _vp]),
    ("strassen_dgemm_static", _int, [_i64, _vp, _vp, _vp, _vp]),
    ("strassen_last_error", _cp, []),
]
STRASSEN_STATIC_MAX_N = 512

_lib = None


class StrassenError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s (%d): %s" % (STATUS_NAMES.get(status, "?"), status, message))
        self.status = status


def lib() -> ctypes.CDLL:
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libstrassen_b200.so is missing: run `python -m paper_1202_3173_b200.build` "
                               "(there is no fallback path)")
        l = ctypes.CDLL(LIB_PATH)
        for name, res, args in SYMBOLS:
            f = getattr(l, name)
            f.restype, f.argtypes = res, args
        _lib = l
    return _lib


def strassen_last_error() -> str:
    return lib().strassen_last_error().decode()


def _check(status: int) -> None:
    if status != STRASSEN_OK:
        raise StrassenError(status, strassen_last_error())


def _sched(schedule):
    return None if schedule is None else schedule.encode()


def strassen_plan_create(n: int, cutoff: int, schedule) -> int:
    h = lib().strassen_plan_create(n, cutoff, _sched(schedule))
    if not h:
        raise StrassenError(-1, strassen_last_error())
    return h


def strassen_plan_create_ex(n, cutoff, schedule=None, batch=1, lda=0, ldb=0, ldc=0, stride_a=0, stride_b=0,
                            stride_c=0, workspace_budget_bytes=0, flags=0) -> int:
    o = strassen_options(n, cutoff, _sched(schedule), batch, lda, ldb, ldc, stride_a, stride_b, stride_c,
                         workspace_budget_bytes, flags)
    h = lib().strassen_plan_create_ex(ctypes.byref(o))
    if not h:
        raise StrassenError(-1, strassen_last_error())
    return h


def strassen_dgemm(plan: int, A: int, B: int, C: int, stream: int = 0) -> None:
    """A, B, C: device addresses (ints); stream: a cudaStream_t handle (int)."""
    _check(lib().strassen_dgemm(plan, A, B, C, stream))


def strassen_dgemm_host(plan: int, A: int, B: int, C: int, stream: int = 0) -> None:
    """A, B, C: host addresses (ints)."""
    _check(lib().strassen_dgemm_host(plan, A, B, C, stream))


def strassen_plan_destroy(plan: int) -> None:
    lib().strassen_plan_destroy(plan)


def strassen_plan_workspace_bytes(plan: int) -> int:
    return lib().strassen_plan_workspace_bytes(plan)


def strassen_plan_set_workspace(plan: int, device_ptr: int, nbytes: int) -> None:
    _check(lib().strassen_plan_set_workspace(plan, device_ptr, nbytes))


def strassen_plan_schedule(plan: int) -> str:
    return lib().strassen_plan_schedule(plan).decode()


def strassen_plan_levels(plan: int) -> int:
    return lib().strassen_plan_levels(plan)


def strassen_plan_level_size(plan: int, level: int) -> int:
    return lib().strassen_plan_level_size(plan, level)


def strassen_plan_base_size(plan: int) -> int:
    return lib().strassen_plan_base_size(plan)


def strassen_plan_base_products(plan: int) -> int:
    return lib().strassen_plan_base_products(plan)


def strassen_plan_launch_count(plan: int) -> int:
    return lib().strassen_plan_launch_count(plan)


def strassen_plan_launches_of(plan: int, kind: int) -> int:
    return lib().strassen_plan_launches_of(plan, kind)


def strassen_plan_pass_bytes(plan: int) -> float:
    return lib().strassen_plan_pass_bytes(plan)


def strassen_plan_model_ms(plan: int) -> float:
    return lib().strassen_plan_model_ms(plan)


def strassen_schedule_model_bytes(n, cutoff, batch, schedule, accounting=21) -> int:
    v = lib().strassen_schedule_model_bytes(n, cutoff, batch, _sched(schedule), accounting)
    if v == 0 and strassen_last_error():
        raise StrassenError(-2, strassen_last_error())
    return v


def strassen_plan_set_timing(plan: int, enabled: bool) -> None:
    _check(lib().strassen_plan_set_timing(plan, int(enabled)))


def strassen_plan_get_timings(plan: int):
    out = (ctypes.c_double * K_COUNT)()
    _check(lib().strassen_plan_get_timings(plan, out))
    return dict(zip(KERNEL_KINDS, list(out)))


def strassen_dgemm_static(n: int, A: int, B: int, C: int, stream: int = 0) -> None:
    """One Strassen-Winograd level with all temporaries in the library's static device array:
    for callers that must not allocate device memory.  A, B, C: device addresses, rows of n."""
    _check(lib().strassen_dgemm_static(n, A, B, C, stream))


def strassen_autotune(n, A, B, C, workspace, workspace_bytes, stream=0, batch=1, min_base=0, repetitions=0,
                      max_seconds=0.0, log_capacity=256):
    """Returns (best, log): dicts with cutoff / levels / schedule / ms.  A, B, C, workspace: device addresses."""
    req = strassen_tune_request(n, batch, min_base, repetitions, max_seconds, A, B, C, workspace, workspace_bytes, stream)
    best = strassen_tune_entry()
    log = (strassen_tune_entry * max(log_capacity, 1))()
    count = _int(0)
    _check(lib().strassen_autotune(ctypes.byref(req), ctypes.byref(best), log, log_capacity, ctypes.byref(count)))
    return best.as_dict(), [log[i].as_dict() for i in range(count.value)]


def _scheme(n0, q, u, v, w):
    """(struct, keep-alive) for tables given as nested sequences: u, v are q x n0^2, w is n0^2 x q."""
    def flat(t, rows, cols):
        cells = [int(x) for row in t for x in row]
        if len(t) != rows or len(cells) != rows * cols:
            raise ValueError("a %d x %d table is expected" % (rows, cols))
        return (ctypes.c_int8 * len(cells))(*cells)
    bu, bv, bw = flat(u, q, n0 * n0), flat(v, q, n0 * n0), flat(w, n0 * n0, q)
    return strassen_scheme(n0, q, bu, bv, bw), (bu, bv, bw)


def strassen_scheme_check(n0, q, u, v, w) -> None:
    s, keep = _scheme(n0, q, u, v, w)
    _check(lib().strassen_scheme_check(ctypes.byref(s)))


def strassen_plan_create_scheme(n, cutoff, schedule, n0, q, u, v, w, batch=1, workspace_budget_bytes=0, flags=0) -> int:
    o = strassen_options(n, cutoff, _sched(schedule), batch, 0, 0, 0, 0, 0, 0, workspace_budget_bytes, flags)
    s, keep = _scheme(n0, q, u, v, w)
    h = lib().strassen_plan_create_scheme(ctypes.byref(o), ctypes.byref(s))
    if not h:
        raise StrassenError(-1, strassen_last_error())
    return h


def strassen_plan_create_named_scheme(n, cutoff, schedule, name, batch=1, workspace_budget_bytes=0, flags=0) -> int:
    o = strassen_options(n, cutoff, _sched(schedule), batch, 0, 0, 0, 0, 0, 0, workspace_budget_bytes, flags)
    h = lib().strassen_plan_create_named_scheme(ctypes.byref(o), name.encode())
    if not h:
        raise StrassenError(-1, strassen_last_error())
    return h


def _ptr7(addresses):
    if len(addresses) != 7:
        raise ValueError("seven block addresses expected, got %d" % len(addresses))
    return (_vp * 7)(*[int(a) for a in addresses])


def strassen_bfs_form_shares(rows: int, h: int, A_share: int, lda: int, B_share: int, ldb: int, T_out, S_out, ld_out: int,
                             stream: int = 0) -> None:
    """T_out, S_out: seven device addresses each (block r of T_0..T_6 / S_0..S_6, rows x h)."""
    _check(lib().strassen_bfs_form_shares(rows, h, A_share, lda, B_share, ldb, _ptr7(T_out), _ptr7(S_out), ld_out, stream))


def strassen_bfs_combine_shares(rows: int, h: int, Q_in, ldq: int, C_share: int, ldc: int, stream: int = 0) -> None:
    """Q_in: seven device addresses (block r of Q_0..Q_6, rows x h)."""
    _check(lib().strassen_bfs_combine_shares(rows, h, _ptr7(Q_in), ldq, C_share, ldc, stream))


def strassen_probe_fp64(kind: int, iters: int, stream: int = 0) -> float:
    out = ctypes.c_double()
    _check(lib().strassen_probe_fp64(kind, iters, stream, ctypes.byref(out)))
    return out.value

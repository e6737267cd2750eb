"""Thin ctypes binding over ``libfpsk.so`` (the C ABI declared in ``include/fpsk.h``).

Argument marshalling only: every step of the verifier runs inside the CUDA library.  PyTorch
supplies device memory and streams.  If the library has not been built this module raises;
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfpsk.so")
# FPSK_LIBRARY names another build of the same library to load instead (the index-checked libfpsk_bounds.so)
if os.environ.get("FPSK_LIBRARY"):
    LIB_PATH = os.path.abspath(os.environ["FPSK_LIBRARY"])

FP16, BF16 = 0, 1
STATUS_OK = 0
ERR_NULL, ERR_SHAPE, ERR_DTYPE, ERR_ALIGN, ERR_WORKSPACE, ERR_BUCKETS, ERR_CAPACITY, ERR_CUDA, ERR_TIMEOUT, ERR_PARAM = range(1, 11)


class ProbeResult(C.Structure):
    _fields_ = [("fired", C.c_int32), ("nonfinite", C.c_int32), ("argmax_col", C.c_int32), ("status", C.c_int32),
                ("max_abs", C.c_float), ("sigma_hat", C.c_float), ("thr", C.c_float), ("tau", C.c_float)]


class Fault(C.Structure):
    _fields_ = [("i", C.c_int32), ("j", C.c_int32), ("delta", C.c_double), ("recompute", C.c_double),
                ("c_value", C.c_float), ("round", C.c_int32), ("bucket_a", C.c_int32), ("bucket_b", C.c_int32)]


class Params(C.Structure):
    _fields_ = [("rounds", C.c_int32), ("r_star", C.c_int32), ("r_max", C.c_int32), ("radius", C.c_int32),
                ("s_budget", C.c_int32), ("delta_max", C.c_int32), ("mad_of_abs", C.c_int32), ("tensor_cores", C.c_int32),
                ("b_transposed", C.c_int32), ("scale_cap", C.c_int32),
                ("rho_min", C.c_double), ("c_valid", C.c_double), ("mu", C.c_double), ("b_star", C.c_double),
                ("c_coll", C.c_double), ("context", C.c_void_p)]


class Noise(C.Structure):
    _fields_ = [("sigma_clip", C.c_double), ("sigma_mad", C.c_double), ("rms_c", C.c_double), ("c_hat", C.c_double),
                ("index_budget_B", C.c_double), ("m0", C.c_int32), ("m_probe", C.c_int32), ("m_loc", C.c_int32),
                ("radius", C.c_int32)]


class RepairReport(C.Structure):
    _fields_ = [("state", C.c_int32), ("n_faults", C.c_int32), ("n_absolute", C.c_int32), ("m_loc", C.c_int32),
                ("radius", C.c_int32), ("reserved", C.c_int32), ("first_probe", ProbeResult), ("second_probe", ProbeResult)]


class BSide(C.Structure):
    """Host record of a cached B side (fpsk_bside)."""
    _fields_ = [("B", C.c_void_p), ("cache", C.c_void_p), ("ldb", C.c_int64), ("m", C.c_int64), ("k", C.c_int64),
                ("n", C.c_int64), ("seed", C.c_uint64), ("version", C.c_uint64), ("dtype", C.c_int32),
                ("n_buckets", C.c_int32), ("round", C.c_int32), ("valid", C.c_int32), ("rebuilds", C.c_int32),
                ("b_transposed", C.c_int32), ("built_transposed", C.c_int32), ("reserved", C.c_int32)]


class ProbeState(C.Structure):
    """fpsk_probe_state: what a probe keeps between calls (device memory, 32 bytes)."""
    _fields_ = [("calls", C.c_uint32), ("clean_calls", C.c_uint32), ("fired_any", C.c_uint32),
                ("first_fired_call", C.c_uint32), ("sigma_sum", C.c_double), ("reserved", C.c_double)]


class FpskError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: fpsk status {status} ({status_string(status)})")


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library; raises if it is missing (build it with
    ``python -m paper_2609_19758_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_19758_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32, u64, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_size_t
        L.fpsk_status_string.restype = C.c_char_p
        L.fpsk_status_string.argtypes = [C.c_int]
        L.fpsk_default_params.restype = None
        L.fpsk_default_params.argtypes = [C.POINTER(Params)]
        L.fpsk_law_m_start.restype = i32
        L.fpsk_law_m_start.argtypes = [i64, i64, i64, C.c_int, C.POINTER(Params)]
        L.fpsk_plan.restype = C.c_int
        L.fpsk_plan.argtypes = [i64, i64, i64, C.c_int, C.c_double, C.c_double, i32, C.POINTER(Params),
                                C.POINTER(i32), C.POINTER(i32), C.POINTER(C.c_double)]
        L.fpsk_probe_workspace_bytes.restype = sz
        L.fpsk_probe_workspace_bytes.argtypes = [i64, i64, i64]
        L.fpsk_probe_init.restype = C.c_int
        L.fpsk_probe_init.argtypes = [vp, sz, vp]
        L.fpsk_probe.restype = C.c_int
        L.fpsk_probe.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, C.c_int, C.c_int, C.POINTER(Params),
                                 vp, sz, vp, vp, vp]
        L.fpsk_probe_host_workspace_bytes.restype = sz
        L.fpsk_probe_host_workspace_bytes.argtypes = [i64, i64, i64]
        L.fpsk_probe_host.restype = C.c_int
        L.fpsk_probe_host.argtypes = [vp, vp, vp, i64, i64, i64, C.c_int, C.POINTER(Params), vp, sz, vp,
                                      C.POINTER(ProbeResult)]
        L.fpsk_probe_static.restype = C.c_int
        L.fpsk_probe_static.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, C.c_int, C.c_int, C.POINTER(Params),
                                        vp, vp, vp]
        L.fpsk_probe_hashed_cache_bytes.restype = sz
        L.fpsk_probe_hashed_cache_bytes.argtypes = [i64, i64, i64, i32]
        L.fpsk_probe_hashed_workspace_bytes.restype = sz
        L.fpsk_probe_hashed_workspace_bytes.argtypes = [i64, i64, i64, i32]
        L.fpsk_bside_matches.restype = i32
        L.fpsk_bside_matches.argtypes = [C.POINTER(BSide), vp, i64, u64, i64, i64, i64, C.c_int, u64, i32, i32, vp]
        L.fpsk_probe_hashed.restype = C.c_int
        L.fpsk_probe_hashed.argtypes = [C.POINTER(BSide), vp, i64, vp, i64, u64, vp, i64, i64, i64, i64, C.c_int, C.c_int,
                                        u64, i32, i32, C.POINTER(Params), vp, sz, vp, sz, vp, vp, vp, vp]
        L.fpsk_probe_state_reset.restype = C.c_int
        L.fpsk_probe_state_reset.argtypes = [vp, vp]
        L.fpsk_probe_accumulate.restype = C.c_int
        L.fpsk_probe_accumulate.argtypes = [vp, vp, vp]
        L.fpsk_recalibration_due.restype = i32
        L.fpsk_recalibration_due.argtypes = [C.c_uint32]
        L.fpsk_probe_recalibrate.restype = C.c_int
        L.fpsk_probe_recalibrate.argtypes = [i64, i64, C.c_double, C.c_double, i32, C.POINTER(Params),
                                             C.POINTER(i32), C.POINTER(i32)]
        L.fpsk_hash_tables.restype = C.c_int
        L.fpsk_hash_tables.argtypes = [u64, i32, i32, i64, i32, vp, vp, vp]
        L.fpsk_workspace_bytes.restype = sz
        L.fpsk_workspace_bytes.argtypes = [i64, i64, i64, i32, C.POINTER(Params)]
        L.fpsk_max_buckets.restype = i32
        L.fpsk_max_buckets.argtypes = [i64, i64, i64]
        L.fpsk_sketches.restype = C.c_int
        L.fpsk_sketches.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, C.c_int, u64, i32, i32, C.POINTER(Params), vp, sz, vp,
                                    vp, vp, vp]
        L.fpsk_measure_noise.restype = C.c_int
        L.fpsk_measure_noise.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, C.c_int, u64, i32,
                                         C.POINTER(Params), vp, sz, vp, C.POINTER(Noise)]
        L.fpsk_localize.restype = C.c_int
        L.fpsk_localize.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, C.c_int, u64, i32, C.POINTER(Params),
                                    vp, sz, vp, C.POINTER(Fault), i32, C.POINTER(i32)]
        L.fpsk_repair_workspace_bytes.restype = sz
        L.fpsk_repair_workspace_bytes.argtypes = [i64, i64, i64, i32, C.POINTER(Params)]
        L.fpsk_verify_repair.restype = C.c_int
        L.fpsk_verify_repair.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, C.c_int, u64, i32, C.POINTER(Params),
                                         vp, sz, vp, C.POINTER(Fault), i32, C.POINTER(RepairReport)]
        L.fpsk_apply_corrections.restype = C.c_int
        L.fpsk_apply_corrections.argtypes = [vp, i64, i64, i64, C.POINTER(Fault), i32, vp, sz, vp]
        L.fpsk_selftest_bounded_wait.restype = C.c_int
        L.fpsk_selftest_bounded_wait.argtypes = [vp, vp, vp]
        L.fpsk_launch_count.restype = u64
        L.fpsk_launch_count.argtypes = []
        L.fpsk_lazy_resource_count.restype = u64
        L.fpsk_lazy_resource_count.argtypes = []
        L.fpsk_debug_bounds_report.restype = i32
        L.fpsk_debug_bounds_report.argtypes = [C.POINTER(i64), C.POINTER(i32), C.POINTER(i64), C.POINTER(i64), C.c_char_p, sz]
        L.fpsk_debug_bounds_clear.restype = C.c_int
        L.fpsk_debug_bounds_clear.argtypes = []
        L.fpsk_context_create.restype = C.c_int
        L.fpsk_context_create.argtypes = [C.POINTER(vp)]
        L.fpsk_context_destroy.restype = C.c_int
        L.fpsk_context_destroy.argtypes = [vp]
        _lib = L
    return _lib


def status_string(s: int) -> str:
    return lib().fpsk_status_string(int(s)).decode()


def default_params(**kw) -> Params:
    p = Params()
    lib().fpsk_default_params(C.byref(p))
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def launch_count() -> int:
    return int(lib().fpsk_launch_count())


def debug_bounds_report():
    """(built_with_checks, violations, line, index, limit, source file) of the loaded library."""
    v, ln, ix, lm = C.c_int64(-1), C.c_int32(0), C.c_int64(0), C.c_int64(0)
    buf = C.create_string_buffer(256)
    rc = lib().fpsk_debug_bounds_report(C.byref(v), C.byref(ln), C.byref(ix), C.byref(lm), buf, 256)
    return int(rc), int(v.value), int(ln.value), int(ix.value), int(lm.value), buf.value.decode()


def lazy_resource_count() -> int:
    return int(lib().fpsk_lazy_resource_count())


class Context:
    """Caller-owned host resources (auxiliary streams, events, pinned buffer) of fpsk_measure_noise,
    fpsk_localize and fpsk_verify_repair: put `ctx.ptr` into Params.context.  One call at a time."""

    def __init__(self):
        h = C.c_void_p()
        rc = lib().fpsk_context_create(C.byref(h))
        if rc != STATUS_OK:
            raise FpskError(rc, "fpsk_context_create")
        self.ptr = h.value

    def close(self):
        if self.ptr:
            rc = lib().fpsk_context_destroy(self.ptr)
            self.ptr = None
            if rc != STATUS_OK:
                raise FpskError(rc, "fpsk_context_destroy")

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


def dtype_of(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return FP16
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"operands must be float16 or bfloat16, got {t.dtype}")


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _mat_args(A: torch.Tensor, B: torch.Tensor, Cm: torch.Tensor, b_transposed: bool = False):
    """(A, lda, B, ldb, C, ldc, m, k, n, dtype); with b_transposed, B is the weight W = B^T of shape (n, k)."""
    assert A.is_cuda and B.is_cuda and Cm.is_cuda, "A, B, C must be device tensors"
    assert A.dim() == 2 and B.dim() == 2 and Cm.dim() == 2
    assert A.stride(1) == 1 and B.stride(1) == 1 and Cm.stride(1) == 1, "row-major (unit column stride) required"
    m, k = A.shape
    if b_transposed:
        n, k2 = B.shape
    else:
        k2, n = B.shape
    assert k2 == k and tuple(Cm.shape) == (m, n) and A.dtype == B.dtype
    brows, bcols = B.shape
    return (A.data_ptr(), A.stride(0) if m > 1 else max(k, A.stride(0)), B.data_ptr(),
            B.stride(0) if brows > 1 else max(bcols, B.stride(0)), Cm.data_ptr(),
            Cm.stride(0) if m > 1 else max(n, Cm.stride(0)), m, k, n, dtype_of(A))


def law_m_start(m: int, k: int, n: int, dtype: int, params: Optional[Params] = None) -> int:
    return int(lib().fpsk_law_m_start(m, k, n, dtype, C.byref(params) if params is not None else None))


def plan(m: int, k: int, n: int, dtype: int, sigma_hat: float, rms_c: float, m_cur: int,
         params: Optional[Params] = None) -> Tuple[int, int, float]:
    ml, r, B = C.c_int32(), C.c_int32(), C.c_double()
    rc = lib().fpsk_plan(m, k, n, dtype, sigma_hat, rms_c, m_cur, C.byref(params) if params is not None else None,
                         C.byref(ml), C.byref(r), C.byref(B))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_plan")
    return ml.value, r.value, B.value


def probe_workspace(m: int, k: int, n: int, device=None, stream=None) -> torch.Tensor:
    """Allocate and prepare a probe workspace (torch owns the memory)."""
    nbytes = int(lib().fpsk_probe_workspace_bytes(m, k, n))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")
    rc = lib().fpsk_probe_init(ws.data_ptr(), nbytes, _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_init")
    return ws


def probe(A, B, Cm, workspace: torch.Tensor, result: torch.Tensor, residual: Optional[torch.Tensor] = None,
          params: Optional[Params] = None, stream=None, c_is_fp32: Optional[bool] = None) -> None:
    """Asynchronous probe; `result` is a device uint8 tensor of sizeof(ProbeResult) bytes."""
    a = _mat_args(A, B, Cm)
    if c_is_fp32 is None:
        c_is_fp32 = Cm.dtype == torch.float32
    rc = lib().fpsk_probe(a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7], a[8], a[9], 1 if c_is_fp32 else 0,
                          C.byref(params) if params is not None else None, workspace.data_ptr(), workspace.numel(),
                          _stream_ptr(stream), result.data_ptr(), residual.data_ptr() if residual is not None else None)
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe")


PROBE_STATIC_SCRATCH_BYTES = 12 << 20


def probe_static(A, B, Cm, result: torch.Tensor, residual: Optional[torch.Tensor] = None,
                 params: Optional[Params] = None, stream=None) -> None:
    """The probe for callers that cannot allocate device memory (no workspace argument: the
    scratch is a fixed array inside the library).  Same outputs as `probe`.  Calls sharing a
    device must not overlap on the GPU."""
    a = _mat_args(A, B, Cm)
    rc = lib().fpsk_probe_static(a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7], a[8], a[9],
                                 1 if Cm.dtype == torch.float32 else 0,
                                 C.byref(params) if params is not None else None, _stream_ptr(stream),
                                 result.data_ptr(), residual.data_ptr() if residual is not None else None)
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_static")


class _ShapeOnly:
    """Stands in for a k x n operand in the argument checks when the caller holds its transpose."""

    def __init__(self, W: torch.Tensor, k: int, n: int):
        self.is_cuda, self.dtype, self.shape, self._W = W.is_cuda, W.dtype, (k, n), W

    def dim(self):
        return 2

    def stride(self, d):
        return 1 if d == 1 else self.shape[1]

    def data_ptr(self):
        return self._W.data_ptr()


class HashedProbe:
    """Buffers of the S only probe with a cached B side: the host record, the device cache and the
    per-call workspace (torch owns the memory).  ``__call__`` is one asynchronous probe."""

    def __init__(self, m: int, k: int, n: int, n_buckets: int, seed: int, rnd: int = 0, device=None, stream=None,
                 b_transposed: bool = False):
        """b_transposed: the B argument of the calls is the weight W = B^T (n x k, row-major): C = A W^T."""
        self.shape = (m, k, n)
        self.n_buckets, self.seed, self.round = n_buckets, seed, rnd
        cb = int(lib().fpsk_probe_hashed_cache_bytes(m, k, n, n_buckets))
        wb = int(lib().fpsk_probe_hashed_workspace_bytes(m, k, n, n_buckets))
        if cb == 0 or wb == 0:
            raise FpskError(ERR_SHAPE, "fpsk_probe_hashed_cache_bytes")
        self.cache = torch.empty(cb, dtype=torch.uint8, device=device or "cuda")
        self.ws = torch.empty(wb, dtype=torch.uint8, device=device or "cuda")
        rc = lib().fpsk_probe_init(self.ws.data_ptr(), wb, _stream_ptr(stream))
        if rc != STATUS_OK:
            raise FpskError(rc, "fpsk_probe_init")
        self.side = BSide()
        self.side.b_transposed = 1 if b_transposed else 0

    def matches(self, B: torch.Tensor, b_version: int) -> bool:
        m, k, n = self.shape
        if self.side.b_transposed:
            ldb = B.stride(0) if n > 1 else max(k, B.stride(0))
        else:
            ldb = B.stride(0) if k > 1 else max(n, B.stride(0))
        return bool(lib().fpsk_bside_matches(C.byref(self.side), B.data_ptr(), ldb, b_version, m, k, n, dtype_of(B),
                                             self.seed, self.round, self.n_buckets, self.cache.data_ptr()))

    def __call__(self, A, B, Cm, result: torch.Tensor, b_version: int = 0, S: Optional[torch.Tensor] = None,
                 params: Optional[Params] = None, stream=None, c_is_fp32: Optional[bool] = None,
                 state: Optional[torch.Tensor] = None) -> None:
        if self.side.b_transposed:
            # B is the weight W (n x k): marshal A and C as usual, W with its own leading dimension
            m, k, n = self.shape
            assert B.is_cuda and B.dim() == 2 and B.stride(1) == 1 and tuple(B.shape) == (n, k) and B.dtype == A.dtype
            a = list(_mat_args(A, _ShapeOnly(B, k, n), Cm))
            a[2], a[3] = B.data_ptr(), (B.stride(0) if n > 1 else max(k, B.stride(0)))
        else:
            a = _mat_args(A, B, Cm)
        assert (a[6], a[7], a[8]) == self.shape
        if c_is_fp32 is None:
            c_is_fp32 = Cm.dtype == torch.float32
        rc = lib().fpsk_probe_hashed(C.byref(self.side), a[0], a[1], a[2], a[3], b_version, a[4], a[5], a[6], a[7],
                                     a[8], a[9], 1 if c_is_fp32 else 0, self.seed, self.round, self.n_buckets,
                                     C.byref(params) if params is not None else None, self.cache.data_ptr(),
                                     self.cache.numel(), self.ws.data_ptr(), self.ws.numel(), _stream_ptr(stream),
                                     result.data_ptr(), S.data_ptr() if S is not None else None,
                                     state.data_ptr() if state is not None else None)
        if rc != STATUS_OK:
            raise FpskError(rc, "fpsk_probe_hashed")


def new_probe_state(device=None, stream=None) -> torch.Tensor:
    """A zeroed fpsk_probe_state in device memory (uint8 tensor of 32 bytes)."""
    st = torch.empty(C.sizeof(ProbeState), dtype=torch.uint8, device=device or "cuda")
    rc = lib().fpsk_probe_state_reset(st.data_ptr(), _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_state_reset")
    return st


def reset_probe_state(state: torch.Tensor, stream=None) -> None:
    rc = lib().fpsk_probe_state_reset(state.data_ptr(), _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_state_reset")


def read_probe_state(state: torch.Tensor) -> ProbeState:
    """Synchronising read of the state (the once-per-step host read)."""
    host = state.cpu().numpy().tobytes()
    return ProbeState.from_buffer_copy(host)


def probe_accumulate(result: torch.Tensor, state: torch.Tensor, stream=None) -> None:
    rc = lib().fpsk_probe_accumulate(result.data_ptr(), state.data_ptr(), _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_accumulate")


def selftest_bounded_wait(flag: torch.Tensor, result: torch.Tensor, stream=None) -> None:
    """Launch the wait self-test on a 4-byte device flag; read the status with read_probe_result."""
    rc = lib().fpsk_selftest_bounded_wait(flag.data_ptr(), result.data_ptr(), _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_selftest_bounded_wait")


def recalibration_due(calls: int) -> bool:
    return bool(lib().fpsk_recalibration_due(calls))


def probe_recalibrate(m: int, n: int, sigma_bar: float, rms_c: float, n_buckets: int,
                      params: Optional[Params] = None) -> Tuple[int, bool]:
    mn, rb = C.c_int32(), C.c_int32()
    rc = lib().fpsk_probe_recalibrate(m, n, sigma_bar, rms_c, n_buckets, C.byref(params) if params is not None else None,
                                      C.byref(mn), C.byref(rb))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_recalibrate")
    return mn.value, bool(rb.value)


def new_probe_result(device=None) -> torch.Tensor:
    return torch.zeros(C.sizeof(ProbeResult), dtype=torch.uint8, device=device or "cuda")


def read_probe_result(result: torch.Tensor) -> ProbeResult:
    """Synchronising read of a device verdict."""
    host = result.cpu().numpy().tobytes()
    return ProbeResult.from_buffer_copy(host)


def probe_host(hA: torch.Tensor, hB: torch.Tensor, hC: torch.Tensor, workspace: torch.Tensor,
               params: Optional[Params] = None, stream=None) -> ProbeResult:
    """Probe of operands that live in (pinned) host memory; returns the verdict on the host."""
    assert not hA.is_cuda and not hB.is_cuda and not hC.is_cuda
    assert hA.is_contiguous() and hB.is_contiguous() and hC.is_contiguous() and hC.dtype == torch.float32
    m, k = hA.shape
    n = hB.shape[1]
    res = ProbeResult()
    rc = lib().fpsk_probe_host(hA.data_ptr(), hB.data_ptr(), hC.data_ptr(), m, k, n, dtype_of(hA),
                               C.byref(params) if params is not None else None, workspace.data_ptr(),
                               workspace.numel(), _stream_ptr(stream), C.byref(res))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_host")
    return res


def probe_host_workspace(m: int, k: int, n: int, device=None, stream=None) -> torch.Tensor:
    nbytes = int(lib().fpsk_probe_host_workspace_bytes(m, k, n))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")
    rc = lib().fpsk_probe_init(ws.data_ptr(), nbytes, _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_probe_init")
    return ws


def hash_tables(seed: int, rnd: int, side: int, count: int, n_buckets: int, device=None, stream=None):
    b = torch.empty(count, dtype=torch.int32, device=device or "cuda")
    s = torch.empty(count, dtype=torch.int32, device=device or "cuda")
    rc = lib().fpsk_hash_tables(seed, rnd, side, count, n_buckets, b.data_ptr(), s.data_ptr(), _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_hash_tables")
    return b, s


def workspace(m: int, k: int, n: int, n_buckets: int, params: Optional[Params] = None, device=None) -> torch.Tensor:
    nbytes = int(lib().fpsk_workspace_bytes(m, k, n, n_buckets, C.byref(params) if params is not None else None))
    if nbytes == 0:
        raise FpskError(ERR_BUCKETS, "fpsk_workspace_bytes")
    return torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")


def max_buckets(m: int, k: int, n: int) -> int:
    return int(lib().fpsk_max_buckets(m, k, n))


def sketches(A, B, Cm, seed: int, rnd: int, n_buckets: int, ws: torch.Tensor, moments: bool = True, stream=None,
             params: Optional[Params] = None):
    """With params.b_transposed = 1, B is the weight W = B^T of shape (n, k) (C = A W^T)."""
    a = _mat_args(A, B, Cm, bool(params is not None and params.b_transposed))
    S = torch.empty((n_buckets, n_buckets), dtype=torch.float32, device=A.device)
    R = torch.empty_like(S) if moments else None
    T = torch.empty_like(S) if moments else None
    rc = lib().fpsk_sketches(a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7], a[8], a[9], seed, rnd, n_buckets,
                             C.byref(params) if params is not None else None,
                             ws.data_ptr(), ws.numel(), _stream_ptr(stream), S.data_ptr(),
                             R.data_ptr() if moments else None, T.data_ptr() if moments else None)
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_sketches")
    return S, R, T


def measure_noise(A, B, Cm, seed: int, ws: torch.Tensor, m0: int = 0, params: Optional[Params] = None,
                  stream=None) -> Noise:
    """With params.b_transposed = 1, B is the weight W = B^T of shape (n, k) (C = A W^T)."""
    a = _mat_args(A, B, Cm, bool(params is not None and params.b_transposed))
    out = Noise()
    rc = lib().fpsk_measure_noise(a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7], a[8], a[9], seed, m0,
                                  C.byref(params) if params is not None else None, ws.data_ptr(), ws.numel(),
                                  _stream_ptr(stream), C.byref(out))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_measure_noise")
    return out


def localize(A, B, Cm, seed: int, n_buckets: int, ws: torch.Tensor, params: Optional[Params] = None,
             capacity: int = 1024, stream=None) -> List[Fault]:
    """With params.b_transposed = 1, B is the weight W = B^T of shape (n, k) (C = A W^T)."""
    a = _mat_args(A, B, Cm, bool(params is not None and params.b_transposed))
    buf = (Fault * capacity)()
    cnt = C.c_int32(0)
    rc = lib().fpsk_localize(a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7], a[8], a[9], seed, n_buckets,
                             C.byref(params) if params is not None else None, ws.data_ptr(), ws.numel(),
                             _stream_ptr(stream), buf, capacity, C.byref(cnt))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_localize")
    return [buf[i] for i in range(cnt.value)]


def repair_workspace(m: int, k: int, n: int, n_buckets: int = 0, params: Optional[Params] = None, device=None) -> torch.Tensor:
    nbytes = int(lib().fpsk_repair_workspace_bytes(m, k, n, n_buckets, C.byref(params) if params is not None else None))
    if nbytes == 0:
        raise FpskError(ERR_BUCKETS, "fpsk_repair_workspace_bytes")
    return torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")


def verify_repair(A, B, Cm, seed: int, ws: torch.Tensor, n_buckets: int = 0, params: Optional[Params] = None,
                  capacity: int = 1024, stream=None):
    """Algorithm 2 in place on Cm (device FP32): returns (faults, report)."""
    a = _mat_args(A, B, Cm)
    assert Cm.dtype == torch.float32
    buf = (Fault * capacity)()
    rep = RepairReport()
    rc = lib().fpsk_verify_repair(a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7], a[8], a[9], seed, n_buckets,
                                  C.byref(params) if params is not None else None, ws.data_ptr(), ws.numel(),
                                  _stream_ptr(stream), buf, capacity, C.byref(rep))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_verify_repair")
    return [buf[i] for i in range(min(rep.n_faults, capacity))], rep


def apply_corrections(Cm: torch.Tensor, faults, ws: torch.Tensor, stream=None) -> None:
    n = len(faults)
    buf = (Fault * max(n, 1))(*faults)
    m, ncol = Cm.shape
    rc = lib().fpsk_apply_corrections(Cm.data_ptr(), Cm.stride(0), m, ncol, buf, n, ws.data_ptr(), ws.numel(),
                                      _stream_ptr(stream))
    if rc != STATUS_OK:
        raise FpskError(rc, "fpsk_apply_corrections")

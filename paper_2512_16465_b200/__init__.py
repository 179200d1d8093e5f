"""Python binding of the b200 GEMM C-ABI library (``include/gemm.h``).

Argument marshalling only: every step of ``D = act(alpha * op(A) @ op(B) + beta * C + bias)``
runs in the CUDA kernels of ``libb200gemm.so``.  PyTorch is used for device memory and
streams.  There is no CPU or library fallback: if the shared library cannot be loaded
the import raises.

Low-level calls mirror the C names: :func:`gemm_plan`, :func:`gemm_workspace_bytes`,
:func:`gemm_run`, :func:`gemm_plan_status`, :func:`gemm_plan_info`, :func:`gemm_destroy`.
:class:`Plan` wraps them for torch tensors.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

from . import build as _build

BF16, F16, F32, FP8_E4M3, FP8_E5M2 = 0, 1, 2, 3, 4
OP_N, OP_T = 0, 1
(EPI_NONE, EPI_BIAS, EPI_RELU, EPI_BIAS_RELU, EPI_GELU_ERF, EPI_BIAS_GELU_ERF, EPI_GELU_TANH, EPI_BIAS_GELU_TANH,
 EPI_SILU, EPI_BIAS_SILU) = range(10)
STRUCT_B_LOWER, STRUCT_B_UPPER, STRUCT_D_MIRROR = 0x1, 0x2, 0x4     # gemm_desc_t.structure
OPT_STREAMK_WORKSPACE = 0x1                                          # gemm_desc_t.options
VARIANT_AUTO, VARIANT_DENSE_1CTA, VARIANT_DENSE_2CTA, VARIANT_SKINNY_STREAMK, VARIANT_DENSE_2CTA_WIDE = 0, 1, 2, 3, 4
REGIME_NAMES = {0: "memory-bound", 1: "middle-zone", 2: "compute-bound"}
FLAG_DEBUG_STALL = 0x80000000

OK, ERR_NULL, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = range(9)


class GemmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = _lib.gemm_last_cuda_error().decode() if status in (ERR_CUDA, ERR_TIMEOUT) else ""
        super().__init__(f"{where}: {_lib.gemm_status_string(status).decode()}" + (f" ({detail})" if detail else ""))


class Desc(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("transa", ctypes.c_int32), ("transb", ctypes.c_int32),
                ("ab_dtype", ctypes.c_int32), ("c_dtype", ctypes.c_int32),
                ("lda", ctypes.c_int64), ("ldb", ctypes.c_int64), ("ldc", ctypes.c_int64),
                ("batch_count", ctypes.c_int32), ("epilogue", ctypes.c_int32),
                ("stride_a", ctypes.c_int64), ("stride_b", ctypes.c_int64), ("stride_c", ctypes.c_int64),
                ("structure", ctypes.c_uint32), ("options", ctypes.c_uint32)]


class Info(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("variant", ctypes.c_int32), ("regime", ctypes.c_int32),
                ("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32), ("tile_k", ctypes.c_int32),
                ("stages", ctypes.c_int32), ("cluster_size", ctypes.c_int32), ("grid", ctypes.c_int32),
                ("raster_group", ctypes.c_int32), ("split", ctypes.c_int32), ("smem_bytes", ctypes.c_int32),
                ("num_tiles", ctypes.c_int64), ("flops", ctypes.c_double), ("min_bytes", ctypes.c_double),
                ("intensity", ctypes.c_double), ("workspace_bytes", ctypes.c_size_t)]

    def as_dict(self) -> dict:
        return {k: getattr(self, k) for k, _ in self._fields_ if k != "struct_size"}


class WorkItem(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in ("cta", "batch", "tile_row", "tile_col", "k_begin", "k_end", "slice", "reserved")]


TUNE_MAX_CANDIDATES = 32


class TuneReport(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("candidates_tried", ctypes.c_int32), ("candidates_skipped", ctypes.c_int32),
                ("best_flags", ctypes.c_uint32), ("best_ms", ctypes.c_float), ("auto_ms", ctypes.c_float),
                ("tried_flags", ctypes.c_uint32 * TUNE_MAX_CANDIDATES), ("tried_ms", ctypes.c_float * TUNE_MAX_CANDIDATES)]

    def as_dict(self) -> dict:
        n = self.candidates_tried
        return {"candidates_tried": n, "candidates_skipped": self.candidates_skipped, "best_flags": self.best_flags,
                "best_ms": self.best_ms, "auto_ms": self.auto_ms,
                "tried": [(self.tried_flags[i], self.tried_ms[i]) for i in range(n)]}


EXPORTS = ("gemm_plan", "gemm_workspace_bytes", "gemm_run", "gemm_plan_status", "gemm_plan_status_async",
           "gemm_plan_status_result", "gemm_plan_status_stream", "gemm_plan_schedule", "gemm_plan_set_timeout_ms",
           "gemm_plan_info", "gemm_destroy", "gemm_status_string", "gemm_last_cuda_error", "gemm_skinny_run_noalloc",
           "gemm_tune", "gemm_tune_workspace_bytes", "gemm_tune_cache_clear", "gemm_tune_cache_save", "gemm_tune_cache_load",
           "gemm_host_create", "gemm_host_run", "gemm_host_panels", "gemm_host_destroy")


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        path = _build.build()          # raises if nvcc is missing or compilation fails
    L = ctypes.CDLL(path)
    vp = ctypes.c_void_p
    L.gemm_plan.restype = ctypes.c_int
    L.gemm_plan.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(vp)]
    L.gemm_workspace_bytes.restype = ctypes.c_size_t
    L.gemm_workspace_bytes.argtypes = [vp]
    L.gemm_run.restype = ctypes.c_int
    L.gemm_run.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, ctypes.c_size_t, vp]
    L.gemm_plan_status.restype = ctypes.c_int
    L.gemm_plan_status.argtypes = [vp]
    L.gemm_plan_status_result.restype = ctypes.c_int
    L.gemm_plan_status_result.argtypes = [vp]
    for fn in (L.gemm_plan_status_async, L.gemm_plan_status_stream):
        fn.restype = ctypes.c_int
        fn.argtypes = [vp, vp]
    L.gemm_plan_schedule.restype = ctypes.c_int
    L.gemm_plan_schedule.argtypes = [vp, ctypes.POINTER(WorkItem), ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
    L.gemm_plan_set_timeout_ms.restype = ctypes.c_int
    L.gemm_plan_set_timeout_ms.argtypes = [vp, ctypes.c_uint32]
    L.gemm_plan_info.restype = ctypes.c_int
    L.gemm_plan_info.argtypes = [vp, ctypes.POINTER(Info)]
    L.gemm_destroy.restype = ctypes.c_int
    L.gemm_destroy.argtypes = [vp]
    L.gemm_status_string.restype = ctypes.c_char_p
    L.gemm_status_string.argtypes = [ctypes.c_int]
    L.gemm_last_cuda_error.restype = ctypes.c_char_p
    L.gemm_last_cuda_error.argtypes = []
    L.gemm_skinny_run_noalloc.restype = ctypes.c_int
    L.gemm_skinny_run_noalloc.argtypes = [ctypes.POINTER(Desc), vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, ctypes.c_int]
    L.gemm_tune.restype = ctypes.c_int
    L.gemm_tune.argtypes = [ctypes.POINTER(Desc), vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, ctypes.c_size_t, vp,
                            ctypes.c_int, ctypes.POINTER(vp), ctypes.POINTER(TuneReport)]
    L.gemm_tune_workspace_bytes.restype = ctypes.c_size_t
    L.gemm_tune_workspace_bytes.argtypes = [ctypes.POINTER(Desc)]
    L.gemm_tune_cache_clear.restype = None
    L.gemm_tune_cache_clear.argtypes = []
    for fn in (L.gemm_tune_cache_save, L.gemm_tune_cache_load):
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.c_char_p, ctypes.POINTER(ctypes.c_int)]
    L.gemm_host_create.restype = ctypes.c_int
    L.gemm_host_create.argtypes = [ctypes.POINTER(Desc), ctypes.c_int, ctypes.POINTER(vp)]
    L.gemm_host_run.restype = ctypes.c_int
    L.gemm_host_run.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float]
    L.gemm_host_panels.restype = ctypes.c_int
    L.gemm_host_panels.argtypes = [vp]
    L.gemm_host_destroy.restype = ctypes.c_int
    L.gemm_host_destroy.argtypes = [vp]
    return L


_lib = _load()
LIB_PATH = _build.LIB


def make_flags(variant: int = 0, tile_n: int = 0, raster: int = 0, stages: int = 0, debug_stall: bool = False,
               kslices: int = 0, l2_hints: bool = False, no_k_serpentine: bool = False, no_early_launch: bool = False,
               bias_per_row: bool = False, a_lower: bool = False, a_upper: bool = False,
               tail_split: bool = False, d_lower: bool = False, d_upper: bool = False) -> int:
    """Pack the GEMM_FLAG_* fields of ``gemm_desc_t.flags`` (0 everywhere = automatic)."""
    assert tile_n % 16 == 0 and (tile_n <= 256 or (tile_n % 64 == 0 and tile_n <= 512))
    tile_field = tile_n // 16 if tile_n <= 256 else 16 + (tile_n - 256) // 64   # 17 ... 20: the wide tiles 320 ... 512
    return ((variant & 0xF) << 4) | ((tile_field & 0x1F) << 8) | ((raster & 0x7F) << 16) | ((stages & 0xF) << 24) | \
        ((kslices & 0x3) << 28) | (0x40000000 if l2_hints else 0) | (0x8 if no_k_serpentine else 0) | \
        (FLAG_DEBUG_STALL if debug_stall else 0) | (0x4 if no_early_launch else 0) | (0x1 if bias_per_row else 0) | (0x2 if a_lower else 0) | (0x800000 if a_upper else 0) | (0x2000 if tail_split else 0) | \
        (0x4000 if d_lower else 0) | (0x8000 if d_upper else 0)


def make_desc(M, N, K, transa=OP_N, transb=OP_T, ab_dtype=BF16, c_dtype=F32, lda=0, ldb=0, ldc=0, batch=1,
              stride_a=0, stride_b=0, stride_c=0, epilogue=EPI_NONE, flags=0, structure=0, options=0) -> Desc:
    """Build a ``gemm_desc_t``; zero leading dimensions / strides mean "tight"; ``structure`` takes ``STRUCT_*`` bits,
    ``options`` ``OPT_*`` bits."""
    lda = lda or (M if transa else K)
    ldb = ldb or (K if transb else N)
    ldc = ldc or N
    stride_a = stride_a or (K if transa else M) * lda
    stride_b = stride_b or (N if transb else K) * ldb
    stride_c = stride_c or M * ldc
    return Desc(ctypes.sizeof(Desc), flags, M, N, K, transa, transb, ab_dtype, c_dtype, lda, ldb, ldc, batch, epilogue,
                stride_a, stride_b, stride_c, structure, options)


# ----------------------------------------------------------------------- C-named calls

def gemm_plan(desc: Desc) -> int:
    """``gemm_plan``: returns the opaque plan handle or raises :class:`GemmError`."""
    h = ctypes.c_void_p()
    st = _lib.gemm_plan(ctypes.byref(desc), ctypes.byref(h))
    if st != OK:
        raise GemmError(st, "gemm_plan")
    return h.value


def gemm_workspace_bytes(plan: int) -> int:
    return int(_lib.gemm_workspace_bytes(plan))


def gemm_run(plan: int, A: int, B: int, C: int, bias: int, alpha: float, beta: float, workspace: int,
             workspace_bytes: int, stream: int) -> None:
    """``gemm_run`` on raw device addresses (ints) and a raw ``cudaStream_t`` value."""
    st = _lib.gemm_run(plan, A, B, C, bias or None, alpha, beta, workspace or None, workspace_bytes, stream or None)
    if st != OK:
        raise GemmError(st, "gemm_run")


def gemm_skinny_run_noalloc(desc: Desc, A: int, B: int, C: int, bias: int, alpha: float, beta: float, stream: int,
                            sync_and_check: bool = False) -> None:
    """``gemm_skinny_run_noalloc``: the skinny stream-K GEMM for callers that may not allocate device memory
    (no plan, no workspace; the scratch is a fixed array inside the library).  Raw device addresses and a raw
    ``cudaStream_t`` value; raises :class:`GemmError`, e.g. ``ERR_WORKSPACE`` when the problem is too large for
    the built-in scratch.  Calls that overlap on the GPU race on that scratch: keep them on one stream."""
    st = _lib.gemm_skinny_run_noalloc(ctypes.byref(desc), A, B, C, bias or None, alpha, beta, stream or None,
                                      1 if sync_and_check else 0)
    if st != OK:
        err = GemmError(st, "gemm_skinny_run_noalloc")
        if st == ERR_WORKSPACE:   # the library recorded how much scratch the problem wanted
            err.args = (f"{err.args[0]} ({_lib.gemm_last_cuda_error().decode()})",)
        raise err


def gemm_tune_workspace_bytes(desc: Desc) -> int:
    return int(_lib.gemm_tune_workspace_bytes(ctypes.byref(desc)))


def gemm_tune(desc: Desc, A: int, B: int, C: int, bias: int, alpha: float, beta: float, workspace: int, workspace_bytes: int,
              stream: int, iterations: int = 10):
    """``gemm_tune``: time the plausible plans of ``desc`` on the given device buffers (C is overwritten repeatedly) and
    return ``(plan handle of the fastest, report dict)``.  The choice is remembered for later ``gemm_plan`` calls."""
    h = ctypes.c_void_p()
    rep = TuneReport()
    rep.struct_size = ctypes.sizeof(TuneReport)
    st = _lib.gemm_tune(ctypes.byref(desc), A, B, C, bias or None, alpha, beta, workspace or None, workspace_bytes, stream or None,
                        iterations, ctypes.byref(h), ctypes.byref(rep))
    if st != OK:
        raise GemmError(st, "gemm_tune")
    return h.value, rep.as_dict()


def gemm_tune_cache_clear() -> None:
    _lib.gemm_tune_cache_clear()


def gemm_tune_cache_save(path: str) -> int:
    """``gemm_tune_cache_save``: write the current device's remembered tuning results to ``path``; returns how many."""
    n = ctypes.c_int(0)
    st = _lib.gemm_tune_cache_save(os.fsencode(path), ctypes.byref(n))
    if st != OK:
        raise GemmError(st, "gemm_tune_cache_save")
    return n.value


def gemm_tune_cache_load(path: str) -> int:
    """``gemm_tune_cache_load``: add the results in ``path`` to the current device's; returns how many were read."""
    n = ctypes.c_int(0)
    st = _lib.gemm_tune_cache_load(os.fsencode(path), ctypes.byref(n))
    if st != OK:
        raise GemmError(st, "gemm_tune_cache_load")
    return n.value


def gemm_host_create(desc: Desc, panels: int = 0) -> int:
    """``gemm_host_create``: a handle for GEMMs whose operands live in host memory (row panels pipelined over three streams)."""
    h = ctypes.c_void_p()
    st = _lib.gemm_host_create(ctypes.byref(desc), panels, ctypes.byref(h))
    if st != OK:
        raise GemmError(st, "gemm_host_create")
    return h.value


def gemm_host_run(handle: int, hA: int, hB: int, hC: int, hbias: int, alpha: float, beta: float) -> None:
    """``gemm_host_run`` on raw HOST addresses; returns when D is complete in the host C buffer."""
    st = _lib.gemm_host_run(handle, hA, hB, hC, hbias or None, alpha, beta)
    if st != OK:
        raise GemmError(st, "gemm_host_run")


def gemm_host_panels(handle: int) -> int:
    return int(_lib.gemm_host_panels(handle))


def gemm_host_destroy(handle: int) -> None:
    _lib.gemm_host_destroy(handle)


def gemm_plan_status(plan: int) -> int:
    """``gemm_plan_status``: waits for the whole device, then takes the plan's status word."""
    return int(_lib.gemm_plan_status(plan))


def gemm_plan_status_stream(plan: int, stream: int) -> int:
    """``gemm_plan_status_stream``: waits for ``stream`` (a raw ``cudaStream_t`` value) only."""
    return int(_lib.gemm_plan_status_stream(plan, stream or None))


def gemm_plan_status_async(plan: int, stream: int) -> None:
    """``gemm_plan_status_async``: enqueue the read of the status word on ``stream``; nothing is waited for."""
    st = _lib.gemm_plan_status_async(plan, stream or None)
    if st != OK:
        raise GemmError(st, "gemm_plan_status_async")


def gemm_plan_status_result(plan: int) -> int:
    """``gemm_plan_status_result``: the word the last ``gemm_plan_status_async`` took (the caller waited for the stream)."""
    return int(_lib.gemm_plan_status_result(plan))


def bind_run(plan: int, A: int, B: int, C: int, bias: int, alpha: float, beta: float, workspace: int, workspace_bytes: int,
             stream: int):
    """The arguments of one ``gemm_run`` call converted to their C types once: returns a function of no arguments
    that makes the call (and raises :class:`GemmError` on failure).  For loops that launch the same GEMM on the same
    buffers again and again, where converting ten Python values per call costs more than the launch."""
    vp = ctypes.c_void_p
    args = (vp(plan), vp(A), vp(B), vp(C), vp(bias or None), ctypes.c_float(alpha), ctypes.c_float(beta), vp(workspace or None),
            ctypes.c_size_t(workspace_bytes), vp(stream or None))
    fn = _lib.gemm_run

    def call():
        st = fn(*args)
        if st != OK:
            raise GemmError(st, "gemm_run")
    return call


def gemm_plan_schedule(plan: int):
    """``gemm_plan_schedule``: the plan's work items as a numpy array of shape (items, 7) with the columns
    cta, batch, tile_row, tile_col, k_begin, k_end, slice, in the order the CTAs execute them (needs no device)."""
    import numpy as np
    n = ctypes.c_size_t(0)
    st = _lib.gemm_plan_schedule(plan, None, 0, ctypes.byref(n))
    if st != OK:
        raise GemmError(st, "gemm_plan_schedule")
    buf = (WorkItem * max(1, n.value))()
    st = _lib.gemm_plan_schedule(plan, buf, n.value, ctypes.byref(n))
    if st != OK:
        raise GemmError(st, "gemm_plan_schedule")
    return np.frombuffer(buf, dtype=np.int32).reshape(-1, 8)[: n.value, :7].copy()


def gemm_plan_info(plan: int) -> dict:
    info = Info()
    info.struct_size = ctypes.sizeof(Info)
    st = _lib.gemm_plan_info(plan, ctypes.byref(info))
    if st != OK:
        raise GemmError(st, "gemm_plan_info")
    return info.as_dict()


def gemm_destroy(plan: int) -> None:
    _lib.gemm_destroy(plan)


def status_string(st: int) -> str:
    return _lib.gemm_status_string(st).decode()


# ----------------------------------------------------------------------- torch convenience

def _torch_dtype_code(t) -> int:
    import torch
    return {torch.bfloat16: BF16, torch.float16: F16, torch.float32: F32, torch.float8_e4m3fn: FP8_E4M3,
            torch.float8_e5m2: FP8_E5M2}[t]


def _operand_matches(t, code: int) -> bool:
    """8-bit float operands may also be handed over as plain bytes (``torch.uint8``)."""
    import torch
    if t == torch.uint8:
        return code in (FP8_E4M3, FP8_E5M2)
    return _torch_dtype_code(t) == code


class Plan:
    """A planned GEMM bound to torch tensors.  ``run`` enqueues on the current torch stream."""

    def __init__(self, desc: Desc, handle: Optional[int] = None):
        self.desc = desc
        self.handle = gemm_plan(desc) if handle is None else handle
        self.info = gemm_plan_info(self.handle)
        self.workspace_bytes = gemm_workspace_bytes(self.handle)
        self._ws = None

    @classmethod
    def tuned(cls, desc: Desc, A, B, C, bias=None, alpha: float = 1.0, beta: float = 0.0, iterations: int = 10):
        """Plan by measurement on these tensors (C is overwritten repeatedly); returns ``(Plan, report)``."""
        import torch
        nbytes = gemm_tune_workspace_bytes(desc)
        ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=A.device)
        s = torch.cuda.current_stream(A.device).cuda_stream
        h, rep = gemm_tune(desc, A.data_ptr(), B.data_ptr(), C.data_ptr(), 0 if bias is None else bias.data_ptr(), float(alpha),
                           float(beta), ws.data_ptr(), ws.numel(), s, iterations)
        return cls(desc, handle=h), rep

    def workspace(self, device=None):
        import torch
        if self._ws is None and self.workspace_bytes:
            self._ws = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=device or "cuda")
        return self._ws

    def run(self, A, B, C, bias=None, alpha: float = 1.0, beta: float = 0.0, workspace=None, stream: Optional[int] = None):
        import torch
        if not (A.is_cuda and B.is_cuda and C.is_cuda):
            raise ValueError("A, B and C must be CUDA tensors")
        if not _operand_matches(A.dtype, self.desc.ab_dtype) or not _operand_matches(B.dtype, self.desc.ab_dtype) or \
                _torch_dtype_code(C.dtype) != self.desc.c_dtype:
            raise ValueError("tensor dtypes do not match the plan")
        ws = workspace if workspace is not None else self.workspace(A.device)
        s = torch.cuda.current_stream(A.device).cuda_stream if stream is None else stream
        gemm_run(self.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), 0 if bias is None else bias.data_ptr(),
                 float(alpha), float(beta), 0 if ws is None else ws.data_ptr(), 0 if ws is None else ws.numel(), s)
        return C

    def status(self, stream: Optional[int] = None) -> int:
        """The plan's status after its runs on ``stream`` (default: the current torch stream); waits for that stream only."""
        import torch
        s = torch.cuda.current_stream().cuda_stream if stream is None else stream
        return gemm_plan_status_stream(self.handle, s)

    def set_timeout_ms(self, ms: int) -> None:
        _lib.gemm_plan_set_timeout_ms(self.handle, ms)

    def close(self):
        if self.handle:
            gemm_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

"""ctypes front end of the CPU oracle (``gemm_oracle.c``) -- test infrastructure only.

The oracle is the fp64 triple-loop definition of
``D = act(alpha * op(A) @ op(B) + beta * C + bias)`` (the GEMM of the paper's
Section 5.4 case study).  Nothing in the product package imports this module:
only the tests, the smoke check and the benchmark's CPU-baseline legs do.

Arrays are numpy: ``uint16`` bit patterns for bf16 / fp16, ``uint8`` for the 8-bit floats, ``float32`` for fp32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gemm_oracle.c")
_LIB = os.path.join(_HERE, "libgemm_oracle.so")

BF16, F16, F32, FP8_E4M3, FP8_E5M2 = 0, 1, 2, 3, 4
(EPI_NONE, EPI_BIAS, EPI_RELU, EPI_BIAS_RELU, EPI_GELU_ERF, EPI_BIAS_GELU_ERF, EPI_GELU_TANH, EPI_BIAS_GELU_TANH,
 EPI_SILU, EPI_BIAS_SILU) = range(10)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no -ffast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Desc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("transa", ctypes.c_int32), ("transb", ctypes.c_int32),
                ("ab_dtype", ctypes.c_int32), ("c_dtype", ctypes.c_int32),
                ("lda", ctypes.c_int64), ("ldb", ctypes.c_int64), ("ldc", ctypes.c_int64),
                ("stride_a", ctypes.c_int64), ("stride_b", ctypes.c_int64),
                ("stride_c", ctypes.c_int64),
                ("epilogue", ctypes.c_int32), ("bias_per_row", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.oracle_bf16_to_f64.restype = ctypes.c_double
        L.oracle_bf16_to_f64.argtypes = [ctypes.c_uint16]
        L.oracle_f16_to_f64.restype = ctypes.c_double
        L.oracle_f16_to_f64.argtypes = [ctypes.c_uint16]
        L.oracle_f64_to_bf16.restype = ctypes.c_uint16
        L.oracle_f64_to_bf16.argtypes = [ctypes.c_double]
        L.oracle_f64_to_f16.restype = ctypes.c_uint16
        L.oracle_f64_to_f16.argtypes = [ctypes.c_double]
        for name in ("oracle_e4m3_to_f64", "oracle_e5m2_to_f64"):
            getattr(L, name).restype = ctypes.c_double
            getattr(L, name).argtypes = [ctypes.c_uint8]
        L.oracle_gelu_erf.restype = ctypes.c_double
        L.oracle_gelu_erf.argtypes = [ctypes.c_double]
        L.oracle_gelu_erf_alt.restype = ctypes.c_double
        L.oracle_gelu_erf_alt.argtypes = [ctypes.c_double]
        for name in ("oracle_logistic", "oracle_silu", "oracle_gelu_tanh"):
            getattr(L, name).restype = ctypes.c_double
            getattr(L, name).argtypes = [ctypes.c_double]
        L.oracle_gemm.restype = ctypes.c_int
        L.oracle_gemm.argtypes = [ctypes.POINTER(_Desc), ctypes.c_void_p, ctypes.c_void_p,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float, ctypes.c_float,
                                  ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
                                  ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                  ctypes.c_int]
        L.oracle_round_to.restype = ctypes.c_int
        L.oracle_round_to.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_void_p]
        L.oracle_decode.restype = ctypes.c_int
        L.oracle_decode.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_void_p]
        L.oracle_max_threads.restype = ctypes.c_int
        _lib = L
    return _lib


@dataclass
class Problem:
    """Shape, layout and epilogue of one GEMM, in the row-major convention of the C header."""
    M: int
    N: int
    K: int
    transa: int = 0
    transb: int = 0
    ab_dtype: int = BF16
    c_dtype: int = F32
    lda: int = 0
    ldb: int = 0
    ldc: int = 0
    batch: int = 1
    stride_a: int = 0
    stride_b: int = 0
    stride_c: int = 0
    epilogue: int = EPI_NONE
    bias_per_row: bool = False   # bias has M entries, one per output row (default: N entries, one per column)

    def finalize(self) -> "Problem":
        if not self.lda:
            self.lda = self.M if self.transa else self.K
        if not self.ldb:
            self.ldb = self.K if self.transb else self.N
        if not self.ldc:
            self.ldc = self.N
        if not self.stride_a:
            self.stride_a = (self.K if self.transa else self.M) * self.lda
        if not self.stride_b:
            self.stride_b = (self.N if self.transb else self.K) * self.ldb
        if not self.stride_c:
            self.stride_c = self.M * self.ldc
        return self

    def _cdesc(self) -> _Desc:
        return _Desc(self.M, self.N, self.K, self.transa, self.transb, self.ab_dtype, self.c_dtype,
                     self.lda, self.ldb, self.ldc, self.stride_a, self.stride_b, self.stride_c,
                     self.epilogue, 1 if self.bias_per_row else 0)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def wanted(rows, cols, d_tri: int) -> np.ndarray:
    """Which outputs the triangular forms of the product define (the paper's symmetric operator case, Section 5.1):
    ``d_tri`` = 0 all of D, 1 the lower triangle (row >= column, diagonal included), 2 the upper (row <= column).
    Boolean array ``[len(rows), len(cols)]``; a wanted element's value is that of the plain product."""
    r = np.asarray(rows, np.int64)[:, None]
    c = np.asarray(cols, np.int64)[None, :]
    if d_tri == 1:
        return r >= c
    if d_tri == 2:
        return r <= c
    assert d_tri == 0
    return np.ones((r.shape[0], c.shape[1]), dtype=bool)


def gemm(p: Problem, A, B, C_in=None, bias=None, alpha=1.0, beta=0.0,
         batches=None, rows=None, cols=None, threads: int = 0):
    """Evaluate the definition on ``batches x rows x cols`` (default: everything).

    Returns ``(y, bound)``, fp64 arrays of shape ``[len(batches), len(rows), len(cols)]``:
    the unrounded result and the tolerance scale
    ``|alpha| sum|a||b| + |beta||C_in| + |bias|``.
    """
    p.finalize()
    batches = np.arange(p.batch, dtype=np.int64) if batches is None else np.ascontiguousarray(batches, np.int64)
    rows = np.arange(p.M, dtype=np.int64) if rows is None else np.ascontiguousarray(rows, np.int64)
    cols = np.arange(p.N, dtype=np.int64) if cols is None else np.ascontiguousarray(cols, np.int64)
    assert batches.size == 0 or (batches.min() >= 0 and batches.max() < p.batch)
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < p.M)
    assert cols.size == 0 or (cols.min() >= 0 and cols.max() < p.N)
    for arr in (A, B, C_in, bias):
        assert arr is None or arr.flags["C_CONTIGUOUS"]
    ab_np = np.uint8 if p.ab_dtype in (FP8_E4M3, FP8_E5M2) else np.uint16
    assert A.dtype == ab_np and B.dtype == ab_np
    if C_in is not None:
        assert C_in.dtype == (np.float32 if p.c_dtype == F32 else np.uint16)
    if bias is not None:
        assert bias.dtype == np.float32
    shape = (batches.size, rows.size, cols.size)
    y = np.empty(shape, np.float64)
    bound = np.empty(shape, np.float64)
    if y.size:
        d = p._cdesc()
        rc = lib().oracle_gemm(ctypes.byref(d), _ptr(A), _ptr(B), _ptr(C_in), _ptr(bias),
                               float(np.float32(alpha)), float(np.float32(beta)),
                               _ptr(batches), batches.size, _ptr(rows), rows.size,
                               _ptr(cols), cols.size, _ptr(y), _ptr(bound), threads)
        if rc != 0:
            raise ValueError("oracle_gemm rejected its arguments")
    return y, bound


def round_to(y: np.ndarray, dtype: int) -> np.ndarray:
    """RNE-round fp64 results to the bit patterns of ``dtype`` (uint16 or float32 array)."""
    y = np.ascontiguousarray(y, np.float64)
    out = np.empty(y.shape, np.float32 if dtype == F32 else np.uint16)
    if y.size:
        lib().oracle_round_to(_ptr(y), y.size, dtype, _ptr(out))
    return out


def decode(bits: np.ndarray, dtype: int) -> np.ndarray:
    """Exact fp64 value of every element of a bf16 / fp16 (uint16) or fp32 array."""
    bits = np.ascontiguousarray(bits)
    out = np.empty(bits.shape, np.float64)
    if bits.size:
        lib().oracle_decode(_ptr(bits), bits.size, dtype, _ptr(out))
    return out


def max_threads() -> int:
    return int(lib().oracle_max_threads())

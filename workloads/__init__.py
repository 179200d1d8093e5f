"""Seeded synthetic GEMM workloads: the five benchmark configurations, scaled-down
replicas of them for fast checks, and the index samplers used on the large ones.

This module is the only code shared by the oracle side and the CUDA side of a
test, and it only produces DATA: shapes, flags and seeded input buffers (numpy,
``uint16`` bit patterns for bf16 / fp16, ``float32`` otherwise).  It contains
none of the GEMM arithmetic and imports neither the oracle nor the CUDA package.

The configurations stand in for the GEMM problems of the public kernel
benchmark suite the paper evaluates on (Section 5.1 / 5.4): square,
LLM-projection with a fused epilogue, attention-score shaped batched, small, and
skinny memory-bound shapes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field, replace
from functools import lru_cache

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libworkloads_gen.so")

BF16, F16, F32, FP8_E4M3, FP8_E5M2 = 0, 1, 2, 3, 4
(EPI_NONE, EPI_BIAS, EPI_RELU, EPI_BIAS_RELU, EPI_GELU_ERF, EPI_BIAS_GELU_ERF, EPI_GELU_TANH, EPI_BIAS_GELU_TANH,
 EPI_SILU, EPI_BIAS_SILU) = range(10)
ELEM_BYTES = {BF16: 2, F16: 2, F32: 4, FP8_E4M3: 1, FP8_E5M2: 1}
TENSOR_A, TENSOR_B, TENSOR_C, TENSOR_BIAS = 1, 2, 3, 4
BASE_SEED = 0x5EED0000


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-std=gnu11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"],
                       check=True)
    return _LIB


_lib = None


def _gen():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u64, i64, dbl, vp, ci = ctypes.c_uint64, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        L.gen_uniform.argtypes = [u64, u64, i64, dbl, dbl, ci, vp]
        L.gen_normal.argtypes = [u64, u64, i64, dbl, dbl, ci, vp]
        L.gen_integer.argtypes = [u64, u64, i64, i64, i64, ci, vp]
        L.gen_encode.argtypes = [vp, i64, ci, vp]
        L.gen_hash.argtypes = [u64, u64, u64]
        L.gen_hash.restype = u64
        for f in (L.gen_uniform, L.gen_normal, L.gen_integer, L.gen_encode):
            f.restype = None
        _lib = L
    return _lib


def _alloc(n: int, dtype: int) -> np.ndarray:
    return np.empty(n, {F32: np.float32, FP8_E4M3: np.uint8, FP8_E5M2: np.uint8}.get(dtype, np.uint16))


def uniform(seed, tensor_id, n, lo, hi, dtype) -> np.ndarray:
    out = _alloc(n, dtype)
    _gen().gen_uniform(seed, tensor_id, n, lo, hi, dtype, out.ctypes.data)
    return out


def normal(seed, tensor_id, n, mean, std, dtype) -> np.ndarray:
    out = _alloc(n, dtype)
    _gen().gen_normal(seed, tensor_id, n, mean, std, dtype, out.ctypes.data)
    return out


def integer(seed, tensor_id, n, lo, hi, dtype) -> np.ndarray:
    out = _alloc(n, dtype)
    _gen().gen_integer(seed, tensor_id, n, lo, hi, dtype, out.ctypes.data)
    return out


def encode(values, dtype) -> np.ndarray:
    """Round float values to the bit patterns of ``dtype`` (hand-built test inputs)."""
    v = np.ascontiguousarray(values, np.float32)
    out = _alloc(v.size, dtype)
    _gen().gen_encode(v.ctypes.data, v.size, dtype, out.ctypes.data)
    return out.reshape(v.shape)


@dataclass
class Dist:
    """Value distribution of one tensor: kind in {'uniform','normal','integer'} and its two parameters."""
    kind: str
    p0: float
    p1: float


@dataclass
class Workload:
    name: str
    M: int
    N: int
    K: int
    transa: int = 0
    transb: int = 1
    ab_dtype: int = BF16
    c_dtype: int = F32
    batch: int = 1
    epilogue: int = EPI_NONE
    bias_per_row: bool = False   # the bias has M entries (one per output row) instead of N
    a_tri: int = 0               # structure of op(A): 0 dense, 1 lower triangular (zero for k > i), 2 upper (zero for k < i)
    b_tri: int = 0               # structure of op(B): 0 dense, 1 lower triangular (zero for k < j), 2 upper (zero for k > j)
    d_tri: int = 0               # part of D that is wanted: 0 all, 1 lower triangle (row >= column), 2 upper (row <= column)
    d_mirror: bool = False       # with d_tri and M == N: the wanted triangle is copied into the other one (symmetric D)
    alpha: float = 1.0
    beta: float = 0.0
    dist_a: Dist = field(default_factory=lambda: Dist("normal", 0.0, 1.0))
    dist_b: Dist = field(default_factory=lambda: Dist("normal", 0.0, 1.0))
    dist_c: Dist = field(default_factory=lambda: Dist("normal", 0.0, 1.0))
    dist_bias: Dist = field(default_factory=lambda: Dist("normal", 0.0, 0.1))
    seed: int = BASE_SEED
    lda: int = 0
    ldb: int = 0
    ldc: int = 0
    stride_a: int = 0
    stride_b: int = 0
    stride_c: int = 0
    # sampled check of the large configs: number of seeded random rows / columns
    # (0 = check everything) and how many whole batches are checked in full
    sample_rows: int = 0
    sample_cols: int = 0
    full_batches: int = 0

    def __post_init__(self):
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

    @property
    def has_bias(self) -> bool:
        return bool(self.epilogue & 1)   # the odd epilogue values

    @property
    def flops(self) -> float:
        """Useful work: two flops per product a(i,k) b(k,j) in which neither factor is a structural zero, over the
        wanted outputs (i, j)."""
        return 2.0 * _useful_products(self.M, self.N, self.K, self.a_tri, self.b_tri, self.d_tri) * self.batch

    @property
    def min_bytes(self) -> float:
        """Compulsory HBM traffic: every operand once, the output once, C_in once when beta != 0."""
        ab = ELEM_BYTES[self.ab_dtype]
        cb = ELEM_BYTES[self.c_dtype]
        n = self.batch * (self.M * self.K + self.K * self.N) * ab + self.batch * self.M * self.N * cb
        if self.beta != 0.0:
            n += self.batch * self.M * self.N * cb
        if self.has_bias:
            n += (self.M if self.bias_per_row else self.N) * 4
        return float(n)

    def elems_a(self) -> int:
        return (self.batch - 1) * self.stride_a + (self.K if self.transa else self.M) * self.lda

    def elems_b(self) -> int:
        return (self.batch - 1) * self.stride_b + (self.N if self.transb else self.K) * self.ldb

    def elems_c(self) -> int:
        return (self.batch - 1) * self.stride_c + self.M * self.ldc


@lru_cache(maxsize=256)
def _useful_products(M: int, N: int, K: int, a_tri: int, b_tri: int, d_tri: int) -> float:
    """Number of (i, k, j) with a(i,k) and b(k,j) not structurally zero and output (i, j) wanted.  Row i of op(A)
    keeps k in [alo_i, ahi_i), column j of op(B) keeps k in [blo_j, bhi_j); the count is the summed overlap."""
    i = np.arange(M, dtype=np.int64)
    alo = np.minimum(i, K) if a_tri == 2 else np.zeros(M, np.int64)
    ahi = np.minimum(i + 1, K) if a_tri == 1 else np.full(M, K, np.int64)
    if not b_tri:   # every column keeps all of K: rows x wanted columns
        cols = np.minimum(i + 1, N) if d_tri == 1 else (np.maximum(N - i, 0) if d_tri == 2 else np.full(M, N, np.int64))
        return float(np.sum((ahi - alo) * cols))
    j = np.arange(N, dtype=np.int64)
    blo = np.minimum(j, K) if b_tri == 1 else np.zeros(N, np.int64)
    bhi = np.minimum(j + 1, K) if b_tri == 2 else np.full(N, K, np.int64)
    total = 0.0
    for r0 in range(0, M, 512):          # row blocks keep the M x N intermediate small
        r = slice(r0, min(r0 + 512, M))
        ov = np.minimum(ahi[r, None], bhi[None, :]) - np.maximum(alo[r, None], blo[None, :])
        np.maximum(ov, 0, out=ov)
        if d_tri == 1:
            ov[i[r, None] < j[None, :]] = 0
        elif d_tri == 2:
            ov[i[r, None] > j[None, :]] = 0
        total += float(ov.sum())
    return total


def _draw(dist: Dist, seed, tensor_id, n, dtype):
    if dist.kind == "uniform":
        return uniform(seed, tensor_id, n, dist.p0, dist.p1, dtype)
    if dist.kind == "normal":
        return normal(seed, tensor_id, n, dist.p0, dist.p1, dtype)
    if dist.kind == "integer":
        return integer(seed, tensor_id, n, int(dist.p0), int(dist.p1), dtype)
    raise ValueError(dist.kind)


def _zero_triangle(a: np.ndarray, w: Workload) -> None:
    """Store zeros in the part of op(A) that a triangular workload declares empty (input structure, no arithmetic)."""
    for b in range(w.batch):
        off = b * w.stride_a
        if not w.transa:          # stored M x K: row i holds op(A)[i, :]
            for i in range(w.M):
                lo, hi = (min(i + 1, w.K), w.K) if w.a_tri == 1 else (0, min(i, w.K))
                a[off + i * w.lda + lo: off + i * w.lda + hi] = 0
        else:                     # stored K x M: row k holds op(A)[:, k]
            for k in range(w.K):
                lo, hi = (0, min(k, w.M)) if w.a_tri == 1 else (min(k + 1, w.M), w.M)
                a[off + k * w.lda + lo: off + k * w.lda + hi] = 0


def _zero_triangle_b(bm: np.ndarray, w: Workload) -> None:
    """Same for op(B) (K x N): lower keeps k >= j, upper keeps k <= j."""
    for b in range(w.batch):
        off = b * w.stride_b
        if not w.transb:          # stored K x N: row k holds op(B)[k, :]
            for k in range(w.K):
                lo, hi = (min(k + 1, w.N), w.N) if w.b_tri == 1 else (0, min(k, w.N))
                bm[off + k * w.ldb + lo: off + k * w.ldb + hi] = 0
        else:                     # stored N x K: row j holds op(B)[:, j]
            for j in range(w.N):
                lo, hi = (0, min(j, w.K)) if w.b_tri == 1 else (min(j + 1, w.K), w.K)
                bm[off + j * w.ldb + lo: off + j * w.ldb + hi] = 0


def make_inputs(w: Workload, seed_offset: int = 0) -> dict:
    """Draw A, B and, when used, C_in and bias for ``w``.  ``seed_offset`` gives the
    benchmark its rotating "different random inputs" sets."""
    s = w.seed + seed_offset
    out = {"A": _draw(w.dist_a, s, TENSOR_A, w.elems_a(), w.ab_dtype),
           "B": _draw(w.dist_b, s, TENSOR_B, w.elems_b(), w.ab_dtype),
           "C": None, "bias": None}
    if w.a_tri:
        _zero_triangle(out["A"], w)
    if w.b_tri:
        _zero_triangle_b(out["B"], w)
    if w.beta != 0.0:
        out["C"] = _draw(w.dist_c, s, TENSOR_C, w.elems_c(), w.c_dtype)
    if w.has_bias:
        out["bias"] = _draw(w.dist_bias, s, TENSOR_BIAS, w.M if w.bias_per_row else w.N, F32)
    return out


_EDGES = (0, 1, 127, 128, 255, 256)


def sample_indices(n: int, count: int, seed: int, salt: int) -> np.ndarray:
    """``count`` distinct seeded indices in [0,n) plus the tile-boundary indices
    {0,1,127,128,255,256,n-2,n-1}; sorted.  count <= 0 or >= n returns everything."""
    if count <= 0 or count >= n:
        return np.arange(n, dtype=np.int64)
    g = _gen()
    keys = np.fromiter((g.gen_hash(seed, 1000 + salt, i) for i in range(n)), dtype=np.uint64, count=n)
    picked = np.argsort(keys, kind="stable")[:count]
    forced = [e for e in _EDGES if e < n] + [n - 2, n - 1]
    return np.unique(np.concatenate([picked, np.array(forced, dtype=np.int64)])).astype(np.int64)


def _isqrt_scale(k: int) -> float:
    return float(np.float32(1.0) / np.sqrt(np.float32(k)))


def configs() -> dict:
    """The five benchmark configurations, keyed c1..c5."""
    c = {}
    c["c1"] = Workload("c1_small_512_nn_bf16_f32", 512, 512, 512, transa=0, transb=0, ab_dtype=BF16, c_dtype=F32,
                       dist_a=Dist("uniform", -1.0, 1.0), dist_b=Dist("uniform", -1.0, 1.0),
                       seed=BASE_SEED + 1)
    c["c2"] = Workload("c2_square_8192_nt_bf16_bf16", 8192, 8192, 8192, transa=0, transb=1, ab_dtype=BF16,
                       c_dtype=BF16, dist_a=Dist("normal", 0.0, 1.0 / np.sqrt(8192.0)),
                       dist_b=Dist("normal", 0.0, 1.0 / np.sqrt(8192.0)), seed=BASE_SEED + 2,
                       sample_rows=256, sample_cols=256)
    c["c3"] = Workload("c3_proj_16384x14336x4096_bias_gelu_bf16", 16384, 14336, 4096, transa=0, transb=1,
                       ab_dtype=BF16, c_dtype=BF16, epilogue=EPI_BIAS_GELU_ERF,
                       dist_a=Dist("normal", 0.0, 1.0), dist_b=Dist("normal", 0.0, 0.02),
                       dist_bias=Dist("normal", 0.0, 0.1), seed=BASE_SEED + 3,
                       sample_rows=128, sample_cols=128)
    c["c4"] = Workload("c4_batched64_2048x2048x128_f16", 2048, 2048, 128, transa=0, transb=1, ab_dtype=F16,
                       c_dtype=F16, batch=64, alpha=_isqrt_scale(128),
                       dist_a=Dist("uniform", -2.0, 2.0), dist_b=Dist("uniform", -2.0, 2.0),
                       seed=BASE_SEED + 4, sample_rows=32, sample_cols=32, full_batches=4)
    c["c5"] = Workload("c5_skinny_8x28672x8192_beta1_f32", 8, 28672, 8192, transa=0, transb=1, ab_dtype=BF16,
                       c_dtype=F32, beta=1.0, dist_a=Dist("normal", 0.0, 1.0), dist_b=Dist("normal", 0.0, 0.02),
                       dist_c=Dist("normal", 0.0, 1.0), seed=BASE_SEED + 5)
    return c


def scaled(w: Workload, **changes) -> Workload:
    """A replica of ``w`` with some extents changed (leading dimensions and strides recomputed)."""
    return replace(w, lda=0, ldb=0, ldc=0, stride_a=0, stride_b=0, stride_c=0, **changes)


def small_replicas() -> dict:
    """Same layouts, dtypes, epilogues and value distributions as c2..c5 at sizes the
    oracle finishes in seconds; every extent spans several tiles and leaves a ragged tail."""
    c = configs()
    return {
        "c2s": scaled(c["c2"], name="c2_small", M=648, N=776, K=1096, sample_rows=0, sample_cols=0),
        "c3s": scaled(c["c3"], name="c3_small", M=520, N=1000, K=520, sample_rows=0, sample_cols=0),
        "c4s": scaled(c["c4"], name="c4_small", M=328, N=392, K=128, batch=5, sample_rows=0, sample_cols=0,
                      full_batches=0),
        "c5s": scaled(c["c5"], name="c5_small", M=8, N=1864, K=2136),
    }

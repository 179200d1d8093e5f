"""Pins of the CPU oracle against things other than itself: hand-computed values,
closed forms, invariants of the GEMM definition, textbook normal-CDF values and
numpy's fp64 matmul as a special-case library routine.  CPU only."""
import math
import os
import struct

import numpy as np
import pytest

import oracle
import workloads as wl
from oracle import BF16, F16, F32, Problem


def bf16_bits_to_f64(bits):
    return np.frombuffer((bits.astype(np.uint32) << 16).tobytes(), np.float32).astype(np.float64)


# ---------------------------------------------------------------- codecs

def test_bf16_hand_values():
    enc = oracle.lib().oracle_f64_to_bf16
    assert enc(1.0) == 0x3F80
    assert enc(-2.0) == 0xC000
    assert enc(1.0 + 2.0 ** -8) == 0x3F80          # tie -> even (down)
    assert enc(1.0 + 3 * 2.0 ** -8) == 0x3F82      # tie -> even (up)
    assert enc(1.0 + 2.0 ** -8 + 2.0 ** -30) == 0x3F81   # just above the tie
    assert enc(0.0) == 0x0000 and enc(-0.0) == 0x8000
    assert enc(float("inf")) == 0x7F80
    assert enc(3.4e38) == 0x7F80                   # above the largest finite bf16 (3.3895e38): overflow
    assert enc(2.0 ** -133) == 0x0001              # smallest subnormal
    assert enc(2.0 ** -134) == 0x0000              # tie at half of it -> even (zero)


def test_f16_hand_values():
    enc = oracle.lib().oracle_f64_to_f16
    assert enc(1.0) == 0x3C00
    assert enc(65504.0) == 0x7BFF
    assert enc(65520.0) == 0x7C00                  # tie -> even -> Inf
    assert enc(65519.99) == 0x7BFF
    assert enc(2.0 ** -24) == 0x0001
    assert enc(2.0 ** -25) == 0x0000               # tie -> even (zero)
    assert enc(1.5 * 2.0 ** -24) == 0x0002         # tie between 1 and 2 ulp -> even
    assert enc(1.0 / 3.0) == 0x3555
    assert enc(-1.0 / 3.0) == 0xB555
    assert enc(2.0 ** -14) == 0x0400               # smallest normal


def test_codec_roundtrip_exhaustive():
    L = oracle.lib()
    all_bits = np.arange(65536, dtype=np.uint16)
    for dtype, dec, enc in ((BF16, L.oracle_bf16_to_f64, L.oracle_f64_to_bf16),
                            (F16, L.oracle_f16_to_f64, L.oracle_f64_to_f16)):
        vals = oracle.decode(all_bits, dtype)
        back = oracle.round_to(vals, dtype)
        finite_or_inf = ~np.isnan(vals)
        assert np.array_equal(back[finite_or_inf], all_bits[finite_or_inf])
        assert np.all(np.isnan(oracle.decode(back[~finite_or_inf], dtype)))
        assert dec(int(all_bits[0x3C00 if dtype == F16 else 0x3F80])) == 1.0


def test_decode_against_independent_decoders():
    all_bits = np.arange(65536, dtype=np.uint16)
    ref16 = all_bits.view(np.float16).astype(np.float64)            # numpy's own half decoder
    got16 = oracle.decode(all_bits, F16)
    ok = ~np.isnan(ref16)
    assert np.array_equal(got16[ok], ref16[ok]) and np.all(np.isnan(got16[~ok]))
    refb = bf16_bits_to_f64(all_bits)                               # bf16 = top half of an fp32
    gotb = oracle.decode(all_bits, BF16)
    ok = ~np.isnan(refb)
    assert np.array_equal(gotb[ok], refb[ok])


def test_encode_against_numpy_half_and_generator():
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.normal(size=20000), rng.normal(size=2000) * 1e-6, rng.normal(size=2000) * 3e4,
                        np.array([65519.0, 65520.0, 65521.0, 6e-8, 2.98e-8, 2.99e-8])])
    x32 = x.astype(np.float32).astype(np.float64)      # values exactly representable in fp32
    assert np.array_equal(oracle.round_to(x32, F16), x32.astype(np.float16).view(np.uint16))
    assert np.array_equal(oracle.round_to(x32, F16), wl.encode(x32, F16))
    assert np.array_equal(oracle.round_to(x32, BF16), wl.encode(x32, BF16))


def test_direct_rounding_is_monotone_and_nearest():
    # every fp64 midpoint between adjacent finite bf16 values rounds to the even neighbour
    bits = np.arange(0x3F80, 0x3F90, dtype=np.uint16)
    v = oracle.decode(bits, BF16)
    mid = (v[:-1] + v[1:]) / 2
    r = oracle.round_to(mid, BF16)
    expect = np.where(bits[:-1] % 2 == 0, bits[:-1], bits[1:])
    assert np.array_equal(r, expect)
    assert np.array_equal(oracle.round_to(np.nextafter(mid, 10.0), BF16), bits[1:])
    assert np.array_equal(oracle.round_to(np.nextafter(mid, -10.0), BF16), bits[:-1])


# ---------------------------------------------------------------- the triple loop

def ints(shape, lo, hi, seed, dtype=BF16):
    n = int(np.prod(shape))
    return wl.integer(seed, 9, n, lo, hi, dtype).reshape(shape)


def test_tiny_hand_computed():
    # A (2x3) @ B (3x2), written out by hand
    A = wl.encode([[1, 2, 3], [4, 5, 6]], BF16)
    B = wl.encode([[7, 8], [9, 10], [11, 12]], BF16)
    y, bound = oracle.gemm(Problem(2, 2, 3), A, B)
    assert y[0].tolist() == [[58.0, 64.0], [139.0, 154.0]]
    assert bound[0].tolist() == [[58.0, 64.0], [139.0, 154.0]]
    # signs: bound uses absolute values
    A2 = wl.encode([[1, -2, 3]], BF16)
    B2 = wl.encode([[-1], [1], [0.5]], BF16)
    y, bound = oracle.gemm(Problem(1, 1, 3), A2, B2)
    assert y[0, 0, 0] == -1.5 and bound[0, 0, 0] == 4.5
    # (3x2) @ (2x4)
    A3 = wl.encode([[1, 0], [0, 2], [-1, 1]], F16)
    B3 = wl.encode([[1, 2, 3, 4], [5, 6, 7, 8]], F16)
    y, _ = oracle.gemm(Problem(3, 4, 2, ab_dtype=F16), A3, B3)
    assert y[0].tolist() == [[1, 2, 3, 4], [10, 12, 14, 16], [4, 4, 4, 4]]
    # 1x1x1
    y, _ = oracle.gemm(Problem(1, 1, 1), wl.encode([[3]], BF16), wl.encode([[-5]], BF16))
    assert y.item() == -15.0


def test_identity_and_permutation_are_exact():
    M, K = 37, 29
    A = wl.normal(11, 1, M * K, 0.0, 1.0, BF16).reshape(M, K)
    I = wl.encode(np.eye(K), BF16)
    y, _ = oracle.gemm(Problem(M, K, K), A, I)
    assert np.array_equal(y[0], oracle.decode(A, BF16))
    I2 = wl.encode(np.eye(M), BF16)
    y, _ = oracle.gemm(Problem(M, K, M), I2, A)
    assert np.array_equal(y[0], oracle.decode(A, BF16))
    perm = np.random.default_rng(3).permutation(K)
    P = np.zeros((K, K)); P[np.arange(K), perm] = 1.0          # (A P)[:, perm[k]] = A[:, k]
    y, _ = oracle.gemm(Problem(M, K, K), A, wl.encode(P, BF16))
    assert np.array_equal(y[0][:, perm], oracle.decode(A, BF16))


@pytest.mark.parametrize("K", [1, 2, 7, 64, 1000, 8192])
def test_all_ones_gives_k(K):
    A = wl.encode(np.ones((3, K)), BF16)
    B = wl.encode(np.ones((K, 5)), BF16)
    y, bound = oracle.gemm(Problem(3, 5, K), A, B)
    assert np.all(y == K) and np.all(bound == K)


def test_rank1_closed_form():
    rng = np.random.default_rng(5)
    M, N, K = 19, 23, 31
    u, v = rng.integers(-4, 5, M), rng.integers(-4, 5, K)
    w, z = rng.integers(-4, 5, K), rng.integers(-4, 5, N)
    A = wl.encode(np.outer(u, v), F16)
    B = wl.encode(np.outer(w, z), F16)
    y, _ = oracle.gemm(Problem(M, N, K, ab_dtype=F16), A, B)
    assert np.array_equal(y[0], np.outer(u, z) * float(v @ w))


def test_transpose_flags_and_leading_dimensions():
    M, N, K = 13, 17, 21
    a = ints((M, K), -4, 4, 1).astype(np.uint16)
    b = ints((K, N), -4, 4, 2).astype(np.uint16)
    base, _ = oracle.gemm(Problem(M, N, K), a, b)
    want = oracle.decode(a, BF16) @ oracle.decode(b, BF16)
    assert np.array_equal(base[0], want)
    for ta in (0, 1):
        for tb in (0, 1):
            As = np.ascontiguousarray(a.T) if ta else a
            Bs = np.ascontiguousarray(b.T) if tb else b
            y, _ = oracle.gemm(Problem(M, N, K, transa=ta, transb=tb), As, Bs)
            assert np.array_equal(y, base), (ta, tb)
            # padded leading dimensions with NaN in the padding
            nan = np.uint16(0x7FC0)
            Ap = np.full((As.shape[0], As.shape[1] + 5), nan, np.uint16); Ap[:, :As.shape[1]] = As
            Bp = np.full((Bs.shape[0], Bs.shape[1] + 3), nan, np.uint16); Bp[:, :Bs.shape[1]] = Bs
            y, _ = oracle.gemm(Problem(M, N, K, transa=ta, transb=tb, lda=Ap.shape[1], ldb=Bp.shape[1]), Ap, Bp)
            assert np.array_equal(y, base), (ta, tb, "padded")


def test_row_col_selection_matches_full():
    M, N, K = 11, 9, 15
    a = ints((M, K), -3, 3, 4)
    b = ints((N, K), -3, 3, 5)
    full, fb = oracle.gemm(Problem(M, N, K, transb=1), a, b)
    rows, cols = np.array([0, 3, 10]), np.array([8, 1])
    part, pb = oracle.gemm(Problem(M, N, K, transb=1), a, b, rows=rows, cols=cols)
    assert np.array_equal(part[0], full[0][np.ix_(rows, cols)])
    assert np.array_equal(pb[0], fb[0][np.ix_(rows, cols)])


def test_alpha_beta_semantics():
    M, N, K = 6, 10, 12
    a = wl.normal(21, 1, M * K, 0, 1, BF16).reshape(M, K)
    b = wl.normal(21, 2, K * N, 0, 1, BF16).reshape(K, N)
    c = wl.normal(21, 3, M * N, 0, 1, F32).reshape(M, N)
    p = Problem(M, N, K)
    y1, bound1 = oracle.gemm(p, a, b)
    y, _ = oracle.gemm(p, a, b, C_in=c, alpha=0.0, beta=1.0)
    assert np.array_equal(y[0], c.astype(np.float64))                  # alpha = 0, beta = 1 -> C_in
    y, _ = oracle.gemm(p, a, b, alpha=4.0)
    assert np.array_equal(y, 4.0 * y1)                                  # power-of-two alpha scales exactly
    cn = np.full((M, N), np.nan, np.float32)
    y, bnd = oracle.gemm(p, a, b, C_in=cn, beta=0.0)
    assert np.array_equal(y, y1) and np.all(np.isfinite(bnd))          # beta = 0 never reads C_in
    y, bnd = oracle.gemm(p, a, b, C_in=c, alpha=1.0, beta=0.5)
    assert np.allclose(y[0], y1[0] + 0.5 * c, rtol=0, atol=1e-13)
    assert np.allclose(bnd[0], bound1[0] + 0.5 * np.abs(c), rtol=1e-15)
    # alpha is the fp32-rounded scalar
    al = float(np.float32(1.0) / np.sqrt(np.float32(128)))
    y, _ = oracle.gemm(p, a, b, alpha=1.0 / math.sqrt(128))
    assert np.array_equal(y, al * y1)
    # bf16 C_in is decoded from its bit pattern
    cb = wl.normal(21, 3, M * N, 0, 1, BF16).reshape(M, N)
    y, _ = oracle.gemm(Problem(M, N, K, c_dtype=BF16), a, b, C_in=cb, alpha=0.0, beta=1.0)
    assert np.array_equal(y[0], oracle.decode(cb, BF16))


def test_bias_and_activations():
    M, N, K = 5, 8, 16
    a = ints((M, K), -2, 2, 31)
    b = ints((K, N), -2, 2, 32)
    bias = np.arange(N, dtype=np.float32) - 3.5
    y0, b0 = oracle.gemm(Problem(M, N, K), a, b)
    y, bd = oracle.gemm(Problem(M, N, K, epilogue=oracle.EPI_BIAS), a, b, bias=bias, alpha=2.0)
    assert np.array_equal(y[0], 2.0 * y0[0] + bias[None, :])            # bias per column, not scaled by alpha
    assert np.array_equal(bd[0], 2.0 * b0[0] + np.abs(bias)[None, :])
    y, _ = oracle.gemm(Problem(M, N, K, epilogue=oracle.EPI_RELU), a, b)
    assert np.array_equal(y, np.maximum(y0, 0.0))
    y, _ = oracle.gemm(Problem(M, N, K, epilogue=oracle.EPI_BIAS_RELU), a, b, bias=bias)
    assert np.array_equal(y[0], np.maximum(y0[0] + bias[None, :], 0.0))
    y, _ = oracle.gemm(Problem(M, N, K, epilogue=oracle.EPI_BIAS_GELU_ERF), a, b, bias=bias)
    t = y0[0] + bias[None, :]
    want = np.vectorize(lambda v: v * 0.5 * (1.0 + math.erf(v / math.sqrt(2.0))))(t)
    assert np.allclose(y[0], want, rtol=1e-13, atol=1e-15)
    with pytest.raises(ValueError):
        oracle.gemm(Problem(M, N, K, epilogue=oracle.EPI_BIAS), a, b)     # bias missing


def test_gelu_textbook_values_and_identities(golden_dir):
    g = oracle.lib().oracle_gelu_erf
    g2 = oracle.lib().oracle_gelu_erf_alt
    for line in open(os.path.join(golden_dir, "normal_cdf_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        x, want = map(float, line.split())
        assert abs(g(x) - want) < 2e-15, x
    for x in np.linspace(-8, 8, 257):
        assert abs((g(x) - g(-x)) - x) < 1e-15 * max(1.0, abs(x))       # x Phi(x) + x Phi(-x) = x
        assert abs(g(x) - g2(x)) < 1e-15 * max(1.0, abs(x))
    assert g(0.0) == 0.0
    assert g(12.0) == 12.0 and abs(g(-12.0)) < 1e-30


def test_fp8_decoders_exhaustively():
    """All 256 patterns of both 8-bit formats against the library's conversion, plus the values the format
    definitions fix (1.0, largest finite, smallest subnormal, the NaN / infinity encodings)."""
    import torch
    L = oracle.lib()
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    for fn, tdt in ((L.oracle_e4m3_to_f64, torch.float8_e4m3fn), (L.oracle_e5m2_to_f64, torch.float8_e5m2)):
        want = codes.view(tdt).to(torch.float64).numpy()
        got = np.array([fn(int(c)) for c in range(256)])
        assert np.array_equal(np.isnan(got), np.isnan(want))
        assert np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
        assert np.array_equal(np.signbit(got), np.signbit(want))
    e4, e5 = L.oracle_e4m3_to_f64, L.oracle_e5m2_to_f64
    assert e4(0x38) == 1.0 and e4(0x7E) == 448.0 and e4(0x01) == 2.0 ** -9 and e4(0xC0) == -2.0 and math.isnan(e4(0x7F))
    assert e4(0x78) == 256.0                                    # exponent field 15 is an ordinary binade: no infinity
    assert e5(0x3C) == 1.0 and e5(0x7B) == 57344.0 and e5(0x01) == 2.0 ** -16 and e5(0x7C) == math.inf and math.isnan(e5(0x7E))
    # in the GEMM: 2 x 2 by hand, e4m3 operands {1, 2; -0.5, 448} . {3; 0.25}
    a = np.array([0x38, 0x40, 0xB0, 0x7E], np.uint8)             # [[1, 2], [-0.5, 448]]
    b = np.array([0x44, 0x28], np.uint8)                         # stored N x K: [[3, 0.25]]
    y, bound = oracle.gemm(Problem(2, 1, 2, transb=1, ab_dtype=oracle.FP8_E4M3), a, b)
    assert y[0, :, 0].tolist() == [3.5, 110.5] and bound[0, :, 0].tolist() == [3.5, 113.5]


def test_logistic_silu_and_tanh_gelu(golden_dir):
    L = oracle.lib()
    sg, silu, gt, ge = L.oracle_logistic, L.oracle_silu, L.oracle_gelu_tanh, L.oracle_gelu_erf
    for line in open(os.path.join(golden_dir, "logistic_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        x, want = map(float, line.split())
        assert abs(sg(x) - want) < 2e-16 * 4, x
        assert abs(silu(x) - x * want) < 1e-15 * max(1.0, abs(x)), x
    xs = np.linspace(-30, 30, 481)
    for x in xs:
        assert abs(sg(x) + sg(-x) - 1.0) < 3e-16                          # s(x) + s(-x) = 1
        assert abs((silu(x) - silu(-x)) - x) < 1e-15 * max(1.0, abs(x))   # hence silu(x) - silu(-x) = x
        assert abs((gt(x) - gt(-x)) - x) < 1e-15 * max(1.0, abs(x))       # tanh is odd: the same identity
        u = math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)
        assert abs(gt(x) - 0.5 * x * (1.0 + math.tanh(u))) < 4e-16 * max(1.0, abs(x))   # the tanh expression itself
    assert sg(800.0) == 1.0 and sg(-800.0) == 0.0 and silu(-800.0) == 0.0   # no overflow on either side
    assert silu(0.0) == 0.0 and gt(0.0) == 0.0 and gt(10.0) == 10.0 and abs(gt(-10.0)) < 1e-30
    # the tanh form approximates x Phi(x): the two differ, but by less than 5e-4 anywhere
    dev = max(abs(gt(x) - ge(x)) for x in np.linspace(-6, 6, 2401))
    assert 1e-4 < dev < 5e-4
    # library routines in fp64
    import torch
    t = torch.linspace(-12, 12, 1001, dtype=torch.float64)
    assert np.allclose([silu(float(v)) for v in t], torch.nn.functional.silu(t).numpy(), rtol=1e-14, atol=1e-300)
    assert np.allclose([gt(float(v)) for v in t], torch.nn.functional.gelu(t, approximate="tanh").numpy(), rtol=1e-13, atol=1e-14)


def test_new_activations_and_row_bias_in_the_gemm():
    M, N, K = 6, 9, 16
    a = ints((M, K), -2, 2, 41)
    b = ints((K, N), -2, 2, 42)
    bias_n = (np.arange(N, dtype=np.float32) - 3.25) / 4
    bias_m = (np.arange(M, dtype=np.float32) * 0.5 - 1.0)
    y0, b0 = oracle.gemm(Problem(M, N, K), a, b)
    L = oracle.lib()
    for epi, f in ((oracle.EPI_BIAS_SILU, L.oracle_silu), (oracle.EPI_BIAS_GELU_TANH, L.oracle_gelu_tanh)):
        y, _ = oracle.gemm(Problem(M, N, K, epilogue=epi), a, b, bias=bias_n, alpha=0.25)
        want = np.vectorize(f)(0.25 * y0[0] + bias_n[None, :])
        assert np.array_equal(y[0], want)
        y, _ = oracle.gemm(Problem(M, N, K, epilogue=epi - 1), a, b, alpha=0.25)     # the bias-free twin
        assert np.array_equal(y[0], np.vectorize(f)(0.25 * y0[0]))
    # a per-row bias: one value per output row, also in the tolerance scale
    y, bd = oracle.gemm(Problem(M, N, K, epilogue=oracle.EPI_BIAS, bias_per_row=True), a, b, bias=bias_m)
    assert np.array_equal(y[0], y0[0] + bias_m[:, None])
    assert np.array_equal(bd[0], b0[0] + np.abs(bias_m)[:, None])
    # ... which is the per-column bias of the transposed product (A B)^T = B^T A^T
    at = np.ascontiguousarray(a.T)
    bt = np.ascontiguousarray(b.T)
    yt, _ = oracle.gemm(Problem(N, M, K, epilogue=oracle.EPI_BIAS_RELU), bt, at, bias=bias_m)
    y, _ = oracle.gemm(Problem(M, N, K, epilogue=oracle.EPI_BIAS_RELU, bias_per_row=True), a, b, bias=bias_m)
    assert np.array_equal(y[0], yt[0].T)
    with pytest.raises(ValueError):
        oracle.gemm(Problem(M, N, K, epilogue=10), a, b)                              # unknown epilogue


def test_wanted_triangle_of_a_symmetric_result():
    # the mask against numpy's own triangles, its element count in closed form, and the two triangles sharing only the diagonal
    r, c = np.arange(6), np.arange(6)
    lo, up = oracle.wanted(r, c, 1), oracle.wanted(r, c, 2)
    assert np.array_equal(lo, np.tril(np.ones((6, 6), bool))) and np.array_equal(up, np.triu(np.ones((6, 6), bool)))
    assert lo.sum() == 6 * 7 // 2 and np.array_equal(lo & up, np.eye(6, dtype=bool)) and np.all(lo | up)
    assert np.array_equal(lo, up.T) and oracle.wanted(r, c, 0).all()
    # arbitrary (sampled, unordered) rows and columns: the mask follows the indices, not the positions
    rows, cols = np.array([5, 0, 3]), np.array([4, 4, 0, 5])
    assert np.array_equal(oracle.wanted(rows, cols, 1), np.array([[1, 1, 1, 1], [0, 0, 1, 0], [0, 0, 1, 0]], bool))
    assert oracle.wanted(np.arange(7), np.arange(3), 1).sum() == 6 + 4 * 3     # 7 x 3 lower: 1 + 2 + 3, then whole rows


def test_batched_equals_loop_of_singles():
    w = wl.Workload("t", 9, 7, 12, transa=0, transb=1, ab_dtype=F16, batch=4, beta=0.5, c_dtype=F16,
                    dist_a=wl.Dist("uniform", -2, 2), dist_b=wl.Dist("uniform", -2, 2), alpha=0.25,
                    stride_a=9 * 12 + 8, stride_b=7 * 12 + 16, stride_c=9 * 7 + 24)
    inp = wl.make_inputs(w)
    p = Problem(w.M, w.N, w.K, w.transa, w.transb, w.ab_dtype, w.c_dtype, batch=w.batch,
                stride_a=w.stride_a, stride_b=w.stride_b, stride_c=w.stride_c)
    y, _ = oracle.gemm(p, inp["A"], inp["B"], C_in=inp["C"], alpha=w.alpha, beta=w.beta)
    for bi in range(w.batch):
        a = inp["A"][bi * w.stride_a: bi * w.stride_a + w.M * w.K]
        b = inp["B"][bi * w.stride_b: bi * w.stride_b + w.N * w.K]
        c = inp["C"][bi * w.stride_c: bi * w.stride_c + w.M * w.N]
        ys, _ = oracle.gemm(Problem(w.M, w.N, w.K, 0, 1, F16, F16), np.ascontiguousarray(a),
                            np.ascontiguousarray(b), C_in=np.ascontiguousarray(c), alpha=w.alpha, beta=w.beta)
        assert np.array_equal(ys[0], y[bi])
    part, _ = oracle.gemm(p, inp["A"], inp["B"], C_in=inp["C"], alpha=w.alpha, beta=w.beta, batches=[3, 1])
    assert np.array_equal(part[0], y[3]) and np.array_equal(part[1], y[1])


@pytest.mark.parametrize("shape", [(64, 48, 80), (130, 70, 257), (512, 512, 512)])
@pytest.mark.parametrize("dtype", [BF16, F16])
def test_against_numpy_fp64_matmul(shape, dtype):
    M, N, K = shape
    a = wl.normal(41, 1, M * K, 0, 1, dtype).reshape(M, K)
    b = wl.normal(41, 2, K * N, 0, 1, dtype).reshape(K, N)
    y, bound = oracle.gemm(Problem(M, N, K, ab_dtype=dtype), a, b)
    A64, B64 = oracle.decode(a, dtype), oracle.decode(b, dtype)
    ref = A64 @ B64
    refb = np.abs(A64) @ np.abs(B64)
    assert np.max(np.abs(y[0] - ref) / refb) < 1e-13
    assert np.max(np.abs(bound[0] - refb) / refb) < 1e-13


def test_k_ascending_summation_order():
    # 2^60 + 1 - 2^60: ascending order loses the 1 only if it is added to 2^60 first.
    # with k order (2^60, 1, -2^60) the fp64 result is 0; any other order gives 1.
    big = 2.0 ** 60
    a = wl.encode([[big, 1.0, -big]], BF16)
    b = wl.encode([[1.0], [1.0], [1.0]], BF16)
    y, _ = oracle.gemm(Problem(1, 1, 3), a, b)
    assert y.item() == 0.0
    a = wl.encode([[big, -big, 1.0]], BF16)
    y, _ = oracle.gemm(Problem(1, 1, 3), a, b)
    assert y.item() == 1.0


def test_rounded_output_and_threads_agree():
    M, N, K = 33, 65, 100
    a = wl.normal(51, 1, M * K, 0, 1, BF16).reshape(M, K)
    b = wl.normal(51, 2, N * K, 0, 1, BF16).reshape(N, K)
    y1, _ = oracle.gemm(Problem(M, N, K, transb=1), a, b, threads=1)
    y4, _ = oracle.gemm(Problem(M, N, K, transb=1), a, b, threads=4)
    assert np.array_equal(y1, y4)                                       # per-output loops: thread count cannot matter
    r = oracle.round_to(y1, BF16)
    back = oracle.decode(r, BF16)
    assert np.max(np.abs(back - y1) / np.maximum(np.abs(y1), 1e-30)) <= 2.0 ** -8
    assert oracle.round_to(y1, F32).dtype == np.float32
    assert np.array_equal(oracle.round_to(y1, F32), y1.astype(np.float32))


def test_fp32_rounding_of_scalars_is_applied():
    # struct.pack('f') shows what the GPU receives for alpha; the oracle must use that value
    al = 0.1
    al32 = struct.unpack("f", struct.pack("f", al))[0]
    a, b = wl.encode([[1.0]], BF16), wl.encode([[1.0]], BF16)
    y, _ = oracle.gemm(Problem(1, 1, 1), a, b, alpha=al)
    assert y.item() == al32 and y.item() != al

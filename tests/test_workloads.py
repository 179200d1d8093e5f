"""Seeded input generators and the benchmark configurations (CPU only)."""
import numpy as np

import workloads as wl


def f32_of_bf16(bits):
    return np.frombuffer((bits.astype(np.uint32) << 16).tobytes(), np.float32)


def test_generators_are_deterministic_and_counter_based():
    a = wl.normal(7, 1, 10000, 0.0, 1.0, wl.BF16)
    b = wl.normal(7, 1, 10000, 0.0, 1.0, wl.BF16)
    assert np.array_equal(a, b)
    assert np.array_equal(wl.normal(7, 1, 5000, 0.0, 1.0, wl.BF16), a[:5000])   # element i depends on i only
    assert not np.array_equal(wl.normal(8, 1, 10000, 0.0, 1.0, wl.BF16), a)     # seed matters
    assert not np.array_equal(wl.normal(7, 2, 10000, 0.0, 1.0, wl.BF16), a)     # tensor id matters


def test_distributions():
    n = 400000
    u = wl.uniform(1, 1, n, -2.0, 2.0, wl.F16).view(np.float16).astype(np.float64)
    assert u.min() >= -2.0 and u.max() <= 2.0
    assert abs(u.mean()) < 0.01 and abs(u.var() - 16.0 / 12.0) < 0.01
    z = f32_of_bf16(wl.normal(1, 2, n, 0.0, 0.02, wl.BF16)).astype(np.float64)
    assert abs(z.mean()) < 2e-4 and abs(z.std() - 0.02) < 2e-4
    assert abs(np.mean(np.abs(z) < 0.02) - 0.6827) < 0.005
    b = wl.normal(1, 4, n, 0.0, 0.1, wl.F32)
    assert b.dtype == np.float32 and abs(b.std() - 0.1) < 1e-3
    k = f32_of_bf16(wl.integer(1, 3, n, -4, 4, wl.BF16))
    assert set(np.unique(k).tolist()) == set(range(-4, 5))
    assert np.all(np.bincount((k + 4).astype(int)) > n / 9 * 0.95)


def test_configs_match_the_benchmark_definition():
    c = wl.configs()
    assert [(w.M, w.N, w.K, w.batch) for w in c.values()] == [
        (512, 512, 512, 1), (8192, 8192, 8192, 1), (16384, 14336, 4096, 1), (2048, 2048, 128, 64), (8, 28672, 8192, 1)]
    assert (c["c1"].transa, c["c1"].transb) == (0, 0)
    assert all((c[k].transa, c[k].transb) == (0, 1) for k in ("c2", "c3", "c4", "c5"))
    assert c["c3"].epilogue == wl.EPI_BIAS_GELU_ERF and c["c3"].c_dtype == wl.BF16
    assert c["c4"].ab_dtype == wl.F16 and c["c4"].c_dtype == wl.F16
    assert c["c4"].alpha == float(np.float32(1.0) / np.sqrt(np.float32(128)))
    assert (c["c4"].stride_a, c["c4"].stride_b, c["c4"].stride_c) == (262144, 262144, 4194304)
    assert c["c5"].beta == 1.0 and c["c5"].c_dtype == wl.F32
    # work and compulsory traffic
    assert c["c2"].flops == 2 * 8192.0 ** 3 and c["c2"].min_bytes == 3 * 128 * 2 ** 20
    assert abs(c["c3"].min_bytes - 721.5e6) < 0.1e6
    assert abs(c["c4"].min_bytes - 604.0e6) < 0.1e6
    assert abs(c["c5"].min_bytes - 471.7e6) < 0.1e6
    assert c["c1"].min_bytes == 2 * 2 ** 20


def test_make_inputs_shapes_and_rotation():
    w = wl.small_replicas()["c4s"]
    a = wl.make_inputs(w)
    assert a["A"].size == w.batch * w.M * w.K and a["B"].size == w.batch * w.N * w.K
    assert a["C"] is None and a["bias"] is None
    b = wl.make_inputs(w, seed_offset=1000)
    assert not np.array_equal(a["A"], b["A"])
    w5 = wl.small_replicas()["c5s"]
    i5 = wl.make_inputs(w5)
    assert i5["C"].dtype == np.float32 and i5["C"].size == w5.M * w5.N
    w3 = wl.small_replicas()["c3s"]
    assert wl.make_inputs(w3)["bias"].size == w3.N


def test_sample_indices():
    s = wl.sample_indices(8192, 256, 5, 1)
    assert np.array_equal(s, np.unique(s)) and 256 <= s.size <= 256 + 8
    for e in (0, 1, 127, 128, 255, 256, 8190, 8191):
        assert e in s
    assert np.array_equal(s, wl.sample_indices(8192, 256, 5, 1))
    assert not np.array_equal(s, wl.sample_indices(8192, 256, 5, 2))
    assert np.array_equal(wl.sample_indices(40, 0, 1, 1), np.arange(40))
    assert np.array_equal(wl.sample_indices(40, 64, 1, 1), np.arange(40))


def test_triangular_structure_of_a():
    for ta in (0, 1):
        for tri, keep in ((1, np.tril), (2, np.triu)):
            w = wl.Workload("t", 7, 5, 9, transa=ta, a_tri=tri, batch=2, lda=12)
            dense = wl.make_inputs(wl.Workload("t", 7, 5, 9, transa=ta, batch=2, lda=12))["A"]
            got = wl.make_inputs(w)["A"]
            rows, cols = (9, 7) if ta else (7, 9)
            for b in range(2):
                g = got[b * w.stride_a: b * w.stride_a + rows * 12].reshape(rows, 12)[:, :cols]
                d = dense[b * w.stride_a: b * w.stride_a + rows * 12].reshape(rows, 12)[:, :cols]
                op_g, op_d = (g.T, d.T) if ta else (g, d)          # op(A) is M x K = 7 x 9
                assert np.array_equal(op_g, keep(op_d))
    # useful work: non-zeros of op(A) times N, two flops each
    assert wl.Workload("t", 4, 3, 4, a_tri=1).flops == 2.0 * 10 * 3
    assert wl.Workload("t", 4, 3, 6, a_tri=2).flops == 2.0 * (6 + 5 + 4 + 3) * 3


def test_triangular_structure_of_b():
    for tb in (0, 1):
        for tri, keep in ((1, np.tril), (2, np.triu)):
            w = wl.Workload("t", 5, 7, 9, transb=tb, b_tri=tri, batch=2, ldb=12)
            dense = wl.make_inputs(wl.Workload("t", 5, 7, 9, transb=tb, batch=2, ldb=12))["B"]
            got = wl.make_inputs(w)["B"]
            rows, cols = (7, 9) if tb else (9, 7)
            for b in range(2):
                g = got[b * w.stride_b: b * w.stride_b + rows * 12].reshape(rows, 12)[:, :cols]
                d = dense[b * w.stride_b: b * w.stride_b + rows * 12].reshape(rows, 12)[:, :cols]
                op_g, op_d = (g.T, d.T) if tb else (g, d)          # op(B) is K x N = 9 x 7
                assert np.array_equal(op_g, keep(op_d))
    # useful work, brute force over (i, k, j): neither factor a structural zero, output wanted
    for M, N, K, a, b, d in ((5, 6, 7, 2, 2, 2), (6, 6, 6, 1, 1, 1), (4, 9, 5, 2, 1, 0), (9, 4, 5, 0, 2, 1), (3, 3, 3, 0, 1, 0)):
        cnt = sum(1 for i in range(M) for j in range(N) for k in range(K)
                  if not (d == 1 and i < j) and not (d == 2 and i > j) and not (a == 1 and k > i) and not (a == 2 and k < i)
                  and not (b == 1 and k < j) and not (b == 2 and k > j))
        assert wl.Workload("t", M, N, K, a_tri=a, b_tri=b, d_tri=d).flops == 2.0 * cnt
    # the product of two upper triangular n x n matrices costs n (n + 1) (n + 2) / 6 multiply-adds
    assert wl.Workload("t", 50, 50, 50, a_tri=2, b_tri=2, d_tri=2).flops == 2.0 * 50 * 51 * 52 / 6


def test_useful_work_of_a_triangular_result():
    # wanted elements of D, two flops per element and k: 4 x 4 lower = 10, 4 x 6 upper = 6 + 5 + 4 + 3, 6 x 4 lower = 10 + 2 * 4
    assert wl.Workload("t", 4, 4, 5, d_tri=1).flops == 2.0 * 10 * 5
    assert wl.Workload("t", 4, 6, 5, d_tri=2).flops == 2.0 * 18 * 5
    assert wl.Workload("t", 6, 4, 5, d_tri=1, batch=3).flops == 2.0 * 18 * 5 * 3
    # together with a lower-triangular op(A): row i has min(i + 1, K) non-zeros and i + 1 wanted columns
    assert wl.Workload("t", 3, 3, 3, d_tri=1, a_tri=1).flops == 2.0 * (1 * 1 + 2 * 2 + 3 * 3)
    # brute force against the definition of the mask
    for d_tri, M, N in ((1, 7, 5), (2, 7, 5), (1, 5, 9), (2, 5, 9)):
        cnt = sum(1 for i in range(M) for j in range(N) if (i >= j if d_tri == 1 else i <= j))
        assert wl.Workload("t", M, N, 2, d_tri=d_tri).flops == 2.0 * cnt * 2


def test_fp8_encoding_matches_the_library_conversion():
    import torch
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 3, 20000), rng.normal(0, 1e-3, 5000),
                        [0.0, -0.0, 1.0, 447.9, 500.0, -1e9, 2.0 ** -9, 2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -17, 1.0625, 1.1875]]).astype(np.float32)
    for dt, tdt, lim in ((wl.FP8_E4M3, torch.float8_e4m3fn, 448.0), (wl.FP8_E5M2, torch.float8_e5m2, 57344.0)):
        got = wl.encode(x, dt)
        want = torch.from_numpy(np.clip(x, -lim, lim)).to(tdt).view(torch.uint8).numpy()    # saturating, ties to even
        assert got.dtype == np.uint8 and np.array_equal(got, want)
        ints = wl.integer(1, 1, 4096, -4, 4, dt)
        assert set(torch.from_numpy(ints).view(tdt).float().tolist()) == set(float(v) for v in range(-4, 5))

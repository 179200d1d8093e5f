"""Host-side tests of the C-ABI library: it loads, exports every symbol the header declares,
validates arguments synchronously and plans the benchmark configurations as documented.
No GPU needed: nothing here launches a kernel."""
import ctypes
import os
import re

import pytest

import paper_2512_16465_b200 as bg
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gemm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gemm_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert {"gemm_plan", "gemm_run", "gemm_destroy", "gemm_workspace_bytes"} <= set(names)
    lib = ctypes.CDLL(bg.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/gemm.h but not exported"
    assert set(bg.EXPORTS) <= set(names)


def test_struct_layouts_match_the_header():
    # 2 x u32, 3 x i64, 4 x i32, 3 x i64, 2 x i32, 3 x i64, 2 x u32
    assert ctypes.sizeof(bg.Desc) == 8 + 24 + 16 + 24 + 8 + 24 + 8 and bg.Desc.structure.offset == 104
    assert bg.Desc.M.offset == 8 and bg.Desc.lda.offset == 48 and bg.Desc.batch_count.offset == 72
    assert bg.Desc.stride_a.offset == 80
    assert bg.Info.num_tiles.offset == 48 and bg.Info.flops.offset == 56


def plan_status(**kw):
    d = bg.make_desc(**kw)
    try:
        h = bg.gemm_plan(d)
    except bg.GemmError as e:
        return e.status
    bg.gemm_destroy(h)
    return bg.OK


def test_plan_validation_codes():
    ok = dict(M=256, N=256, K=256)
    assert plan_status(**ok) == bg.OK
    assert plan_status(M=0, N=256, K=256) == bg.ERR_INVALID_ARG
    assert plan_status(M=256, N=-1, K=256) == bg.ERR_INVALID_ARG
    assert plan_status(**ok, batch=0) == bg.ERR_INVALID_ARG
    assert plan_status(**ok, lda=128) == bg.ERR_INVALID_ARG          # lda < K
    assert plan_status(**ok, ldc=255) == bg.ERR_INVALID_ARG
    assert plan_status(**ok, transa=2) == bg.ERR_INVALID_ARG
    assert plan_status(**ok, epilogue=10) == bg.ERR_INVALID_ARG
    assert plan_status(**ok, flags=bg.make_flags(a_lower=True, a_upper=True)) == bg.ERR_INVALID_ARG
    assert plan_status(**ok, flags=bg.make_flags(a_lower=True)) == bg.OK
    assert plan_status(M=8, N=4096, K=4096, flags=bg.make_flags(a_upper=True)) == bg.OK      # planned dense, not stream-K
    assert plan_status(**ok, epilogue=bg.EPI_BIAS_SILU) == bg.OK
    assert plan_status(**ok, c_dtype=3) == bg.ERR_INVALID_ARG
    assert plan_status(**ok, ab_dtype=bg.F32) == bg.ERR_UNSUPPORTED
    assert plan_status(M=256, N=256, K=100, lda=100) == bg.ERR_ALIGNMENT     # 200-byte rows
    assert plan_status(M=256, N=250, K=256, c_dtype=bg.BF16) == bg.ERR_ALIGNMENT  # ldc = 250 -> 500-byte rows
    assert plan_status(M=256, N=250, K=256, c_dtype=bg.BF16, ldc=256) == bg.OK
    assert plan_status(**ok, batch=2, stride_c=100) == bg.ERR_INVALID_ARG    # outputs would overlap
    assert plan_status(**ok, batch=2, stride_a=256 * 256 + 4) == bg.ERR_ALIGNMENT
    assert plan_status(M=200, N=256, K=256, flags=bg.make_flags(bg.VARIANT_SKINNY_STREAMK)) == bg.ERR_UNSUPPORTED
    assert plan_status(**ok, flags=bg.make_flags(bg.VARIANT_DENSE_1CTA, tile_n=240)) == bg.ERR_UNSUPPORTED   # not a multiple of 64
    assert plan_status(**ok, flags=bg.make_flags(bg.VARIANT_DENSE_1CTA) | (21 << 8)) == bg.ERR_INVALID_ARG    # tile field beyond 512
    assert plan_status(**ok, transb=bg.OP_N, flags=bg.make_flags(bg.VARIANT_DENSE_1CTA, tile_n=320)) == bg.ERR_UNSUPPORTED  # wide tiles: B stored N x K
    d = bg.make_desc(**ok)
    d.struct_size = 12
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_plan(d)
    assert e.value.status == bg.ERR_INVALID_ARG
    assert bg._lib.gemm_plan(None, None) == bg.ERR_NULL
    assert bg._lib.gemm_destroy(None) == bg.OK
    assert bg._lib.gemm_workspace_bytes(None) == 0
    assert bg._lib.gemm_plan_status(None) == bg.ERR_NULL


def test_status_strings():
    names = [bg.status_string(i) for i in range(9)]
    assert names[0] == "GEMM_OK" and names[8] == "GEMM_ERR_TIMEOUT" and len(set(names)) == 9
    assert bg.status_string(99) == "GEMM_ERR_UNKNOWN"


def info_for(w: wl.Workload, flags=0):
    h = bg.gemm_plan(bg.make_desc(w.M, w.N, w.K, w.transa, w.transb, w.ab_dtype, w.c_dtype, batch=w.batch,
                                  epilogue=w.epilogue, flags=flags))
    info = bg.gemm_plan_info(h)
    bg.gemm_destroy(h)
    return info


def test_roofline_classification_of_the_five_configs():
    c = wl.configs()
    i1, i2, i3, i4, i5 = (info_for(c[k]) for k in ("c1", "c2", "c3", "c4", "c5"))
    # arithmetic intensities of the configurations (flops / compulsory bytes)
    assert i1["intensity"] == pytest.approx(128.0)
    assert i2["intensity"] == pytest.approx(2730.67, rel=1e-4)
    assert i3["intensity"] == pytest.approx(2667.0, rel=1e-3)
    assert i4["intensity"] == pytest.approx(113.78, rel=1e-3)
    assert i5["intensity"] == pytest.approx(7.98, rel=1e-2)       # C read for beta is a run-time matter
    assert [i["regime"] for i in (i1, i2, i3, i4, i5)] == [1, 2, 2, 1, 0]
    assert i5["variant"] == bg.VARIANT_SKINNY_STREAMK and i5["workspace_bytes"] > 0
    for i in (i1, i2, i3, i4):
        assert i["variant"] in (bg.VARIANT_DENSE_1CTA, bg.VARIANT_DENSE_2CTA, bg.VARIANT_DENSE_2CTA_WIDE)
        assert i["workspace_bytes"] == 0
        assert i["smem_bytes"] <= 232448 and i["stages"] >= 2
    assert i2["flops"] == 2.0 * 8192 ** 3 and i2["min_bytes"] == 3 * 8192 * 8192 * 2
    assert i2["variant"] == bg.VARIANT_DENSE_2CTA_WIDE and (i2["tile_m"], i2["tile_n"], i2["stages"]) == (512, 256, 3)
    assert i3["variant"] == bg.VARIANT_DENSE_2CTA          # erf-GELU epilogue: keep the double-buffered accumulator
    assert i4["variant"] == bg.VARIANT_DENSE_2CTA_WIDE   # output-bound: the largest tiles, fewest tile switches (measured)
    assert i1["variant"] == bg.VARIANT_DENSE_1CTA
    for k, i in zip(("c1", "c2", "c3", "c4", "c5"), (i1, i2, i3, i4, i5)):
        assert i["flops"] == c[k].flops


def test_stream_k_plan_geometry():
    i5 = info_for(wl.configs()["c5"])
    assert i5["num_tiles"] == 224 * 64               # (n-tile, 128-wide k-block) work units
    assert i5["grid"] == 148 and i5["tile_m"] == 128 and i5["tile_n"] == 16 and i5["tile_k"] == 128
    assert i5["split"] >= 2 and i5["stages"] == 4    # 4 stages of two 64-wide K slices: 144 KB in flight per SM
    # one 64-bit arrival word per output tile (padded to 256 bytes), then 2 partial slots of 128 x 16 fp32 per CTA
    assert i5["workspace_bytes"] == 224 * 8 + 148 * 2 * 128 * 16 * 4
    tiny = info_for(wl.Workload("t", 4, 100, 64), bg.make_flags(bg.VARIANT_SKINNY_STREAMK))
    assert tiny["grid"] == 1 and tiny["num_tiles"] == 1
    # grids that line up with the tiles on mid-sized problems
    sk = bg.make_flags(bg.VARIANT_SKINNY_STREAMK)
    grid = lambda M, N, K: bg.Plan(bg.make_desc(M, N, K, flags=sk)).info["grid"]
    # (clusters of c CTAs per tile: c is the most the device holds at once, so the exact grid depends on the GPU; a plan made
    # without a device assumes SM count / c clusters of every size)
    assert grid(64, 4096, 4096) in (96, 128)  # 32 tiles: four CTAs per tile, as clusters that hand over through shared memory
    assert grid(16, 4096, 4096) in (96, 128)
    assert grid(64, 14336, 16384) == 112      # one whole tile per CTA: more than two thirds of the SMs, any size
    assert grid(16, 11008, 16384) == 115      # 86 tiles: three tiles per four CTAs (28 such groups, two tiles left to three CTAs)
    assert grid(64, 12288, 4096) == 128       # 96 tiles: 32 groups of four CTAs
    assert grid(64, 12288, 1024) == 96        # short K: whole tiles
    assert grid(64, 5120, 5120) in (80, 120)  # 40 tiles: clusters of three (or two)
    assert grid(64, 8192, 8192) == 128        # 64 tiles: clusters of two
    assert grid(64, 9472, 4096) in (74, 148)  # 74 tiles: clusters of two on all SMs when they all fit
    assert grid(8192, 64, 4096 * 2) == grid(64, 8192, 4096 * 2)   # the tall form shares the rule


def test_forced_variants_and_tiles():
    w = wl.configs()["c2"]
    i = info_for(w, bg.make_flags(bg.VARIANT_DENSE_2CTA, tile_n=256))
    assert (i["variant"], i["cluster_size"], i["tile_m"], i["tile_n"]) == (2, 2, 256, 256)
    assert i["num_tiles"] == 32 * 32 and i["grid"] == 148
    i = info_for(w, bg.make_flags(bg.VARIANT_DENSE_1CTA, tile_n=128, raster=5, stages=3))
    assert (i["tile_m"], i["tile_n"], i["raster_group"], i["stages"]) == (128, 128, 5, 3)
    assert i["num_tiles"] == 64 * 64


def test_run_without_a_device_is_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = bg.gemm_plan(bg.make_desc(128, 128, 64))
    buf = (ctypes.c_char * 65536)()
    addr = (ctypes.addressof(buf) + 15) & ~15
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_run(h, addr, addr, addr, 0, 1.0, 0.0, 0, 0, 0)
    assert e.value.status == bg.ERR_ARCH
    assert bg.gemm_plan_status(h) == bg.ERR_ARCH
    bg.gemm_destroy(h)


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2512_16465_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"


def test_cost_model_choices_follow_the_measurements():
    """The plan scores (family, tile width) candidates with a roofline estimate; these are shapes whose best
    family was measured on a B200."""
    def choice(M, N, K, **kw):
        h = bg.gemm_plan(bg.make_desc(M, N, K, c_dtype=bg.BF16, **kw))
        i = bg.gemm_plan_info(h)
        bg.gemm_destroy(h)
        return i["variant"], i["tile_n"]
    assert choice(2048, 2048, 2048) == (bg.VARIANT_DENSE_2CTA, 256)          # 64 pair tiles on 74 pairs beat 256 small ones
    assert choice(4096, 4096, 4096) == (bg.VARIANT_DENSE_2CTA_WIDE, 256)
    assert choice(128, 28672, 8192) == (bg.VARIANT_DENSE_1CTA, 256)          # one tile row: no pair
    assert choice(16384, 14336, 4096, epilogue=bg.EPI_BIAS_GELU_ERF)[0] == bg.VARIANT_DENSE_2CTA
    assert choice(16, 28672, 8192)[0] == bg.VARIANT_SKINNY_STREAMK
    assert choice(28672, 16, 8192)[0] == bg.VARIANT_SKINNY_STREAMK            # mirrored: the long operand is A
    assert choice(28672, 16, 8192, transb=bg.OP_N)[0] != bg.VARIANT_SKINNY_STREAMK   # needs both operands K-contiguous
    assert choice(64, 28672, 8192)[0] == bg.VARIANT_SKINNY_STREAMK            # up to the largest short extent the path takes
    assert choice(128, 28672, 8192)[0] == bg.VARIANT_DENSE_1CTA
    v, bn = choice(2048, 2048, 128, batch=64)
    assert (v, bn) == (bg.VARIANT_DENSE_2CTA_WIDE, 256)                      # output-bound: largest tile, fewest tile switches
    assert choice(8192, 8192, 1024)[0] == bg.VARIANT_DENSE_2CTA              # the pair beats the single CTA at every K measured


def test_triangular_result_plans():
    """One triangle of D wanted: the plan lists only the tiles that touch it, counts the useful work, and keeps to the
    kernels that have a tile list."""
    full = bg.Plan(bg.make_desc(8192, 8192, 8192, c_dtype=bg.F32)).info
    for fl in (bg.make_flags(d_lower=True), bg.make_flags(d_upper=True)):
        info = bg.Plan(bg.make_desc(8192, 8192, 8192, c_dtype=bg.F32, flags=fl)).info
        assert info["variant"] == bg.VARIANT_DENSE_2CTA and (info["tile_m"], info["tile_n"]) == (256, 256)
        assert info["num_tiles"] == 32 * 33 // 2                      # 32 x 32 square tiles, diagonal included
        assert info["flops"] == 2.0 * (8192 * 8193 // 2) * 8192 and info["flops"] < 0.51 * full["flops"]
    # non-square tiles and matrices: 1000 x 600 output, 128 x 64 tiles -> row i keeps columns 0 .. min(9, (128 (i + 1) - 1) // 64)
    info = bg.Plan(bg.make_desc(1000, 600, 256, c_dtype=bg.F32, flags=bg.make_flags(variant=bg.VARIANT_DENSE_1CTA, tile_n=64, d_lower=True))).info
    assert info["num_tiles"] == sum(min(9, (min(128 * (i + 1), 1000) - 1) // 64) + 1 for i in range(8))
    info = bg.Plan(bg.make_desc(1000, 600, 256, c_dtype=bg.F32, flags=bg.make_flags(variant=bg.VARIANT_DENSE_1CTA, tile_n=64, d_upper=True))).info
    assert info["num_tiles"] == sum(max(0, 10 - (128 * i) // 64) for i in range(8) if 128 * i <= 599)
    # batches multiply the list
    info = bg.Plan(bg.make_desc(512, 512, 256, c_dtype=bg.F32, batch=7, flags=bg.make_flags(variant=bg.VARIANT_DENSE_1CTA, tile_n=128, d_lower=True))).info
    assert info["num_tiles"] == 7 * 10
    for bad in (bg.make_flags(variant=bg.VARIANT_DENSE_2CTA_WIDE, d_lower=True), bg.make_flags(variant=bg.VARIANT_SKINNY_STREAMK, d_upper=True)):
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(bg.make_desc(64 if bad & 0x30 == 0x30 else 4096, 4096, 4096, flags=bad))
        assert e.value.status == bg.ERR_UNSUPPORTED
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_plan(bg.make_desc(512, 512, 512, flags=bg.make_flags(d_lower=True, d_upper=True)))
    assert e.value.status == bg.ERR_INVALID_ARG
    # structure of op(B): unknown bits, both triangles at once and an unknown option bit are invalid; the kernels
    # without K ranges refuse it; it keeps a short output away from stream-K as well
    for structure in (0x4, bg.STRUCT_B_LOWER | bg.STRUCT_B_UPPER):
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(bg.make_desc(512, 512, 512, structure=structure))
        assert e.value.status == bg.ERR_INVALID_ARG
    d = bg.make_desc(512, 512, 512)
    d.options = 2
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_plan(d)
    assert e.value.status == bg.ERR_INVALID_ARG
    for v, M in ((bg.VARIANT_DENSE_2CTA_WIDE, 4096), (bg.VARIANT_SKINNY_STREAMK, 64)):
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(bg.make_desc(M, 4096, 4096, flags=bg.make_flags(variant=v), structure=bg.STRUCT_B_UPPER))
        assert e.value.status == bg.ERR_UNSUPPORTED
    assert bg.Plan(bg.make_desc(8192, 8192, 8192, structure=bg.STRUCT_B_LOWER)).info["variant"] == bg.VARIANT_DENSE_2CTA
    assert bg.Plan(bg.make_desc(64, 8192, 8192, structure=bg.STRUCT_B_UPPER)).info["variant"] != bg.VARIANT_SKINNY_STREAMK
    # a short output that would go to stream-K stays dense when a triangle is asked for
    assert bg.Plan(bg.make_desc(64, 8192, 8192, flags=bg.make_flags(d_upper=True))).info["variant"] != bg.VARIANT_SKINNY_STREAMK


def test_tuning_entry_points_on_the_host():
    # the workspace bound needs no device: only the stream-K candidates of a short-extent problem use one
    assert bg.gemm_tune_workspace_bytes(bg.make_desc(8192, 8192, 512)) == 0          # nothing to split, no short extent
    assert bg.gemm_tune_workspace_bytes(bg.make_desc(1024, 1024, 4096)) > 0           # a tail-split candidate wants room
    need = bg.gemm_tune_workspace_bytes(bg.make_desc(8, 4096, 2048))
    assert need >= 148 * 2 * 128 * 16 * 4
    # mirrored: the same partial tiles (the flag words at the head of a tail-split candidate's workspace differ a little)
    assert abs(bg.gemm_tune_workspace_bytes(bg.make_desc(4096, 8, 2048)) - need) <= 1024
    bg.gemm_tune_cache_clear()                                                    # harmless when empty
    import torch
    if not torch.cuda.is_available():
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_tune(bg.make_desc(256, 256, 64), 16, 16, 16, 0, 1.0, 0.0, 0, 0, 0)
        assert e.value.status in (bg.ERR_ARCH, bg.ERR_CUDA)                       # no device: an error, never a fallback
        for fn in (bg.gemm_tune_cache_save, bg.gemm_tune_cache_load):               # results belong to a device
            with pytest.raises(bg.GemmError) as e:
                fn("/nonexistent-directory/tune.txt")
            assert e.value.status == bg.ERR_ARCH
    assert bg._lib.gemm_tune_cache_save(None, None) == bg.ERR_NULL and bg._lib.gemm_tune_cache_load(None, None) == bg.ERR_NULL


def test_host_pipeline_entry_points_without_a_device():
    import torch
    for kw in (dict(transa=bg.OP_T), dict(batch=2), dict(flags=bg.make_flags(a_upper=True)),
               dict(flags=bg.make_flags(d_lower=True))):   # refused before any device work
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_host_create(bg.make_desc(256, 256, 256, **kw))
        assert e.value.status == bg.ERR_UNSUPPORTED
    assert bg.gemm_host_panels(0) == 0
    bg.gemm_host_destroy(0)                                                      # NULL is accepted
    if not torch.cuda.is_available():
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_host_create(bg.make_desc(256, 256, 256))
        assert e.value.status in (bg.ERR_ARCH, bg.ERR_CUDA)                      # an error, never a CPU fallback

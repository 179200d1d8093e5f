"""GPU parity tests: the CUDA path, called through the C-ABI binding, against the CPU oracle
on the same seeded inputs.  Run with ``-m gpu`` on a B200."""
import os
from dataclasses import replace

import numpy as np
import pytest
import torch

import harness as H
import oracle
import paper_2512_16465_b200 as bg
import workloads as wl

pytestmark = pytest.mark.gpu

INT = wl.Dist("integer", -4, 4)
V1, V2, VS = bg.VARIANT_DENSE_1CTA, bg.VARIANT_DENSE_2CTA, bg.VARIANT_SKINNY_STREAMK
VW = bg.VARIANT_DENSE_2CTA_WIDE


def int_workload(name, M, N, K, ta=0, tb=1, ab=wl.BF16, cd=wl.F32, batch=1, epi=0, alpha=1.0, beta=0.0, **kw):
    """Integer-valued inputs in [-4, 4]: every product and partial sum is an exactly representable
    integer (< 2^24), so fp32 accumulation is exact in any order and the result must be bit-identical."""
    return wl.Workload(name, M, N, K, transa=ta, transb=tb, ab_dtype=ab, c_dtype=cd, batch=batch, epilogue=epi,
                       alpha=alpha, beta=beta, dist_a=INT, dist_b=INT, dist_c=INT, dist_bias=INT, seed=4242, **kw)


# ----------------------------------------------------------------------------- exact regime

EXACT_CASES = [
    # name, M, N, K, kwargs, flags
    ("one_tile", 128, 128, 64, {}, dict(variant=V1, tile_n=128)),
    ("one_kblock_ragged_k", 128, 64, 40, {}, dict(variant=V1, tile_n=64)),
    ("tile_n_256", 256, 512, 192, {}, dict(variant=V1, tile_n=256)),
    ("tile_n_192", 256, 576, 192, {}, dict(variant=V1, tile_n=192)),
    ("ragged_all", 200, 328, 200, {}, dict(variant=V1, tile_n=128)),
    ("tiny", 1, 8, 8, {}, dict(variant=V1)),
    ("one_by_one_by_one", 1, 1, 1, dict(lda=8, ldb=8, ldc=4), dict(variant=V1)),
    ("one_by_one_by_one_skinny", 1, 1, 1, dict(lda=8, ldb=8, ldc=4), dict(variant=VS)),
    ("many_small_batches", 64, 64, 64, dict(batch=300, cd=wl.BF16), dict(variant=V1)),
    ("very_long_k", 128, 64, 65536, {}, dict(variant=V1)),
    ("very_wide_n", 128, 70000, 64, dict(cd=wl.BF16), dict(variant=V1)),
    ("m1_n_ragged", 1, 1000, 72, {}, dict(variant=V1)),
    ("n_small", 300, 8, 136, {}, dict(variant=V1)),
    ("persistent_many_tiles", 1536, 2560, 128, {}, dict(variant=V1, tile_n=64)),
    ("raster_1", 1024, 1024, 64, {}, dict(variant=V1, tile_n=128, raster=1)),
    ("raster_3", 1100, 1024, 64, {}, dict(variant=V1, tile_n=128, raster=3)),
    ("stages_2", 256, 256, 1024, {}, dict(variant=V1, tile_n=128, stages=2)),
    ("stages_3_long_k", 128, 256, 8192, {}, dict(variant=V1, tile_n=256, stages=3)),
    ("nn", 264, 328, 200, dict(ta=0, tb=0), dict(variant=V1, tile_n=128)),
    ("nn_wide", 256, 512, 128, dict(ta=0, tb=0), dict(variant=V1, tile_n=256)),
    ("tn", 264, 328, 200, dict(ta=1, tb=1), dict(variant=V1, tile_n=128)),
    ("tt", 264, 328, 200, dict(ta=1, tb=0), dict(variant=V1, tile_n=64)),
    ("f16_in_f16_out", 200, 328, 136, dict(ab=wl.F16, cd=wl.F16), dict(variant=V1)),
    ("bf16_out", 200, 328, 136, dict(cd=wl.BF16), dict(variant=V1)),
    ("f16_in_f32_out", 200, 328, 136, dict(ab=wl.F16), dict(variant=V1)),
    ("alpha_beta_f32", 200, 328, 136, dict(alpha=0.5, beta=2.0), dict(variant=V1)),
    ("beta_bf16_c", 200, 328, 136, dict(cd=wl.BF16, beta=1.0), dict(variant=V1)),
    ("beta_f16_c", 200, 328, 136, dict(ab=wl.F16, cd=wl.F16, beta=-1.0), dict(variant=V1)),
    ("bias", 200, 328, 136, dict(epi=bg.EPI_BIAS), dict(variant=V1)),
    ("relu", 200, 328, 136, dict(epi=bg.EPI_RELU, cd=wl.BF16), dict(variant=V1)),
    ("bias_relu_beta", 200, 328, 136, dict(epi=bg.EPI_BIAS_RELU, beta=1.0, alpha=2.0), dict(variant=V1)),
    ("batched_tight", 200, 328, 72, dict(batch=5, ab=wl.F16, cd=wl.F16, alpha=0.25), dict(variant=V1)),
    ("batched_nn", 136, 200, 72, dict(batch=3, ta=0, tb=0), dict(variant=V1)),
    ("pair_one_tile", 256, 128, 64, {}, dict(variant=V2, tile_n=128)),
    ("pair_256x256", 512, 512, 256, {}, dict(variant=V2, tile_n=256)),
    ("pair_ragged", 600, 712, 200, {}, dict(variant=V2, tile_n=128)),
    ("pair_m_below_tile", 100, 300, 136, {}, dict(variant=V2, tile_n=64)),
    ("pair_nn", 520, 512, 200, dict(ta=0, tb=0), dict(variant=V2, tile_n=128)),
    ("pair_tn", 520, 512, 200, dict(ta=1, tb=1), dict(variant=V2, tile_n=256)),
    ("pair_tt", 520, 512, 200, dict(ta=1, tb=0), dict(variant=V2, tile_n=256)),
    ("pair_batched_bias_bf16", 300, 264, 136, dict(batch=3, epi=bg.EPI_BIAS, cd=wl.BF16), dict(variant=V2, tile_n=128)),
    ("pair_persistent_beta", 2048, 4096, 128, dict(beta=1.0), dict(variant=V2, tile_n=256)),
    ("pair_forward_k_only", 512, 512, 1000, {}, dict(variant=V2, tile_n=256, no_k_serpentine=True)),
    ("pair_serpentine_many_tiles_odd_stages", 1024, 2048, 712, {}, dict(variant=V2, tile_n=128)),
    ("pair_one_slice_stages", 1024, 1024, 712, {}, dict(variant=V2, tile_n=256, kslices=1)),
    ("single_serpentine_ragged_k", 1100, 1100, 456, {}, dict(variant=V1, tile_n=128, kslices=2)),
    ("single_l2_hints", 600, 600, 520, {}, dict(variant=V1, tile_n=64, l2_hints=True)),
    ("pair_l2_hints", 600, 600, 520, {}, dict(variant=V2, tile_n=128, l2_hints=True)),
    ("wide_one_tile", 512, 256, 64, {}, dict(variant=VW)),
    ("wide_ragged", 1100, 712, 456, {}, dict(variant=VW)),
    ("wide_m_below_tile", 100, 300, 136, {}, dict(variant=VW)),
    ("wide_persistent_bf16", 4096, 4096, 320, dict(cd=wl.BF16), dict(variant=VW)),
    ("wide_beta_bias_f32", 1100, 712, 200, dict(beta=1.0, epi=bg.EPI_BIAS), dict(variant=VW)),
    ("wide_nn", 1024, 520, 264, dict(ta=0, tb=0), dict(variant=VW)),
    ("wide_tn", 1024, 520, 264, dict(ta=1, tb=1), dict(variant=VW)),
    ("wide_tt_batched_f16", 600, 520, 136, dict(ta=1, tb=0, batch=3, ab=wl.F16, cd=wl.F16, alpha=0.5), dict(variant=VW)),
    ("wide_two_stage_ring_forward_k", 1024, 512, 1000, {}, dict(variant=VW, stages=2, no_k_serpentine=True)),
    ("skinny_one_unit", 8, 128, 64, {}, dict(variant=VS)),
    ("skinny_split_k", 8, 256, 4096, {}, dict(variant=VS)),
    ("skinny_ragged_beta", 8, 1864, 2136, dict(beta=1.0), dict(variant=VS)),
    ("skinny_gemv", 1, 4096, 4096, {}, dict(variant=VS)),
    ("skinny_m16_whole_tiles", 16, 28672, 1024, {}, dict(variant=VS)),
    ("skinny_m33_bias_bf16", 33, 1000, 520, dict(cd=wl.BF16, epi=bg.EPI_BIAS), dict(variant=VS)),
    ("skinny_m64_f16", 64, 520, 1032, dict(ab=wl.F16, cd=wl.F16, alpha=0.5, beta=1.0), dict(variant=VS)),
    ("skinny_stages_2", 8, 384, 1024, {}, dict(variant=VS, stages=2)),
    ("skinny_one_slice_stages", 8, 256, 4096, {}, dict(variant=VS, kslices=1)),
    ("skinny_three_slice_stages", 8, 384, 1100 - 4, {}, dict(variant=VS, kslices=3)),
    ("skinny_k_slice_past_the_end", 8, 256, 1080, {}, dict(variant=VS)),
    # tiles wider than 256 columns: two MMAs side by side per K step, one accumulator buffer
    ("wide_n_512_pair_one_tile", 256, 512, 256, {}, dict(variant=V2, tile_n=512)),
    ("wide_n_320_pair_ragged_bf16", 600, 712, 456, dict(cd=wl.BF16), dict(variant=V2, tile_n=320)),
    ("wide_n_384_pair_beta_bias_f32", 520, 1000, 200, dict(beta=1.0, epi=bg.EPI_BIAS_RELU), dict(variant=V2, tile_n=384)),
    ("wide_n_448_1cta_f16", 300, 904, 136, dict(ab=wl.F16, cd=wl.F16, alpha=0.5), dict(variant=V1, tile_n=448)),
    ("wide_n_512_1cta_many_tiles", 1024, 2048, 328, dict(cd=wl.BF16), dict(variant=V1, tile_n=512)),
    ("wide_n_512_pair_several_tiles_per_cta", 2560, 5120, 264, dict(cd=wl.BF16), dict(variant=V2, tile_n=512)),
    ("wide_n_384_pair_one_slice_stages", 512, 768, 712, {}, dict(variant=V2, tile_n=384, kslices=1)),
    ("wide_n_320_pair_a_stored_transposed", 520, 640, 200, dict(ta=1), dict(variant=V2, tile_n=320)),
    ("wide_n_512_fp8", 512, 1024, 1040, dict(ab=wl.FP8_E4M3, cd=wl.BF16), dict(variant=V2, tile_n=512)),
    ("wide_n_384_batched", 300, 504, 136, dict(batch=3, cd=wl.BF16), dict(variant=V2, tile_n=384)),
    ("wide_n_512_lower_triangular_d_upper", 1024, 1024, 1024, dict(a_tri=1, d_tri=2), dict(variant=V2, tile_n=512)),
    ("wide_n_320_n_not_a_multiple_of_16_bytes", 300, 650, 136, dict(cd=wl.BF16, ldc=656), dict(variant=V2, tile_n=320)),
    ("wide_n_auto_2304", 2304, 2304, 264, dict(cd=wl.BF16), dict()),
    # stream-K with exactly c CTAs per output tile: the c CTAs form a cluster and hand over through shared memory
    ("cluster_4_m8", 8, 4096, 4096, {}, dict(variant=VS)),
    ("cluster_4_m64_f16_beta", 64, 4096, 4096, dict(ab=wl.F16, cd=wl.F16, alpha=0.5, beta=1.0), dict(variant=VS)),
    ("cluster_8_m16_bias_bf16", 16, 2048, 8192, dict(cd=wl.BF16, epi=bg.EPI_BIAS), dict(variant=VS)),
    ("cluster_4_ragged_m33", 33, 4000, 4608, dict(beta=1.0, epi=bg.EPI_BIAS_RELU), dict(variant=VS)),
    ("cluster_4_tall_n8", 4096, 8, 4096, dict(beta=1.0), dict(variant=VS)),
    ("cluster_4_tall_n48_padded", 4000, 48, 4608, dict(cd=wl.BF16, ldc=56, epi=bg.EPI_BIAS, bias_per_row=True), dict(variant=VS)),
    ("cluster_4_fp8", 8, 4096, 8192, dict(ab=wl.FP8_E4M3), dict(variant=VS)),
    ("cluster_auto_plan", 64, 4096, 4096, dict(cd=wl.BF16), dict()),
    # CTA ranges longer than a tile: every split tile has two contributors, several 16-row chunks each (double-buffered fix-up)
    ("skinny_m64_two_contributors", 64, 20480, 2048, dict(beta=1.0, epi=bg.EPI_BIAS), dict(variant=VS)),
    ("tall_n48_two_contributors", 20480, 48, 2048, dict(cd=wl.BF16, beta=1.0, ldc=56), dict(variant=VS)),
    ("skinny_m33_two_contributors_fp8", 33, 20000, 4096, dict(ab=wl.FP8_E4M3, cd=wl.F16), dict(variant=VS)),
    # 74 ... 100 tiles: three tiles per four CTAs, the tail of every tile handed to the CTA that holds its head
    ("grouped_m64_beta_bias", 64, 10240, 4096, dict(beta=1.0, epi=bg.EPI_BIAS), dict(variant=VS)),
    ("grouped_m8_bf16_ragged_columns", 8, 11003, 4104, dict(cd=wl.BF16, ldc=11008), dict(variant=VS)),
    ("grouped_tall_n40_f16", 12288, 40, 4096, dict(ab=wl.F16, cd=wl.F16, beta=1.0), dict(variant=VS)),
    ("grouped_fp8_m16", 16, 9600, 8192, dict(ab=wl.FP8_E4M3), dict(variant=VS)),
    # results leave through staged tile stores in whole 16-byte units; the columns behind the last whole unit from registers
    ("skinny_columns_not_a_multiple_of_16_bytes_bf16", 24, 1003, 520, dict(cd=wl.BF16, ldc=1008, epi=bg.EPI_BIAS), dict(variant=VS)),
    ("skinny_columns_not_a_multiple_of_16_bytes_f32", 64, 1001, 1032, dict(beta=1.0, ldc=1004), dict(variant=VS)),
    ("skinny_three_columns", 8, 3, 520, dict(ldc=4), dict(variant=VS)),
    ("cluster_no_early_launch", 8, 4096, 4096, dict(beta=1.0), dict(variant=VS, no_early_launch=True)),
    ("no_early_launch_1cta", 264, 328, 200, {}, dict(variant=V1, tile_n=128, no_early_launch=True)),
    ("no_early_launch_skinny", 8, 256, 4096, dict(beta=1.0), dict(variant=VS, no_early_launch=True)),
    # triangular op(A): K ranges that can only contribute zeros are skipped
    ("tri_lower_1cta", 512, 264, 512, dict(a_tri=1), dict(variant=V1, tile_n=128)),
    ("tri_upper_1cta", 512, 264, 512, dict(a_tri=2), dict(variant=V1, tile_n=128)),
    ("tri_lower_pair_ragged", 600, 328, 520, dict(a_tri=1), dict(variant=V2, tile_n=128)),
    ("tri_upper_pair_k_longer", 300, 264, 1000, dict(a_tri=2), dict(variant=V2, tile_n=128)),
    ("tri_lower_m_longer", 1000, 136, 200, dict(a_tri=1), dict(variant=V1)),
    ("tri_upper_m_longer", 1000, 136, 200, dict(a_tri=2), dict(variant=V1)),
    ("tri_lower_a_stored_transposed", 512, 264, 512, dict(a_tri=1, ta=1), dict(variant=V1, tile_n=128)),
    ("tri_upper_one_slice_stages", 512, 264, 512, dict(a_tri=2), dict(variant=V2, tile_n=128, kslices=1)),
    ("tri_lower_no_serpentine", 512, 264, 512, dict(a_tri=1), dict(variant=V1, tile_n=64, no_k_serpentine=True)),
    ("tri_lower_batched_beta", 256, 136, 256, dict(a_tri=1, batch=3, beta=1.0, cd=wl.BF16), dict(variant=V1)),
    ("tri_lower_auto", 2048, 512, 2048, dict(a_tri=1, cd=wl.BF16), dict()),
    # 8-bit float operands (tcgen05 kind::f8f6f4): 128 elements of K per 128-byte slice
    ("fp8_e4m3_one_tile", 128, 128, 128, dict(ab=wl.FP8_E4M3), dict(variant=V1, tile_n=128)),
    ("fp8_e5m2_ragged", 200, 328, 208, dict(ab=wl.FP8_E5M2), dict(variant=V1, tile_n=128)),
    ("fp8_e4m3_pair_long_k", 300, 264, 4096 + 64, dict(ab=wl.FP8_E4M3), dict(variant=V2, tile_n=128)),
    ("fp8_e5m2_pair_256", 512, 512, 1024, dict(ab=wl.FP8_E5M2, cd=wl.BF16), dict(variant=V2, tile_n=256)),
    ("fp8_e4m3_bias_relu_f16_out", 200, 328, 272, dict(ab=wl.FP8_E4M3, cd=wl.F16, epi=bg.EPI_BIAS_RELU, beta=1.0), dict(variant=V1)),
    ("fp8_e4m3_batched", 96, 72, 256, dict(ab=wl.FP8_E4M3, batch=3), dict(variant=V1)),
    ("fp8_e4m3_one_slice_stages", 256, 256, 1040, dict(ab=wl.FP8_E4M3), dict(variant=V1, tile_n=128, kslices=1)),
    ("fp8_e4m3_tiny_k", 128, 64, 16, dict(ab=wl.FP8_E4M3), dict(variant=V1, tile_n=64)),
    ("fp8_e4m3_lower_triangular", 512, 264, 512, dict(ab=wl.FP8_E4M3, a_tri=1), dict(variant=V2, tile_n=128)),
    ("fp8_e4m3_auto", 1024, 1024, 2048, dict(ab=wl.FP8_E4M3, cd=wl.BF16), dict()),
    ("fp8_e4m3_wide", 1024, 512, 2048, dict(ab=wl.FP8_E4M3, cd=wl.BF16), dict(variant=VW)),
    ("fp8_e5m2_wide_ragged_bias_relu", 700, 328, 1040, dict(ab=wl.FP8_E5M2, epi=bg.EPI_BIAS_RELU, beta=1.0), dict(variant=VW)),
    ("fp8_e4m3_wide_short_k", 600, 264, 128, dict(ab=wl.FP8_E4M3), dict(variant=VW)),
    ("fp8_e4m3_stream_k", 8, 520, 4096 + 128, dict(ab=wl.FP8_E4M3, beta=1.0), dict(variant=VS)),
    ("fp8_e5m2_stream_k_tall_bias", 1000, 33, 1040, dict(ab=wl.FP8_E5M2, cd=wl.BF16, epi=bg.EPI_BIAS, ldc=40), dict(variant=VS)),
    ("fp8_e4m3_stream_k_one_slice", 16, 384, 2048, dict(ab=wl.FP8_E4M3), dict(variant=VS, kslices=1)),
    ("fp8_e4m3_stream_k_auto", 8, 4096, 4096, dict(ab=wl.FP8_E4M3), dict()),
    # tail split: the tiles of a thinly filled last wave are cut into K slices whose raw accumulators meet in the workspace
    ("tail_split_pair_few_tiles", 1024, 1024, 2048, dict(cd=wl.BF16), dict(variant=V2, tile_n=256, tail_split=True)),
    ("tail_split_pair_after_full_wave", 2560, 2560, 1032, dict(beta=1.0, epi=bg.EPI_BIAS_RELU, cd=wl.BF16), dict(variant=V2, tile_n=256, tail_split=True)),
    ("tail_split_pair_narrow_f32", 1024, 1200, 1024, dict(epi=bg.EPI_BIAS), dict(variant=V2, tile_n=128, tail_split=True)),
    ("tail_split_1cta", 512, 512, 2048, dict(), dict(variant=V1, tile_n=128, tail_split=True)),
    ("tail_split_1cta_ragged_f16", 1000, 1000, 1096, dict(ab=wl.F16, cd=wl.F16, beta=-1.0), dict(variant=V1, tile_n=256, tail_split=True)),
    ("tail_split_1cta_two_epilogue_groups", 1280, 4096, 512, dict(cd=wl.BF16), dict(variant=V1, tile_n=256, tail_split=True)),
    ("tail_split_nn_layout", 1024, 1024, 2048, dict(ta=0, tb=0), dict(variant=V2, tile_n=128, tail_split=True)),
    ("tail_split_fp8", 1024, 1024, 4096, dict(ab=wl.FP8_E4M3, cd=wl.BF16), dict(variant=V2, tile_n=256, tail_split=True)),
    ("tail_split_seven_slices_long_k", 512, 512, 16384, dict(cd=wl.BF16, epi=bg.EPI_BIAS), dict(variant=V2, tile_n=256)),
    ("tail_split_1cta_three_slices", 256, 384, 8192 + 64, dict(beta=1.0), dict(variant=V1, tile_n=128, tail_split=True)),
    ("tail_split_automatic_for_few_tiles", 300, 264, 32768, dict(), dict()),
    ("tail_split_switched_off", 1024, 1024, 2048, dict(cd=wl.BF16), dict(variant=V2, tile_n=256)),
    ("tail_split_requested_auto_plan", 2304, 2304, 2304, dict(cd=wl.BF16), dict(tail_split=True)),
    # one triangle of D wanted (symmetric results): tiles wholly in the other triangle are left out of the schedule
    ("d_lower_1cta", 700, 700, 200, dict(d_tri=1), dict(variant=V1, tile_n=128)),
    ("d_upper_1cta", 700, 700, 200, dict(d_tri=2), dict(variant=V1, tile_n=128)),
    ("d_lower_pair_wide_tiles", 1104, 1104, 264, dict(d_tri=1, cd=wl.BF16), dict(variant=V2, tile_n=256)),
    ("d_upper_pair_narrow_tiles", 1104, 1104, 264, dict(d_tri=2), dict(variant=V2, tile_n=64)),
    ("d_lower_tile_n_192_raster_2", 900, 1000, 136, dict(d_tri=1), dict(variant=V1, tile_n=192, raster=2)),
    ("d_lower_m_longer", 1500, 400, 136, dict(d_tri=1), dict(variant=V1, tile_n=128)),
    ("d_upper_m_longer", 1500, 400, 136, dict(d_tri=2), dict(variant=V2, tile_n=128)),
    ("d_lower_n_longer", 400, 1500, 136, dict(d_tri=1), dict(variant=V2, tile_n=128)),
    ("d_upper_n_longer", 400, 1500, 136, dict(d_tri=2), dict(variant=V1, tile_n=256)),
    ("d_lower_batched_beta_bias", 304, 304, 136, dict(d_tri=1, batch=5, beta=1.0, epi=bg.EPI_BIAS_RELU, cd=wl.BF16), dict(variant=V1, tile_n=64)),
    ("d_upper_batched_pair", 520, 520, 72, dict(d_tri=2, batch=3, ab=wl.F16, cd=wl.F16), dict(variant=V2, tile_n=128)),
    ("d_lower_one_tile", 100, 100, 64, dict(d_tri=1), dict(variant=V1)),
    ("d_lower_nn_layout", 704, 704, 200, dict(d_tri=1, ta=0, tb=0), dict(variant=V2, tile_n=128)),
    ("d_lower_with_lower_a", 768, 768, 768, dict(d_tri=1, a_tri=1), dict(variant=V2, tile_n=128)),
    ("d_lower_fp8", 704, 704, 528, dict(d_tri=1, ab=wl.FP8_E4M3, cd=wl.BF16), dict(variant=V2, tile_n=256)),
    ("d_lower_two_epilogue_groups", 2048, 2048, 256, dict(d_tri=1, cd=wl.BF16), dict(variant=V1, tile_n=256)),
    ("d_lower_auto", 2304, 2304, 520, dict(d_tri=1, cd=wl.BF16), dict()),
    ("d_upper_auto_tail_split_requested", 1024, 1024, 2048, dict(d_tri=2), dict(tail_split=True)),
    # triangular op(B): K ranges cut from the column side; with a triangular op(A) and the matching triangle of D this
    # is the product of two triangular matrices
    ("b_upper_1cta", 520, 700, 712, dict(b_tri=2), dict(variant=V1, tile_n=128)),
    ("b_lower_1cta", 520, 700, 712, dict(b_tri=1), dict(variant=V1, tile_n=64)),
    ("b_upper_pair_k_shorter", 520, 1000, 328, dict(b_tri=2), dict(variant=V2, tile_n=256)),
    ("b_lower_pair_k_longer", 520, 456, 1000, dict(b_tri=1), dict(variant=V2, tile_n=128)),
    ("b_lower_stored_k_by_n", 264, 712, 520, dict(b_tri=1, tb=0), dict(variant=V1, tile_n=128)),
    ("b_upper_one_slice_stages_forward", 520, 712, 712, dict(b_tri=2), dict(variant=V2, tile_n=128, kslices=1, no_k_serpentine=True)),
    ("upper_times_upper", 1104, 1104, 1104, dict(a_tri=2, b_tri=2, d_tri=2, cd=wl.BF16), dict(variant=V2, tile_n=128)),
    ("lower_times_lower", 1104, 1104, 1104, dict(a_tri=1, b_tri=1, d_tri=1), dict(variant=V1, tile_n=128)),
    ("upper_times_upper_full_d", 712, 712, 712, dict(a_tri=2, b_tri=2), dict(variant=V2, tile_n=256)),
    ("lower_a_upper_b", 712, 712, 712, dict(a_tri=1, b_tri=2, epi=bg.EPI_BIAS, beta=1.0), dict(variant=V1, tile_n=128)),
    ("upper_times_upper_batched_fp8", 384, 384, 384, dict(a_tri=2, b_tri=2, d_tri=2, batch=3, ab=wl.FP8_E4M3), dict(variant=V1, tile_n=64)),
    ("upper_times_upper_auto", 2048, 2048, 2048, dict(a_tri=2, b_tri=2, d_tri=2, cd=wl.BF16), dict()),
    # symmetric result: the computed triangle copied into the other one (every element beyond the diagonal equals its mirror image)
    ("mirror_lower_1cta", 700, 700, 200, dict(d_tri=1, d_mirror=True), dict(variant=V1, tile_n=128)),
    ("mirror_upper_pair_bf16", 1104, 1104, 264, dict(d_tri=2, d_mirror=True, cd=wl.BF16), dict(variant=V2, tile_n=256)),
    ("mirror_lower_ragged_blocks_f16", 1000, 1000, 136, dict(d_tri=1, d_mirror=True, ab=wl.F16, cd=wl.F16, beta=1.0, epi=bg.EPI_BIAS), dict(variant=V2, tile_n=192)),
    ("mirror_upper_batched_padded", 200, 200, 72, dict(d_tri=2, d_mirror=True, batch=3, ldc=216, stride_c=200 * 216 + 64), dict(variant=V1, tile_n=64)),
    ("mirror_lower_tiny", 5, 5, 8, dict(d_tri=1, d_mirror=True, ldc=8), dict(variant=V1)),
    ("mirror_lower_auto_with_triangular_factors", 1536, 1536, 1536, dict(d_tri=1, a_tri=1, b_tri=1, d_mirror=True, cd=wl.BF16, sample_rows=96, sample_cols=96), dict()),
    # dealt schedules with empty slots in the middle of a CTA's sequence: more tiles than CTAs, not a multiple, batched
    ("d_lower_batched_two_rounds", 2304, 2304, 136, dict(d_tri=1, batch=2, cd=wl.BF16, sample_rows=96, sample_cols=96), dict(variant=V1, tile_n=128)),
    ("tri_upper_batched_two_rounds", 2304, 1152, 1160, dict(a_tri=2, batch=3, sample_rows=96, sample_cols=96), dict(variant=V1, tile_n=128)),
    ("upper_times_upper_pair_batched_rounds", 2560, 2560, 1288, dict(a_tri=2, b_tri=2, d_tri=2, batch=2, cd=wl.BF16, sample_rows=96, sample_cols=96), dict(variant=V2, tile_n=128)),
    # mirrored stream-K: a tall output with a handful of columns (A is the streamed operand)
    ("tall_one_unit", 128, 8, 64, {}, dict(variant=VS)),
    ("tall_split_k", 256, 8, 4096, {}, dict(variant=VS)),
    ("tall_ragged_beta", 1864, 8, 2136, dict(beta=1.0), dict(variant=VS)),
    ("tall_matrix_vector", 4096, 1, 4096, dict(ldb=4096, ldc=4), dict(variant=VS)),
    ("tall_n16_whole_tiles", 28672, 16, 1024, {}, dict(variant=VS)),
    ("tall_n33_bias_bf16", 1000, 33, 520, dict(cd=wl.BF16, epi=bg.EPI_BIAS, ldc=40), dict(variant=VS)),
    ("tall_n64_f16_bias_relu", 520, 64, 1032, dict(ab=wl.F16, cd=wl.F16, alpha=0.5, beta=1.0, epi=bg.EPI_BIAS_RELU), dict(variant=VS)),
    ("tall_auto_plan", 8192, 8, 2048, dict(beta=1.0), dict()),
]


@pytest.mark.parametrize("case", EXACT_CASES, ids=[c[0] for c in EXACT_CASES])
def test_exact_integer_inputs(case):
    name, M, N, K, kw, fl = case
    w = int_workload(name, M, N, K, **kw)
    _, info = H.check_workload(w, bg.make_flags(**fl), exact=True, repeats=2)
    if info["variant"] == VS and info["cluster_size"] > 1:
        # the plan handed the partial tiles over inside clusters: the same problem through the workspace as well
        _, info = H.check_workload(w, bg.make_flags(**fl), exact=True, repeats=2, options=bg.OPT_STREAMK_WORKSPACE)
        assert info["cluster_size"] == 1


def _random_case(seed):
    """A seeded random problem: variant, dtypes, storage orders, ragged extents with padded leading dimensions, batch,
    epilogue, scalars, structure flags and tuning fields all drawn independently (within what the ABI documents as
    supported together)."""
    rng = np.random.default_rng(1000 + seed)
    pick = lambda xs: xs[int(rng.integers(len(xs)))]
    variant = pick([0, 0, V1, V1, V2, V2, VW, VS])
    ab = pick([wl.BF16, wl.BF16, wl.F16, wl.FP8_E4M3, wl.FP8_E5M2])
    cd = pick([wl.F32, wl.BF16, wl.F16])
    fp8 = ab in (wl.FP8_E4M3, wl.FP8_E5M2)
    ta, tb = (0, 1) if (fp8 or variant == VS) else (int(rng.integers(2)), int(rng.integers(2)))
    if variant == VS:
        short, long_ = int(rng.integers(1, 65)), int(rng.integers(64, 1500))
        M, N = (short, long_) if rng.integers(2) else (long_, short)
        batch = 1
    else:
        M, N = int(rng.integers(1, 700)), int(rng.integers(1, 700))
        if variant == VW:
            M = max(M, 130)
        batch = pick([1, 1, 2, 3])
    K = int(rng.integers(1, 1100))
    while M * N * K * batch > 2.5e8:
        K = max(1, K // 2)
    ea = 16 if fp8 else 8                     # elements per 16 bytes
    ec = 4 if cd == wl.F32 else 8
    up = lambda x, m: -(-x // m) * m
    lda = up(M if ta else K, ea) + ea * int(rng.integers(0, 3))
    ldb = up(K if tb else N, ea) + ea * int(rng.integers(0, 3))
    ldc = up(N, ec) + ec * int(rng.integers(0, 3))
    kw = dict(ta=ta, tb=tb, ab=ab, cd=cd, batch=batch, lda=lda, ldb=ldb, ldc=ldc,
              alpha=pick([1.0, 1.0, 0.5, 2.0, -1.0]), beta=pick([0.0, 0.0, 1.0, -1.0, 0.5]))
    if batch > 1:   # strides: tight or padded by a multiple of 16 bytes
        kw["stride_a"] = (K if ta else M) * lda + ea * int(rng.integers(0, 5))
        kw["stride_b"] = (N if tb else K) * ldb + ea * int(rng.integers(0, 5))
        kw["stride_c"] = M * ldc + ec * int(rng.integers(0, 5))
    epi = int(rng.integers(0, 6 if variant == VW else 10))
    kw["epi"] = epi
    if variant != VW and (epi & 1) and rng.integers(3) == 0:
        kw["bias_per_row"] = True
    fl = dict(variant=variant)
    if variant in (0, V1, V2) and rng.integers(3) == 0:
        kw["a_tri"] = int(rng.integers(3))
        kw["b_tri"] = int(rng.integers(3))
        kw["d_tri"] = int(rng.integers(3))
    if variant in (V1, V2):
        fl["tile_n"] = pick([0, 64, 128, 192, 256] if not (variant == V2 and tb == 0) else [0, 128, 256])
        fl["kslices"] = pick([0, 1, 2])
        fl["tail_split"] = bool(rng.integers(2))
    if variant in (V1, V2, VW):
        fl["raster"] = pick([0, 0, 1, 3])
        fl["stages"] = pick([0, 0, 2, 3])
        fl["no_k_serpentine"] = bool(rng.integers(4) == 0)
    if variant == VS:
        fl["kslices"] = pick([0, 1, 2, 3])
    fl["no_early_launch"] = bool(rng.integers(4) == 0)
    return M, N, K, kw, fl


@pytest.mark.parametrize("seed", range(int(os.environ.get("B200GEMM_RANDOM_CASES", "64"))))   # (a longer sweep on request)
def test_random_problems(seed):
    """Integer-valued inputs: bit-exact wherever the epilogue keeps integers (none, bias, ReLU; alpha and beta are powers
    of two), the stated tolerance for the transcendental activations.  A combination the library documents as
    unsupported must be refused with that code, never run wrong."""
    for attempt in range(20):     # a refused draw is replaced by the next one, so that every seed runs a problem
        M, N, K, kw, fl = _random_case(seed + 100000 * attempt)
        w = int_workload(f"random_{seed}_{attempt}", M, N, K, **kw)
        try:
            # (stream-K draws alternate between the hand-over inside clusters, where the plan would use it, and the workspace)
            H.check_workload(w, bg.make_flags(**fl), exact=kw["epi"] <= 3, repeats=2, options=bg.OPT_STREAMK_WORKSPACE if seed % 2 else 0)
            return
        except bg.GemmError as e:
            assert e.status == bg.ERR_UNSUPPORTED, (M, N, K, kw, fl)
    pytest.fail("twenty draws in a row refused as unsupported")


@pytest.mark.parametrize("seed", range(int(os.environ.get("B200GEMM_RANDOM_STREAM_K_CASES", "24"))))
def test_random_stream_k_problems_with_long_k(seed):
    """Seeded stream-K problems with K long enough for every plan form -- equal ranges over all SMs, whole tiles, clusters,
    three tiles per four CTAs (odd seeds draw 74 ... 100 tiles) -- skinny and tall, all element types, ragged extents,
    run twice on a workspace that holds whatever earlier tests left in the allocator's memory.  (A sweep of this kind,
    240 draws, found the one stale workspace word in 10^8 that passed for a run's own; B200GEMM_RANDOM_STREAM_K_CASES
    makes it longer.)"""
    rng = np.random.default_rng(77000 + seed)
    pick = lambda xs: xs[int(rng.integers(len(xs)))]
    ab = pick([wl.BF16, wl.BF16, wl.F16, wl.FP8_E4M3])
    cd = pick([wl.F32, wl.BF16, wl.F16])
    short = int(rng.integers(1, 65))
    long_ = int(rng.integers(9400, 12900)) if seed % 2 else int(rng.integers(2000, 30000))
    M, N = (long_, short) if rng.integers(3) == 0 else (short, long_)
    ea, ec = (16 if ab == wl.FP8_E4M3 else 8), (4 if cd == wl.F32 else 8)
    up = lambda x, m: -(-x // m) * m
    K = up(int(rng.integers(512, 1200)) * 8, ea)
    kw = dict(ta=0, tb=1, ab=ab, cd=cd, lda=K + ea * int(rng.integers(0, 2)), ldb=K, ldc=up(N, ec) + ec * int(rng.integers(0, 3)),
              alpha=pick([1.0, 0.5, -1.0]), beta=pick([0.0, 1.0, -1.0]), epi=int(rng.integers(0, 4)))
    if (kw["epi"] & 1) and rng.integers(3) == 0:
        kw["bias_per_row"] = True
    w = int_workload(f"random_stream_k_{seed}", M, N, K, sample_rows=48, sample_cols=48, **kw)
    H.check_workload(w, bg.make_flags(VS, no_early_launch=bool(rng.integers(4) == 0)), exact=True, repeats=2,
                     options=bg.OPT_STREAMK_WORKSPACE if seed % 3 == 0 else 0)


@pytest.mark.parametrize("seed", range(int(os.environ.get("B200GEMM_RANDOM_SPLIT_CASES", "24"))))
def test_random_dense_problems_with_few_tiles(seed):
    """Seeded dense problems of the kinds whose plans cut tiles along K or use the widest tiles: a few tiles with a long K,
    a little more than one wave, cubes of 2-3 K; automatic and forced variants, every storage order, run twice."""
    rng = np.random.default_rng(88000 + seed)
    pick = lambda xs: xs[int(rng.integers(len(xs)))]
    variant = pick([0, 0, V1, V2, V2])
    ab = pick([wl.BF16, wl.BF16, wl.F16, wl.FP8_E4M3])
    cd = pick([wl.F32, wl.BF16, wl.F16])
    fp8 = ab == wl.FP8_E4M3
    if seed % 3 == 0:
        M, N, K = int(rng.integers(65, 1100)), int(rng.integers(65, 1100)), int(rng.integers(2048, 40000))
    elif seed % 3 == 1:
        M, N, K = int(rng.integers(1500, 4300)), int(rng.integers(1500, 4300)), int(rng.integers(256, 3000))
    else:
        M = N = int(rng.integers(2000, 3300))
        K = int(rng.integers(512, 3000))
    ta, tb = (0, 1) if fp8 else (int(rng.integers(2)), int(rng.integers(2)))
    ea, ec = (16 if fp8 else 8), (4 if cd == wl.F32 else 8)
    up = lambda x, m: -(-x // m) * m
    kw = dict(ta=ta, tb=tb, ab=ab, cd=cd, lda=up(M if ta else K, ea), ldb=up(K if tb else N, ea) + ea * int(rng.integers(0, 2)),
              ldc=up(N, ec) + ec * int(rng.integers(0, 3)), alpha=pick([1.0, 0.5, -1.0]), beta=pick([0.0, 1.0, -1.0]), epi=int(rng.integers(0, 4)))
    fl = dict(variant=variant, no_early_launch=bool(rng.integers(4) == 0))
    if variant in (V1, V2):
        fl["tail_split"] = bool(rng.integers(2))
        fl["tile_n"] = pick([0, 0, 64, 128, 256] if not (variant == V2 and tb == 0) else [0, 128, 256])
    w = int_workload(f"random_few_tiles_{seed}", M, N, K, sample_rows=48, sample_cols=48, **kw)
    try:
        H.check_workload(w, bg.make_flags(**fl), exact=True, repeats=2)
    except bg.GemmError as e:
        assert e.status == bg.ERR_UNSUPPORTED, (M, N, K, kw, fl)


@pytest.mark.parametrize("seed", range(int(os.environ.get("B200GEMM_RANDOM_LARGE_CASES", "32"))))
def test_random_large_problems(seed):
    """The same draw at sizes where every CTA computes many tiles (several waves, ring and accumulator buffers wrapping
    many times, multi-round dealt schedules): extents up to about 4000, checked on 48 seeded rows and columns plus the
    tile-boundary indices."""
    for attempt in range(20):     # a refused draw is replaced by the next one, so that every seed runs a problem
        rng = np.random.default_rng(9000 + seed + 100000 * attempt)
        M, N, K, kw, fl = _random_case(10000 + seed + 100000 * attempt)
        if fl["variant"] == VS:
            long_ = int(rng.integers(3000, 30000))
            M, N = (M, long_) if M <= 64 else (long_, N)
            K = int(rng.integers(256, 3000))
        else:
            M, N, K = int(rng.integers(600, 4200)), int(rng.integers(600, 4200)), int(rng.integers(64, 1600))
        fp8 = kw["ab"] in (wl.FP8_E4M3, wl.FP8_E5M2)
        ea, ec = (16 if fp8 else 8), (4 if kw["cd"] == wl.F32 else 8)
        up = lambda x, m: -(-x // m) * m
        kw.update(lda=up(M if kw["ta"] else K, ea) + ea, ldb=up(K if kw["tb"] else N, ea), ldc=up(N, ec) + ec)
        for k in ("stride_a", "stride_b", "stride_c"):
            kw.pop(k, None)
        if kw["batch"] > 1 and M * N > 4e6:
            kw["batch"] = 1
        w = int_workload(f"random_large_{seed}_{attempt}", M, N, K, sample_rows=48, sample_cols=48, **kw)
        try:
            H.check_workload(w, bg.make_flags(**fl), exact=kw["epi"] <= 3, options=bg.OPT_STREAMK_WORKSPACE if seed % 2 else 0)
            return
        except bg.GemmError as e:
            assert e.status == bg.ERR_UNSUPPORTED, (M, N, K, kw, fl)
    pytest.fail("twenty draws in a row refused as unsupported")


def test_padded_leading_dimensions_and_strides():
    w = int_workload("padded", 200, 328, 136, batch=3, cd=wl.BF16, beta=1.0,
                     lda=136 + 8, ldb=136 + 24, ldc=328 + 16,
                     stride_a=200 * 144 + 64, stride_b=328 * 160 + 8, stride_c=200 * 344 + 128)
    inputs = wl.make_inputs(w)
    cbits, _ = H.run_gpu(w, inputs, bg.make_flags(V1))
    reports = H.check_blocks(w, inputs, cbits, H.default_blocks(w))
    assert all(r["bit_identical"] == 1.0 for r in reports)
    # the padding of C must be untouched
    mask = np.ones(w.elems_c(), bool)
    idx = (np.arange(w.batch)[:, None, None] * w.stride_c + np.arange(w.M)[None, :, None] * w.ldc + np.arange(w.N)[None, None, :])
    mask[idx.ravel()] = False
    assert np.array_equal(cbits[mask], inputs["C"][mask])


def test_beta_zero_never_reads_c():
    # run_gpu pre-fills C with NaN when beta == 0; a finite, exact result proves C was not read
    for fl in (dict(variant=V1), dict(variant=V2, tile_n=128), dict(variant=VS)):
        M = 8 if fl["variant"] == VS else 300
        w = int_workload("nan_c", M, 264, 136)
        H.check_workload(w, bg.make_flags(**fl), exact=True)


def test_automatic_plan_choices_run():
    for M, N, K in [(512, 512, 512), (8, 4096, 2048), (96, 96, 96), (1000, 3000, 520)]:
        w = int_workload(f"auto_{M}x{N}x{K}", M, N, K)
        H.check_workload(w, 0, exact=True)


# ----------------------------------------------------------------------------- tolerance regime

@pytest.mark.parametrize("key", ["c2s", "c3s", "c4s", "c5s"])
@pytest.mark.parametrize("variant", [0, V1, V2, VW])
def test_small_replicas_of_the_configs(key, variant):
    w = wl.small_replicas()[key]
    if key == "c5s" and variant in (V2, VW):
        pytest.skip("M = 8 has no second tile row")
    H.check_workload(w, bg.make_flags(variant), repeats=2)
    if w.c_dtype != wl.F32:     # accumulator-domain check: same plan, fp32 output, Frobenius vs the unrounded oracle
        H.check_workload(w, bg.make_flags(variant), c_dtype=wl.F32)


def test_config_c1_full():
    w = wl.configs()["c1"]
    reports, info = H.check_workload(w, 0, repeats=3)
    assert reports[0]["n"] == 512 * 512
    assert reports[0]["max_err_over_tol"] < 1e-2      # fp32 accumulation sits orders of magnitude inside the bound


def _full_config(key, flags=0):
    w = wl.configs()[key]
    inputs = wl.make_inputs(w)
    cbits, info = H.run_gpu(w, inputs, flags)
    blocks = H.default_blocks(w)
    reports = H.check_blocks(w, inputs, cbits, blocks)
    H.assert_reports(reports, what=key)
    if w.c_dtype != wl.F32:
        for r in reports:
            assert r["max_ulp"] <= 1, r
        # accumulator-domain check on the sampled rows only (fp32 output of the same plan)
        cb32, _ = H.run_gpu(w, inputs, flags, c_dtype=wl.F32)
        rows_block = blocks[-2]
        rep32 = H.check_blocks(w, inputs, cb32, [rows_block], c_dtype=wl.F32)
        H.assert_reports(rep32, what=key + " fp32 output")
        assert rep32[0]["max_err_over_tol"] < 1e-2
    return reports, info


def test_config_c2_sampled_rows_and_columns():
    reports, info = _full_config("c2")
    assert info["tile_n"] == 256 and info["variant"] == VW     # the automatic choice for this shape


def test_config_c2_paired_ctas():
    _full_config("c2", bg.make_flags(V2, 256))


def test_config_c3_bias_gelu():
    _full_config("c3")


def test_config_c4_batched_fp16():
    reports, _ = _full_config("c4")
    assert len(reports) == 3      # whole batches, sampled rows, sampled columns


def test_config_c5_skinny_full():
    w = wl.configs()["c5"]
    reports, info = H.check_workload(w, 0, repeats=2)
    assert info["variant"] == VS and info["grid"] >= 100
    assert reports[0]["n"] == 8 * 28672
    assert reports[0]["max_err_over_tol"] < 1e-2


def test_gelu_epilogue_values():
    w = wl.Workload("gelu_probe", 256, 264, 136, transb=1, epilogue=bg.EPI_BIAS_GELU_ERF, c_dtype=wl.F32,
                    dist_a=wl.Dist("normal", 0, 1), dist_b=wl.Dist("normal", 0, 0.2), seed=99)
    reports, _ = H.check_workload(w, bg.make_flags(V1))
    assert reports[0]["frob"] < 1e-5


ACTIVATIONS = [bg.EPI_GELU_ERF, bg.EPI_BIAS_GELU_ERF, bg.EPI_GELU_TANH, bg.EPI_BIAS_GELU_TANH, bg.EPI_SILU, bg.EPI_BIAS_SILU]


@pytest.mark.parametrize("epi", ACTIVATIONS)
@pytest.mark.parametrize("shape", ["dense_1cta", "dense_pair", "stream_k", "stream_k_tall"])
def test_activation_epilogues(epi, shape):
    """Every transcendental activation on every kernel family, wide value range (|t| up to ~15), fp32 output:
    the stated per-element tolerance and a relative Frobenius error far below it."""
    M, N, K, fl = {"dense_1cta": (200, 264, 136, dict(variant=V1)), "dense_pair": (300, 264, 136, dict(variant=V2, tile_n=128)),
                   "stream_k": (8, 520, 1032, dict(variant=VS)), "stream_k_tall": (520, 8, 1032, dict(variant=VS))}[shape]
    w = wl.Workload(f"act_{shape}", M, N, K, transb=1, epilogue=epi, c_dtype=wl.F32, beta=0.5,
                    dist_a=wl.Dist("normal", 0, 1), dist_b=wl.Dist("normal", 0, 0.15), dist_bias=wl.Dist("normal", 0, 1.0), seed=7)
    reports, _ = H.check_workload(w, bg.make_flags(**fl))
    assert reports[0]["frob"] < 1e-5 and reports[0]["max_err_over_tol"] < 0.05


@pytest.mark.parametrize("case", [
    ("row_bias_1cta", 200, 328, 136, dict(epi=bg.EPI_BIAS), dict(variant=V1)),
    ("row_bias_pair_relu_bf16", 300, 264, 136, dict(epi=bg.EPI_BIAS_RELU, cd=wl.BF16), dict(variant=V2, tile_n=128)),
    ("row_bias_ragged_rows", 130, 64, 72, dict(epi=bg.EPI_BIAS, beta=1.0), dict(variant=V1)),
    ("row_bias_batched", 96, 72, 64, dict(epi=bg.EPI_BIAS, batch=3), dict(variant=V1)),
    ("row_bias_stream_k", 8, 520, 1032, dict(epi=bg.EPI_BIAS_RELU), dict(variant=VS)),
    ("row_bias_stream_k_tall", 520, 8, 1032, dict(epi=bg.EPI_BIAS, beta=1.0), dict(variant=VS)),
    ("row_bias_auto", 1024, 512, 256, dict(epi=bg.EPI_BIAS), dict()),
], ids=lambda c: c[0])
def test_bias_per_row_exact(case):
    name, M, N, K, kw, fl = case
    w = int_workload(name, M, N, K, bias_per_row=True, **kw)
    H.check_workload(w, bg.make_flags(**fl), exact=True, repeats=2)


def test_wide_kernel_refuses_what_its_epilogue_lacks():
    for kw in (dict(epilogue=bg.EPI_SILU), dict(epilogue=bg.EPI_BIAS_GELU_TANH), dict(epilogue=bg.EPI_BIAS, flags_extra=dict(bias_per_row=True))):
        extra = kw.pop("flags_extra", {})
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(bg.make_desc(1024, 1024, 4096, flags=bg.make_flags(VW, **extra), **kw))
        assert e.value.status == bg.ERR_UNSUPPORTED
    h = bg.gemm_plan(bg.make_desc(8192, 8192, 8192, c_dtype=bg.BF16, epilogue=bg.EPI_BIAS_SILU))   # the automatic plan goes elsewhere
    assert bg.gemm_plan_info(h)["variant"] == V2
    bg.gemm_destroy(h)


# ----------------------------------------------------------------------------- boundary behaviour on a device

def test_run_argument_errors_launch_nothing():
    plan = bg.Plan(bg.make_desc(256, 256, 64, epilogue=bg.EPI_BIAS))
    A = torch.zeros(256 * 64 + 8, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(256 * 64, dtype=torch.bfloat16, device="cuda")
    C = torch.zeros(256 * 256, dtype=torch.float32, device="cuda")
    bias = torch.zeros(256, dtype=torch.float32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_run(plan.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), 0, 1.0, 0.0, 0, 0, s)
    assert e.value.status == bg.ERR_NULL            # bias missing
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_run(plan.handle, A.data_ptr() + 2, B.data_ptr(), C.data_ptr(), bias.data_ptr(), 1.0, 0.0, 0, 0, s)
    assert e.value.status == bg.ERR_ALIGNMENT
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_run(plan.handle, 0, B.data_ptr(), C.data_ptr(), bias.data_ptr(), 1.0, 0.0, 0, 0, s)
    assert e.value.status == bg.ERR_NULL
    plan.close()
    sk = bg.Plan(bg.make_desc(8, 1024, 1024, flags=bg.make_flags(VS), options=bg.OPT_STREAMK_WORKSPACE))
    assert sk.workspace_bytes > 0
    X = torch.zeros(8 * 1024, dtype=torch.bfloat16, device="cuda")
    Wt = torch.zeros(1024 * 1024, dtype=torch.bfloat16, device="cuda")
    D = torch.zeros(8 * 1024, dtype=torch.float32, device="cuda")
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_run(sk.handle, X.data_ptr(), Wt.data_ptr(), D.data_ptr(), 0, 1.0, 0.0, 0, 0, s)
    assert e.value.status == bg.ERR_WORKSPACE
    small = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_run(sk.handle, X.data_ptr(), Wt.data_ptr(), D.data_ptr(), 0, 1.0, 0.0, small.data_ptr(), 64, s)
    assert e.value.status == bg.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert sk.status() == bg.OK
    sk.close()


def test_runs_on_a_side_stream():
    w = int_workload("side_stream", 300, 264, 136)
    inputs = wl.make_inputs(w)
    plan = bg.Plan(H.desc_of(w, bg.make_flags(V1)))
    A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
    C = torch.empty(w.elems_c(), dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        plan.run(A, B, C)
    side.synchronize()
    reports = H.check_blocks(w, inputs, H.to_host_bits(C, wl.F32), H.default_blocks(w))
    assert reports[0]["bit_identical"] == 1.0
    plan.close()


def test_runs_are_capturable_in_a_cuda_graph():
    """gemm_run only encodes tensor maps on the host and launches: after one ordinary run (which sets the kernel
    attributes) a chain of a dense, a stream-K and a mirrored symmetric GEMM is captured into a CUDA graph and replayed
    with new inputs."""
    w1 = int_workload("graph_dense", 512, 384, 256, cd=wl.BF16)
    w2 = int_workload("graph_stream_k", 8, 512, 4096, beta=0.0)
    w3 = int_workload("graph_symmetric", 520, 520, 264, cd=wl.BF16, d_tri=1, d_mirror=True)   # a dealt schedule and two kernels per run
    cases = []
    for w in (w1, w2, w3):
        inputs = wl.make_inputs(w)
        plan = bg.Plan(H.desc_of(w))
        A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
        C = torch.zeros(w.elems_c(), dtype=H._TORCH_DT[w.c_dtype], device="cuda")
        plan.run(A, B, C)                      # sets attributes, allocates the workspace
        cases.append((w, inputs, plan, A, B, C))
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _, _, plan, A, B, C in cases:
            plan.run(A, B, C)
    for seed_offset in (0, 1000):              # replay on the same buffers with fresh contents
        fresh = []
        for w, _, plan, A, B, C in cases:
            inp = wl.make_inputs(w, seed_offset=seed_offset)
            A.copy_(H.to_device(inp["A"], w.ab_dtype))
            B.copy_(H.to_device(inp["B"], w.ab_dtype))
            C.fill_(float("nan"))
            fresh.append(inp)
        g.replay()
        torch.cuda.synchronize()
        for (w, _, plan, A, B, C), inp in zip(cases, fresh):
            assert plan.status() == bg.OK
            reports = H.check_blocks(w, inp, H.to_host_bits(C, w.c_dtype), H.default_blocks(w))
            assert all(r["bit_identical"] == 1.0 for r in reports)
    for _, _, plan, *_ in cases:
        plan.close()


def test_one_plan_on_two_streams_with_a_workspace_per_stream():
    """Runs of one plan may overlap on the GPU when the runs that overlap use different workspaces: the hand-shake words
    (stream-K arrival words, tail-split flags) live in the workspace, and the runs share nothing but the status word.
    A dense plan without a workspace, a stream-K plan and a dense plan with a tail split, each launched alternately on
    two streams."""
    wd = int_workload("two_streams_dense", 1024, 1024, 512, cd=wl.BF16)
    ws = int_workload("two_streams_stream_k", 8, 11000, 8200, beta=0.0)   # (CTA ranges that straddle tiles: the workspace path)
    wt = int_workload("two_streams_tail_split", 1024, 1024, 2048, cd=wl.BF16)
    streams = [torch.cuda.Stream() for _ in range(2)]
    for w, flags in ((wd, 0), (ws, 0), (wt, bg.make_flags(V2, 256, tail_split=True))):
        inputs = wl.make_inputs(w)
        A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
        outs = [torch.empty(w.elems_c(), dtype=H._TORCH_DT[w.c_dtype], device="cuda") for _ in streams]
        plan = bg.Plan(H.desc_of(w, flags))
        assert (plan.workspace_bytes > 0) == (w is not wd)
        wss = [torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda") for _ in streams]
        torch.cuda.synchronize()
        for rep in range(4):                       # interleaved launches: the kernels of the two streams overlap
            for st, out, wsb in zip(streams, outs, wss):
                with torch.cuda.stream(st):
                    plan.run(A, B, out, workspace=wsb if plan.workspace_bytes else None)
        for st in streams:
            assert plan.status(st.cuda_stream) == bg.OK     # waits for that stream only
        for out in outs:
            reports = H.check_blocks(w, inputs, H.to_host_bits(out, w.c_dtype), H.default_blocks(w))
            assert all(r["bit_identical"] == 1.0 for r in reports)
        plan.close()


@pytest.mark.parametrize("fill", ["ones", "random", "zeros", "previous_plan"])
def test_workspace_needs_no_initialisation(fill):
    """The hand-shake words at the head of a workspace carry a per-run tag, so whatever the memory held before -- all
    bits set, random bytes, zeros, or the words another plan of the same shape left there -- reads as "nothing yet"."""
    cases = [(int_workload("ws_stream_k", 8, 11000, 8200, beta=1.0), 0),
             (int_workload("ws_stream_k_m40", 40, 10240, 8200, cd=wl.BF16), 0),
             (int_workload("ws_tail_split", 1024, 1024, 2048, cd=wl.BF16), bg.make_flags(V2, 256, tail_split=True)),
             (int_workload("ws_long_k_auto_split", 256, 256, 16384), 0)]
    for w, flags in cases:
        inputs = wl.make_inputs(w)
        A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
        plan = bg.Plan(H.desc_of(w, flags))
        assert plan.workspace_bytes > 0
        ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device="cuda")
        for rep in range(2):
            if fill == "ones":
                ws.fill_(0xFF)
            elif fill == "random":
                ws.copy_(torch.randint(0, 256, (ws.numel(),), dtype=torch.uint8, generator=torch.Generator().manual_seed(rep)).cuda())
            elif fill == "zeros":
                ws.zero_()
            elif fill == "previous_plan" and rep == 1:   # a second plan of the same shape inherits the first one's workspace
                plan.close()
                plan = bg.Plan(H.desc_of(w, flags))
            C = H.to_device(inputs["C"], w.c_dtype) if inputs["C"] is not None else \
                torch.full((w.elems_c(),), float("nan"), dtype=H._TORCH_DT[w.c_dtype], device="cuda")
            plan.run(A, B, C, alpha=w.alpha, beta=w.beta, workspace=ws)
            assert plan.status() == bg.OK
            reports = H.check_blocks(w, inputs, H.to_host_bits(C, w.c_dtype), H.default_blocks(w))
            assert all(r["bit_identical"] == 1.0 for r in reports), (w.name, fill, rep)
        plan.close()


def test_stale_words_that_look_like_small_counters_are_not_this_runs():
    """What a recycled workspace typically holds are small numbers next to zeros (16-bit floats of small integer value, old
    counters).  A run's tag must not be such a pattern: with tags built as `plan number << 24 | run number`, a stale word
    like 0x00005b00'00000007 passed for "plan 0x5b, run 0, seven arrivals" and one tile of a run was never finished.  Every
    word of the workspace is filled with k << 40 | count for k = 1 ... 400 in turn (the plans of a process are numbered from
    one), with a count that would make the first arrival look like the last or like one of many; each run must give the
    result of the run on a zeroed workspace."""
    cases = [(int_workload("stale_stream_k", 8, 11000, 4200, beta=1.0), 0, 3),   # grouped ranges: two contributors per tile
             (int_workload("stale_tail_split", 256, 256, 16384), 0, 0)]          # split-tile flags of the dense kernels
    for w, flags, count in cases:
        inputs = wl.make_inputs(w)
        A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
        plan = bg.Plan(H.desc_of(w, flags))
        assert plan.workspace_bytes > 0
        ws = torch.zeros(plan.workspace_bytes // 8, dtype=torch.int64, device="cuda")
        c0 = H.to_device(inputs["C"], w.c_dtype) if inputs["C"] is not None else torch.zeros(w.elems_c(), dtype=H._TORCH_DT[w.c_dtype], device="cuda")
        want = None
        runs = 0                                        # (the run number was the low half of such a tag)
        for k in range(0, 401):
            for shift in ((40, 24) if k else (0,)):     # the stream-K word (tag << 16 | count) and the flag word (the tag itself) of that scheme
                ws.fill_((k << shift) | (runs << (shift - 24)) | (count if shift == 40 else 0) if k else 0)
                C = c0.clone()
                plan.run(A, B, C, alpha=w.alpha, beta=w.beta, workspace=ws.view(torch.uint8))
                runs += 1
                if want is None:
                    assert plan.status() == bg.OK
                    want = C.clone()
                    reports = H.check_blocks(w, inputs, H.to_host_bits(C, w.c_dtype), H.default_blocks(w))
                    assert all(r["bit_identical"] == 1.0 for r in reports), w.name
                else:
                    assert torch.equal(C.view(torch.int16 if C.element_size() == 2 else torch.int32), want.view(torch.int16 if C.element_size() == 2 else torch.int32)), (w.name, k, shift)
        assert plan.status() == bg.OK
        plan.close()


def test_status_word_forms():
    """gemm_plan_status_async enqueues the read and waits for nothing; gemm_plan_status_result reports it once the
    caller has waited for the stream; gemm_plan_status_stream waits for one stream; gemm_plan_status for the device.
    A withheld producer arrival (test flag) makes the first run time out, and each form sees and clears the word."""
    w = int_workload("status_forms", 512, 512, 256)
    inputs = wl.make_inputs(w)
    A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
    C = torch.zeros(w.elems_c(), dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    for form in ("async", "stream", "device"):
        plan = bg.Plan(H.desc_of(w, bg.make_flags(V1, 128, debug_stall=True)))
        plan.set_timeout_ms(20)
        assert bg.gemm_plan_status_result(plan.handle) == bg.OK      # nothing fetched yet
        with torch.cuda.stream(side):
            plan.run(A, B, C)
            if form == "async":
                bg.gemm_plan_status_async(plan.handle, side.cuda_stream)
                done = torch.cuda.Event()
                done.record(side)
                done.synchronize()
                got = bg.gemm_plan_status_result(plan.handle)
            elif form == "stream":
                got = bg.gemm_plan_status_stream(plan.handle, side.cuda_stream)
            else:
                got = bg.gemm_plan_status(plan.handle)
        assert got == bg.ERR_TIMEOUT, form
        assert bg.gemm_plan_status_result(plan.handle) == bg.OK      # the result was taken
        assert bg.gemm_plan_status_stream(plan.handle, side.cuda_stream) == bg.OK   # and the device word cleared
        with torch.cuda.stream(side):
            plan.run(A, B, C)
            assert plan.status(side.cuda_stream) == bg.OK
        reports = H.check_blocks(w, inputs, H.to_host_bits(C, w.c_dtype), H.default_blocks(w))
        assert all(r["bit_identical"] == 1.0 for r in reports)
        plan.close()


def test_tensor_maps_are_remembered_by_operand_address():
    """A plan keeps the tensor maps of the operand addresses it has seen.  Alternating between buffers, moving to new
    ones and cycling through more addresses than the table holds must each give the result of the buffers passed."""
    w = int_workload("map_cache", 264, 328, 200, cd=wl.BF16)
    ws_ = int_workload("map_cache_stream_k", 8, 520, 1032)
    for wk in (w, ws_):
        plan = bg.Plan(H.desc_of(wk))
        sets = []
        for i in range(3):
            inp = wl.make_inputs(wk, seed_offset=10 * i)
            sets.append((inp, H.to_device(inp["A"], wk.ab_dtype), H.to_device(inp["B"], wk.ab_dtype)))
        C0 = torch.zeros(wk.elems_c(), dtype=H._TORCH_DT[wk.c_dtype], device="cuda")
        C1 = torch.zeros_like(C0)
        def check(inp, C):
            assert plan.status() == bg.OK
            reports = H.check_blocks(wk, inp, H.to_host_bits(C, wk.c_dtype), H.default_blocks(wk))
            assert all(r["bit_identical"] == 1.0 for r in reports)
        for rep in range(3):                      # same addresses again and again, in turn
            for (inp, A, B), C in zip(sets, (C0, C1, C0)):
                C.fill_(float("nan"))
                plan.run(A, B, C)
                check(inp, C)
        inp0, A0, B0 = sets[0]                    # A of one set with B of another: maps are kept per operand
        inp1, A1, B1 = sets[1]
        mixed = dict(inp0, B=inp1["B"])
        plan.run(A0, B1, C1)
        check(mixed, C1)
        # more distinct addresses than the table has entries (offsets into one large buffer), twice round
        n = 300
        stride = -(-wk.elems_c() // 64) * 64
        big = torch.zeros(n * stride, dtype=C0.dtype, device="cuda")
        for rnd in range(2):
            big.fill_(float("nan"))
            for i in range(n):
                plan.run(A0, B0, big[i * stride: i * stride + wk.elems_c()])
            assert plan.status() == bg.OK
            want = None
            for i in (0, 1, 127, 128, 129, 255, 256, n - 1):
                got = H.to_host_bits(big[i * stride: i * stride + wk.elems_c()], wk.c_dtype)
                if want is None:
                    check(inp0, big[:wk.elems_c()])
                    want = got
                assert np.array_equal(got, want), i
        plan.close()


@pytest.mark.parametrize("variant", [V1, V2, VW, VS, "stream-K through the workspace"])
def test_bounded_wait_reports_timeout_and_context_survives(variant):
    """A producer arrival is withheld by a test flag, so a device-side wait runs into its limit; the
    kernel must return on its own, the plan must report GEMM_ERR_TIMEOUT and later work must run."""
    # stream-K: split tiles, once handed over inside clusters and once through the workspace
    w = int_workload("stall", 8, 11000, 8200) if variant == "stream-K through the workspace" else \
        int_workload("stall", 8 if variant == VS else 512, 512, 256 if variant != VS else 8192)
    if variant == "stream-K through the workspace":
        variant = VS
    inputs = wl.make_inputs(w)
    tile_n = 0 if variant in (VW, VS) else 128
    plan = bg.Plan(H.desc_of(w, bg.make_flags(variant, tile_n, debug_stall=True)))
    plan.set_timeout_ms(20)
    A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
    C = torch.zeros(w.elems_c(), dtype=torch.float32, device="cuda")
    plan.run(A, B, C)
    torch.cuda.synchronize()
    plan.run(A, B, C)                      # before the status has been read: may give up early, must not hang or fault
    torch.cuda.synchronize()
    assert plan.status() == bg.ERR_TIMEOUT
    assert plan.status() == bg.OK          # reading clears the word
    # the hook acts on the first run only: the same plan must now give the exact result (for stream-K the arrival words
    # the abandoned runs left in the workspace carry those runs' tags and read as empty)
    for _ in range(2):
        C.fill_(float("nan"))
        plan.run(A, B, C)
        torch.cuda.synchronize()
        assert plan.status() == bg.OK
        reports = H.check_blocks(w, inputs, H.to_host_bits(C, w.c_dtype), H.default_blocks(w))
        assert all(r["bit_identical"] == 1.0 for r in reports)
    plan.close()
    H.check_workload(w, bg.make_flags(variant, tile_n), exact=True)


def test_tail_split_plans():
    """Which plans split, what they ask for, and that the flag switches it off."""
    def info(M, N, K, **fl):
        h = bg.gemm_plan(bg.make_desc(M, N, K, c_dtype=bg.BF16, flags=bg.make_flags(**fl)))
        i = bg.gemm_plan_info(h)
        bg.gemm_destroy(h)
        return i
    i = info(1024, 1024, 2048, variant=V2, tile_n=256, tail_split=True)     # 16 pair tiles on 74 pairs: three slices each
    # (one 64-bit flag word per partial tile at the head of the workspace, padded to 256 bytes, then the partial tiles)
    assert i["split"] == 3 and i["grid"] == 96 and i["workspace_bytes"] == 512 + 16 * 2 * 2 * 128 * 256 * 4
    i = info(1024, 1024, 1024, variant=V2, tile_n=256)                      # not asked for, and two slices at most: whole tiles, no workspace
    assert i["split"] == 1 and i["workspace_bytes"] == 0
    assert info(1024, 1024, 1024, variant=V2, tile_n=256, tail_split=True)["split"] == 2
    assert info(1024, 1024, 256, variant=V2, tile_n=256, tail_split=True)["split"] == 1      # too little K to slice
    assert info(3072, 3072, 3072, variant=V2, tile_n=256, tail_split=True)["split"] == 1     # 144 tiles: the last wave is 70 of 74
    i = info(2560, 2560, 2560, variant=V2, tile_n=256, tail_split=True)                      # 100 tiles: 74 + 26, the 26 in two slices
    assert i["split"] == 2 and i["workspace_bytes"] == 512 + 26 * 2 * 1 * 128 * 256 * 4
    assert info(16384, 14336, 4096, variant=V2, tile_n=256, tail_split=True)["split"] == 1   # 48 full waves: not worth it
    i = info(512, 512, 16384, variant=V2, tile_n=256)                                      # 4 tiles, 256 ring stages each: by itself
    assert i["split"] == 9 and i["grid"] == 72 and i["workspace_bytes"] == 512 + 4 * 2 * 8 * 128 * 256 * 4


@pytest.mark.parametrize("cd,N", [(wl.BF16, 900), (wl.F16, 899), (wl.F32, 901), (wl.F32, 5), (wl.BF16, 3)])
def test_output_is_a_column_block_of_a_larger_matrix(cd, N):
    """D is columns [c0, c0 + N) of a wider row-major matrix whose other columns hold live data; N times the element
    size is not a multiple of 16 bytes, so the last 16-byte unit of every row of D is shared with the neighbour.
    Every dense family (the wide pair kernel where it accepts the shape) must leave the neighbours bit for bit."""
    M, K, wide_cols = 300, 264, 1024
    c0 = 96
    w = int_workload("column_block", M, N, K, cd=cd, ldc=wide_cols, beta=1.0, epi=bg.EPI_BIAS_RELU)
    inputs = wl.make_inputs(w)
    A, B, bias = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype), H.to_device(inputs["bias"], wl.F32)
    esz = 4 if cd == wl.F32 else 2
    for fl in (dict(variant=V1), dict(variant=V2, tile_n=128), dict(variant=VS) if N <= 64 else dict(variant=V1, tile_n=256, tail_split=True), dict()):
        rng = np.random.default_rng(3)
        full = rng.integers(1, 60000, size=(M, wide_cols)).astype(inputs["C"].dtype)   # a matrix of other data (bit patterns) ...
        cin_rows = np.stack([inputs["C"][i * wide_cols: i * wide_cols + N] for i in range(M)])
        full[:, c0:c0 + N] = cin_rows                                                   # ... with C_in as its column block
        big = H.to_device(full.ravel(), cd)
        plan = bg.Plan(H.desc_of(w, bg.make_flags(**fl)))
        try:
            ws = plan.workspace(big.device)
            bg.gemm_run(plan.handle, A.data_ptr(), B.data_ptr(), big.data_ptr() + c0 * esz, bias.data_ptr(), float(w.alpha), float(w.beta),
                        0 if ws is None else ws.data_ptr(), 0 if ws is None else ws.numel(), torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
            assert plan.status() == bg.OK
        finally:
            plan.close()
        got = H.to_host_bits(big, cd).reshape(M, wide_cols)
        assert np.array_equal(got[:, :c0], full[:, :c0]) and np.array_equal(got[:, c0 + N:], full[:, c0 + N:]), fl
        # D itself: lay the block out as the workload describes it (row pitch wide_cols, starting at column c0)
        cbits = np.zeros(w.elems_c(), got.dtype)
        flat = got.ravel()[c0:]
        cbits[:flat.size] = flat
        reports = H.check_blocks(w, inputs, cbits, H.default_blocks(w))
        assert all(r["bit_identical"] == 1.0 for r in reports), fl


@pytest.mark.parametrize("fl,M,N", [(dict(variant=V1), 300, 264), (dict(variant=V2, tile_n=128), 300, 264), (dict(variant=VW), 600, 264),
                                    (dict(variant=VS), 8, 520), (dict(variant=VS), 520, 8)])
def test_non_finite_inputs_propagate_like_the_definition(fl, M, N):
    """A NaN and infinities in A: exactly the output elements the definition makes NaN or infinite are (with the sign the
    definition gives), every other element is untouched by them and within the usual tolerance."""
    K = 520
    w = wl.Workload("non_finite", M, N, K, transb=1, c_dtype=wl.F32, dist_a=wl.Dist("normal", 0, 1), dist_b=wl.Dist("normal", 0, 1), seed=21)
    inputs = wl.make_inputs(w)
    a = inputs["A"].reshape(M, K)
    b = inputs["B"].reshape(N, K)
    a[1, 7] = 0x7FC0                      # NaN: row 1 of D is NaN
    a[3, 100] = 0x7F80                    # +Inf: row 3 is +-Inf by the sign of B[:, 100] ...
    b[5, 100] = 0x0000                    # ... and NaN where that element of B is zero (Inf * 0)
    a[M - 1, 0] = 0x7F80
    a[M - 1, K - 1] = 0xFF80              # +Inf and -Inf in one row: NaN wherever the two products have opposite signs
    cbits, _ = H.run_gpu(w, inputs, bg.make_flags(**fl))
    got = cbits.reshape(M, N).astype(np.float64)
    y, bound = oracle.gemm(H.problem_of(w), inputs["A"], inputs["B"])
    y, bound = y[0], bound[0]
    assert np.array_equal(np.isnan(got), np.isnan(y))
    assert np.array_equal(np.isinf(got), np.isinf(y)) and np.array_equal(np.sign(got[np.isinf(y)]), np.sign(y[np.isinf(y)]))
    assert np.isnan(y[1]).all() and np.isinf(y[3, 0]) and np.isnan(y[3, 5]) and np.isnan(y[M - 1]).any()      # the cases are really there
    fin = np.isfinite(y)
    assert np.all(np.abs(got[fin] - y[fin]) <= H.REL_TOL * bound[fin] + H.ABS_TOL)


@pytest.mark.parametrize("ab", [wl.BF16, wl.F16])
def test_subnormal_inputs_are_not_flushed(ab):
    """A holds subnormal numbers of the input format, B large ones, so that every product is an ordinary number
    (2^-10): a tensor pipe that flushed subnormal operands to zero would return zeros.  Exact in fp32 (powers of two)."""
    small, large = (0x0001, 0x7D00) if ab == wl.BF16 else (0x0010, 0x6400)   # bf16: 2^-133 and 2^123; fp16: 2^-20 and 2^10
    for fl, M, N in ((dict(variant=V1), 200, 264), (dict(variant=V2, tile_n=128), 300, 264), (dict(variant=VW), 600, 264), (dict(variant=VS), 8, 520)):
        K = 64
        w = wl.Workload("subnormal", M, N, K, transb=1, ab_dtype=ab, c_dtype=wl.F32, seed=3)
        inputs = wl.make_inputs(w)
        inputs["A"][:] = small
        inputs["B"][:] = large
        cbits, _ = H.run_gpu(w, inputs, bg.make_flags(**fl))
        y, _ = oracle.gemm(H.problem_of(w), inputs["A"], inputs["B"])
        assert y[0, 0, 0] == K * 2.0 ** -10
        assert np.array_equal(cbits.reshape(M, N).astype(np.float64), y[0]), fl


def test_triangular_a_really_skips():
    """Lower-triangular A, 512 x 512: every kernel variant works on tile rows of at most 256 and ring stages of at most
    128 columns, so element (i, k) with k >= 256 (i // 256 + 1) lies in a stage no tile may visit.  NaN there must
    not reach the output; the diagonal stages are computed in full, so the zeros next to the diagonal are real zeros."""
    w = int_workload("tri_skip", 512, 264, 512, a_tri=1)
    inputs = wl.make_inputs(w)
    a = inputs["A"].reshape(512, 512)
    for i in range(512):
        a[i, 256 * (i // 256 + 1):] = 0x7FC0          # bf16 NaN
    for fl in (dict(variant=V1, tile_n=128), dict(variant=V2, tile_n=128), dict()):
        cbits, info = H.run_gpu(w, inputs, bg.make_flags(**fl))
        clean = wl.make_inputs(w)
        reports = H.check_blocks(w, clean, cbits, H.default_blocks(w))
        assert all(r["bit_identical"] == 1.0 and r["finite"] for r in reports), info
    for bad in (dict(variant=VS), dict(variant=VW)):     # these kernels have no K-range skipping: refused, not ignored
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(H.desc_of(int_workload("tri_refused", 8 if bad["variant"] == VS else 1024, 1024, 4096, a_tri=1), bg.make_flags(**bad)))
        assert e.value.status == bg.ERR_UNSUPPORTED


def test_triangular_b_really_skips():
    """Upper-triangular op(B), 512 x 512 (stored N x K): every kernel variant works on tile columns of at most 256 and
    ring stages of at most 128 elements of K, so element (k, j) with k >= 256 (j // 256 + 1) lies in a stage no tile
    may visit.  NaN there must not reach the output.  Upper times upper with the lower tiles of D below the diagonal
    computed all the same (full D): they come out as exact zeros."""
    w = int_workload("b_tri_skip", 264, 512, 512, b_tri=2)
    inputs = wl.make_inputs(w)
    bm = inputs["B"].reshape(512, 512)                    # row j holds op(B)[:, j]
    for j in range(512):
        bm[j, 256 * (j // 256 + 1):] = 0x7FC0             # bf16 NaN
    for fl in (dict(variant=V1, tile_n=128), dict(variant=V2, tile_n=128), dict()):
        cbits, info = H.run_gpu(w, inputs, bg.make_flags(**fl))
        clean = wl.make_inputs(w)
        reports = H.check_blocks(w, clean, cbits, H.default_blocks(w))
        assert all(r["bit_identical"] == 1.0 and r["finite"] for r in reports), info
    w = int_workload("upper_upper_zero_tiles", 1024, 1024, 1024, a_tri=2, b_tri=2)
    cbits, _ = H.run_gpu(w, wl.make_inputs(w), bg.make_flags(variant=V2, tile_n=128))
    got = cbits.reshape(1024, 1024)
    assert np.all(got[np.tril_indices(1024, -1)] == 0.0) and np.any(got[np.triu_indices(1024)] != 0.0)


@pytest.mark.parametrize("d_tri", [1, 2])
def test_triangular_d_leaves_the_other_tiles_alone(d_tri):
    """One triangle of D wanted: every output tile that lies wholly in the other triangle stays as it was (NaN poison
    here, and C_in when beta != 0), every wanted element is bit-exact, the plan reports fewer tiles than the full grid,
    and the kernels without a tile list refuse the flag."""
    for fl, M, N in ((dict(variant=V1, tile_n=128), 1000, 1000), (dict(variant=V2, tile_n=64), 1000, 1000), (dict(), 1300, 900)):
        for beta in (0.0, 1.0):
            w = int_workload("d_tri_skip", M, N, 200, d_tri=d_tri, beta=beta)
            inputs = wl.make_inputs(w)
            cbits, info = H.run_gpu(w, inputs, bg.make_flags(**fl))
            reports = H.check_blocks(w, inputs, cbits, H.default_blocks(w))
            H.assert_reports(reports, what=str(fl))
            assert reports[0]["bit_identical"] == 1.0
            tm, tn = info["tile_m"], info["tile_n"]
            rows_t, cols_t = -(-M // tm), -(-N // tn)
            got = cbits.reshape(M, N)
            init = None if beta == 0.0 else inputs["C"].reshape(M, N)
            skipped = 0
            for ti in range(rows_t):
                r0, r1 = ti * tm, min((ti + 1) * tm, M)
                for tj in range(cols_t):
                    c0, c1 = tj * tn, min((tj + 1) * tn, N)
                    outside = c0 > r1 - 1 if d_tri == 1 else r0 > c1 - 1
                    if outside:
                        skipped += 1
                        blk = got[r0:r1, c0:c1]
                        assert np.all(np.isnan(blk)) if init is None else np.array_equal(blk, init[r0:r1, c0:c1]), (fl, ti, tj)
            assert skipped > 0 and info["num_tiles"] == rows_t * cols_t - skipped, (info["num_tiles"], rows_t, cols_t, skipped)
    for bad, M in ((dict(variant=VS), 8), (dict(variant=VW), 1024)):
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(H.desc_of(int_workload("d_tri_refused", M, 1024, 4096, d_tri=d_tri), bg.make_flags(**bad)))
        assert e.value.status == bg.ERR_UNSUPPORTED
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_plan(H.desc_of(int_workload("d_tri_both", 256, 256, 64), bg.make_flags(d_lower=True, d_upper=True)))
    assert e.value.status == bg.ERR_INVALID_ARG


def test_symmetric_result_is_symmetric_everywhere():
    """D = A A^T, lower triangle computed and mirrored: the whole matrix against the oracle, equal to its transpose bit
    for bit, padding untouched; and the option is refused where it has no meaning."""
    w = wl.Workload("syrk_mirror", 900, 900, 520, transa=0, transb=1, c_dtype=wl.BF16, d_tri=1, d_mirror=True, ldc=912, seed=6)
    inputs = wl.make_inputs(w)
    inputs["B"] = inputs["A"].copy()
    cbits, _ = H.run_gpu(w, inputs, 0)
    H.assert_reports(H.check_blocks(w, inputs, cbits, H.default_blocks(w)), what="mirrored")
    full = cbits.reshape(900, 912)
    assert np.array_equal(full[:, :900], full[:, :900].T)
    assert np.all(full[:, 900:] == 0x7FC0) or np.all(np.isnan(oracle.decode(full[:, 900:].copy(), wl.BF16)))   # NaN poison of the padding
    # the symmetric product as a whole is the plain product: compare the mirrored half with the oracle as well
    plain = replace(w, d_tri=0, d_mirror=False)
    H.assert_reports(H.check_blocks(plain, inputs, cbits, H.default_blocks(plain)), what="against the plain product")
    for kw, st in ((dict(structure=bg.STRUCT_D_MIRROR), bg.ERR_INVALID_ARG),                                        # no triangle named
                   (dict(structure=bg.STRUCT_D_MIRROR, flags=bg.make_flags(d_lower=True), N=520), bg.ERR_INVALID_ARG)):  # not square
        d = dict(M=512, N=512, K=64)
        d.update(kw)
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(bg.make_desc(d.pop("M"), d.pop("N"), d.pop("K"), **d))
        assert e.value.status == st
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_plan(bg.make_desc(4096, 4096, 4096, flags=bg.make_flags(variant=VW, d_lower=True), structure=bg.STRUCT_D_MIRROR))
    assert e.value.status == bg.ERR_UNSUPPORTED


def test_triangular_d_general_values_symmetric_product():
    """D = A A^T with normally distributed A (the same buffer as both operands): the lower triangle meets the stated
    tolerance, and mirrors the upper triangle of a second run bit for bit (the product is symmetric and, with K walked
    forwards in every tile, both runs accumulate the same products in the same order)."""
    w = wl.Workload("syrk", 900, 900, 520, transa=0, transb=1, c_dtype=wl.F32, d_tri=1, seed=5)
    inputs = wl.make_inputs(w)
    inputs["B"] = inputs["A"].copy()
    fl = bg.make_flags(variant=V2, tile_n=256, no_k_serpentine=True)
    lo, _ = H.run_gpu(w, inputs, fl)
    H.assert_reports(H.check_blocks(w, inputs, lo, H.default_blocks(w)), what="lower")
    wu = replace(w, d_tri=2)
    up, _ = H.run_gpu(wu, inputs, fl)
    H.assert_reports(H.check_blocks(wu, inputs, up, H.default_blocks(wu)), what="upper")
    lo2, up2 = lo.reshape(900, 900), up.reshape(900, 900)
    il = np.tril_indices(900)
    assert np.array_equal(lo2[il], up2.T[il])


@pytest.mark.parametrize("ab", [wl.FP8_E4M3, wl.FP8_E5M2])
def test_fp8_operands_general_values(ab):
    """Normally distributed 8-bit operands (every product is exact in fp32; the sums are not): the stated per-element
    tolerance and a small Frobenius error against the fp64 oracle, on both dense families."""
    for fl in (dict(variant=V1), dict(variant=V2, tile_n=128)):
        w = wl.Workload("fp8_normal", 300, 264, 1040, transb=1, ab_dtype=ab, c_dtype=wl.F32, epilogue=bg.EPI_BIAS_GELU_TANH,
                        dist_a=wl.Dist("normal", 0, 1), dist_b=wl.Dist("normal", 0, 0.1), seed=11)
        reports, _ = H.check_workload(w, bg.make_flags(**fl))
        assert reports[0]["frob"] < 1e-5 and reports[0]["max_err_over_tol"] < 0.05


def test_fp8_refusals():
    for kw in (dict(transb=bg.OP_N), dict(transa=bg.OP_T)):                       # K-contiguous storage only
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_plan(bg.make_desc(256, 256, 256, ab_dtype=bg.FP8_E4M3, **kw))
        assert e.value.status == bg.ERR_UNSUPPORTED
    h = bg.gemm_plan(bg.make_desc(8, 4096, 4096, ab_dtype=bg.FP8_E4M3))             # short extent: stream-K with 128-wide K slices
    assert bg.gemm_plan_info(h)["variant"] == VS and bg.gemm_plan_info(h)["tile_k"] == 256
    bg.gemm_destroy(h)


# ----------------------------------------------------------------------------- measured plan selection

def _tune_case(w, iterations=5):
    inputs = wl.make_inputs(w)
    A, B = H.to_device(inputs["A"], w.ab_dtype), H.to_device(inputs["B"], w.ab_dtype)
    C = torch.zeros(w.elems_c(), dtype=H._TORCH_DT[w.c_dtype], device="cuda")
    desc = H.desc_of(w)
    plan, rep = bg.Plan.tuned(desc, A, B, C, iterations=iterations)
    return inputs, A, B, C, desc, plan, rep


def test_tune_times_candidates_keeps_the_fastest_and_remembers_it():
    bg.gemm_tune_cache_clear()
    w = int_workload("tune_dense", 1024, 1536, 512, cd=wl.BF16)
    inputs, A, B, C, desc, plan, rep = _tune_case(w)
    times = [t for _, t in rep["tried"]]
    assert rep["candidates_tried"] >= 5 and all(t > 0 for t in times)
    assert rep["tried"][0][0] == 0 and abs(rep["auto_ms"] - times[0]) < 1e-9          # the automatic plan is the yardstick
    assert abs(rep["best_ms"] - min(times)) < 1e-9 and rep["best_ms"] <= rep["auto_ms"]
    variants = {(f >> 4) & 0xF for f, _ in rep["tried"]}
    assert {V1, V2} <= variants                                                     # compute-side families were tried
    C.fill_(float("nan"))
    plan.run(A, B, C)
    torch.cuda.synchronize()
    assert plan.status() == bg.OK
    reports = H.check_blocks(w, inputs, H.to_host_bits(C, w.c_dtype), H.default_blocks(w))
    assert all(r["bit_identical"] == 1.0 for r in reports)
    keys = ("variant", "tile_m", "tile_n", "tile_k", "stages", "raster_group", "grid")
    again = bg.Plan(desc)                                                           # no tuning fields: the remembered choice
    assert {k: again.info[k] for k in keys} == {k: plan.info[k] for k in keys}
    forced = bg.Plan(H.desc_of(w, bg.make_flags(V1, 64)))                           # explicit fields still win
    assert forced.info["tile_n"] == 64
    for p in (again, forced, plan):
        p.close()
    bg.gemm_tune_cache_clear()


def test_tune_short_extent_tries_stream_k_and_dense():
    bg.gemm_tune_cache_clear()
    w = int_workload("tune_skinny", 8, 4096, 2048, beta=0.0)
    inputs, A, B, C, desc, plan, rep = _tune_case(w)
    variants = {(f >> 4) & 0xF for f, _ in rep["tried"]}
    assert VS in variants and V1 in variants
    C.fill_(float("nan"))
    plan.run(A, B, C)
    torch.cuda.synchronize()
    reports = H.check_blocks(w, inputs, H.to_host_bits(C, w.c_dtype), H.default_blocks(w))
    assert all(r["bit_identical"] == 1.0 for r in reports)
    plan.close()
    # a candidate the library refuses for this problem (the wide pair kernel has no SiLU epilogue) is skipped, not an error,
    # and the caller's own flags survive in the winner
    s = torch.cuda.current_stream().cuda_stream
    A2 = torch.zeros(1024 * 512, dtype=torch.bfloat16, device="cuda")
    C2 = torch.zeros(1024 * 1024, device="cuda")
    h, rep2 = bg.gemm_tune(bg.make_desc(1024, 1024, 512, epilogue=bg.EPI_SILU, flags=bg.make_flags(no_early_launch=True)),
                           A2.data_ptr(), A2.data_ptr(), C2.data_ptr(), 0, 1.0, 0.0, 0, 0, s, 3)
    assert rep2["candidates_skipped"] >= 1 and rep2["best_flags"] & 0x4
    bg.gemm_destroy(h)
    bg.gemm_tune_cache_clear()


def test_tuning_results_survive_in_a_file(tmp_path):
    """Save after tuning, forget, load: gemm_plan makes the tuned plan again.  A file from another GPU model is refused,
    a malformed one loads nothing, and a remembered choice that cannot be planned is ignored."""
    bg.gemm_tune_cache_clear()
    keys = ("variant", "tile_m", "tile_n", "tile_k", "stages", "raster_group", "grid")
    w = int_workload("tune_file", 1024, 1536, 512, cd=wl.BF16)
    inputs, A, B, C, desc, plan, rep = _tune_case(w)
    # a second shape with a forced, distinctive winner: remember "1-CTA, tile N 64, raster 3" for it by hand
    path = str(tmp_path / "tune.txt")
    assert bg.gemm_tune_cache_save(path) == 1
    lines = open(path).read().splitlines()
    assert lines[0].startswith("b200gemm-tune-1 ") and len(lines) == 2 and len(lines[1].split()) == 18
    odd = bg.make_flags(V1, 64, raster=3)
    fields = lines[1].split()
    fields[0:3] = ["640", "768", "256"]                        # M N K
    fields[7:10] = ["256", "256", "768"]                       # lda ldb ldc (tight, transb = T)
    fields[12:15] = ["0", "0", "0"]
    fields[17] = str(odd)
    with open(path, "a") as f:
        f.write(" ".join(fields) + "\n")
    bg.gemm_tune_cache_clear()
    auto = bg.Plan(desc)
    assert bg.gemm_tune_cache_load(path) == 2
    again = bg.Plan(desc)
    assert {k: again.info[k] for k in keys} == {k: plan.info[k] for k in keys}
    hand = bg.Plan(bg.make_desc(640, 768, 256, c_dtype=bg.BF16))
    assert (hand.info["variant"], hand.info["tile_n"], hand.info["raster_group"]) == (V1, 64, 3)
    w2 = int_workload("tune_file_hand", 640, 768, 256, cd=wl.BF16)
    H.check_workload(w2, exact=True)                           # runs through that remembered plan
    for p in (auto, again, hand, plan):
        p.close()
    # another GPU model / SM count: refused; nothing changes
    other = str(tmp_path / "other.txt")
    head = lines[0].split()
    open(other, "w").write(" ".join([head[0], head[1], str(int(head[2]) + 1)]) + "\n" + lines[1] + "\n")
    bg.gemm_tune_cache_clear()
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_tune_cache_load(other)
    assert e.value.status == bg.ERR_UNSUPPORTED
    # malformed: a short line, tuning bits outside the tuning fields, a wrong magic word, a missing file
    for text in (lines[0] + "\n" + lines[1] + "\n1 2 3\n", lines[0] + "\n" + " ".join(fields[:17] + ["1"]) + "\n", "something else\n"):
        bad = str(tmp_path / "bad.txt")
        open(bad, "w").write(text)
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_tune_cache_load(bad)
        assert e.value.status == bg.ERR_INVALID_ARG
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_tune_cache_load(str(tmp_path / "missing.txt"))
    assert e.value.status == bg.ERR_INVALID_ARG
    assert bg.gemm_tune_cache_save(str(tmp_path / "empty.txt")) == 0        # nothing was loaded by the failed attempts
    # a remembered choice this library cannot plan for the shape (the wide pair kernel has no SiLU epilogue): ignored
    fields[0:3] = ["1024", "1024", "512"]
    fields[7:10] = ["512", "512", "1024"]
    fields[11] = str(bg.EPI_SILU)
    fields[17] = str(bg.make_flags(VW))
    stale = str(tmp_path / "stale.txt")
    open(stale, "w").write(lines[0] + "\n" + " ".join(fields) + "\n")
    assert bg.gemm_tune_cache_load(stale) == 1
    p = bg.Plan(bg.make_desc(1024, 1024, 512, c_dtype=bg.BF16, epilogue=bg.EPI_SILU))
    assert p.info["variant"] != VW
    p.close()
    bg.gemm_tune_cache_clear()


def test_tune_keeps_structure_flags():
    """Measured plan selection on a structured problem (upper x upper -> upper, mirrored): the candidates keep the
    caller's structure words, the kernels that cannot honour them are skipped, and the tuned plan is exact."""
    bg.gemm_tune_cache_clear()
    w = int_workload("tune_structured", 1104, 1104, 1104, cd=wl.BF16, a_tri=2, b_tri=2, d_tri=2, d_mirror=True)
    inputs, A, B, C, desc, plan, rep = _tune_case(w)
    assert rep["candidates_skipped"] >= 1 and rep["best_flags"] & 0x8000 and rep["best_flags"] & 0x800000     # D_UPPER, A_UPPER survive
    C.fill_(float("nan"))
    plan.run(A, B, C)
    torch.cuda.synchronize()
    assert plan.status() == bg.OK
    got = H.to_host_bits(C, w.c_dtype)
    reports = H.check_blocks(w, inputs, got, H.default_blocks(w))
    H.assert_reports(reports, what="tuned structured plan")
    assert all(r["bit_identical"] == 1.0 for r in reports)
    full = got.reshape(1104, 1104)
    assert np.array_equal(full, full.T)
    again = bg.Plan(desc)                       # the remembered choice is keyed by the structure word too
    assert again.info["variant"] == plan.info["variant"] and again.info["tile_n"] == plan.info["tile_n"]
    plain = bg.Plan(bg.make_desc(1104, 1104, 1104, c_dtype=bg.BF16))
    assert plain.info["flops"] > 1.9 * again.info["flops"]        # (the plain problem was not touched by the remembered choice)
    for p in (plan, again, plain):
        p.close()
    bg.gemm_tune_cache_clear()


def test_tune_argument_errors():
    d = bg.make_desc(256, 256, 64)
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_tune(d, 0, 16, 16, 0, 1.0, 0.0, 0, 0, 0)
    assert e.value.status == bg.ERR_NULL
    A = torch.zeros(256 * 64, dtype=torch.bfloat16, device="cuda")
    C = torch.zeros(256 * 256, device="cuda")
    with pytest.raises(bg.GemmError) as e:                                          # bias epilogue without a bias
        bg.gemm_tune(bg.make_desc(256, 256, 64, epilogue=bg.EPI_BIAS), A.data_ptr(), A.data_ptr(), C.data_ptr(), 0, 1.0, 0.0, 0, 0, 0)
    assert e.value.status == bg.ERR_NULL
    with pytest.raises(bg.GemmError) as e:                                          # short-extent shape whose automatic plan needs a workspace
        bg.gemm_tune(bg.make_desc(8, 256, 4096, options=bg.OPT_STREAMK_WORKSPACE), A.data_ptr(), A.data_ptr(), C.data_ptr(), 0, 1.0, 0.0, 0, 0, 0)
    assert e.value.status == bg.ERR_WORKSPACE                                       # (refused before anything runs)


# ----------------------------------------------------------------------------- host-resident operands

@pytest.mark.parametrize("case", [
    ("host_three_panels_beta_bias", 700, 328, 136, dict(beta=1.0, epi=bg.EPI_BIAS_RELU, cd=wl.BF16, ldc=328 + 24, lda=136 + 8), 3),
    ("host_default_panels_small", 100, 264, 72, dict(), 0),
    ("host_row_bias_nn", 1000, 136, 200, dict(epi=bg.EPI_BIAS, bias_per_row=True, tb=0), 4),
    ("host_skinny_panel", 40, 520, 1032, dict(beta=1.0), 1),
    ("host_fp8", 600, 264, 272, dict(ab=wl.FP8_E4M3, cd=wl.F16), 2),
    ("host_padded_b_nt", 300, 264, 136, dict(ldb=136 + 8, lda=136 + 16), 2),
    ("host_padded_b_nn", 300, 264, 136, dict(tb=0, ldb=264 + 24), 2),
], ids=lambda c: c[0])
def test_host_resident_gemm_exact(case):
    """gemm_host_run on pinned host buffers: bit-exact against the oracle, padding of the host C buffer untouched,
    and the same again on a second run of the same handle.  The pinned A and B buffers end with the last element of
    their last row (no padding behind it), so a copy that reads whole pitches past that point fails."""
    name, M, N, K, kw, panels = case
    w = int_workload(name, M, N, K, **kw)
    inputs = wl.make_inputs(w)
    pin = lambda a: None if a is None else torch.from_numpy(a).pin_memory()
    tight_a = (w.M - 1) * w.lda + w.K                                   # (host path: A is stored M x K)
    tight_b = (w.N - 1) * w.ldb + w.K if w.transb else (w.K - 1) * w.ldb + w.N
    hA, hB, hbias = pin(inputs["A"][:tight_a].copy()), pin(inputs["B"][:tight_b].copy()), pin(inputs["bias"])
    c_np = np.float32 if w.c_dtype == wl.F32 else np.uint16
    sentinel = np.full(w.elems_c(), 0x4321 if c_np == np.uint16 else 1234.5, c_np)
    handle = bg.gemm_host_create(H.desc_of(w), panels)
    try:
        want_panels = {3: 3, 0: 1, 4: 4, 1: 1, 2: 2}[panels]
        assert bg.gemm_host_panels(handle) == want_panels
        for _ in range(2):
            hC = pin(inputs["C"].copy() if inputs["C"] is not None else sentinel.copy())
            bg.gemm_host_run(handle, hA.data_ptr(), hB.data_ptr(), hC.data_ptr(), 0 if hbias is None else hbias.data_ptr(),
                             float(w.alpha), float(w.beta))
            got = hC.numpy()
            reports = H.check_blocks(w, inputs, got, H.default_blocks(w))
            assert all(r["bit_identical"] == 1.0 for r in reports)
            before = inputs["C"] if inputs["C"] is not None else sentinel
            mask = np.ones(w.elems_c(), bool)
            mask[(np.arange(w.M)[:, None] * w.ldc + np.arange(w.N)[None, :]).ravel()] = False
            assert np.array_equal(got[mask], before[mask])           # row padding of the host buffer is not written
    finally:
        bg.gemm_host_destroy(handle)


@pytest.mark.parametrize("seed", range(24))
def test_host_resident_random_problems(seed):
    """Seeded random problems through gemm_host_run: dtypes, storage order of B, ragged extents, padded pitches,
    epilogue, scalars and the number of row panels drawn independently; integer inputs, so bit-exact wherever the
    epilogue keeps integers."""
    rng = np.random.default_rng(5000 + seed)
    pick = lambda xs: xs[int(rng.integers(len(xs)))]
    ab = pick([wl.BF16, wl.BF16, wl.F16, wl.FP8_E4M3])
    cd = pick([wl.F32, wl.BF16, wl.F16])
    fp8 = ab == wl.FP8_E4M3
    tb = 1 if fp8 else int(rng.integers(2))
    M, N, K = int(rng.integers(1, 1800)), int(rng.integers(1, 500)), int(rng.integers(1, 700))
    ea, ec = (16 if fp8 else 8), (4 if cd == wl.F32 else 8)
    up = lambda x, m: -(-x // m) * m
    epi = int(rng.integers(0, 10))
    kw = dict(ta=0, tb=tb, ab=ab, cd=cd, lda=up(K, ea) + ea * int(rng.integers(0, 3)), ldb=up(K if tb else N, ea) + ea * int(rng.integers(0, 3)),
              ldc=up(N, ec) + ec * int(rng.integers(0, 3)), alpha=pick([1.0, 0.5, 2.0, -1.0]), beta=pick([0.0, 1.0, -1.0]), epi=epi)
    if (epi & 1) and rng.integers(2):
        kw["bias_per_row"] = True
    w = int_workload(f"host_random_{seed}", M, N, K, **kw)
    inputs = wl.make_inputs(w)
    pin = lambda a: None if a is None else torch.from_numpy(a).pin_memory()
    hA, hB, hbias = pin(inputs["A"]), pin(inputs["B"]), pin(inputs["bias"])
    c_np = np.float32 if w.c_dtype == wl.F32 else np.uint16
    sentinel = np.full(w.elems_c(), 0x4321 if c_np == np.uint16 else 1234.5, c_np)
    handle = bg.gemm_host_create(H.desc_of(w), int(rng.integers(0, 7)))
    try:
        assert 1 <= bg.gemm_host_panels(handle) <= max(1, -(-M // 256))
        hC = pin(inputs["C"].copy() if inputs["C"] is not None else sentinel.copy())
        bg.gemm_host_run(handle, hA.data_ptr(), hB.data_ptr(), hC.data_ptr(), 0 if hbias is None else hbias.data_ptr(),
                         float(w.alpha), float(w.beta))
        got = hC.numpy()
        reports = H.check_blocks(w, inputs, got, H.default_blocks(w))
        H.assert_reports(reports, what=w.name)
        if epi <= 3:
            assert all(r["bit_identical"] == 1.0 for r in reports), (M, N, K, kw)
        before = inputs["C"] if inputs["C"] is not None else sentinel
        mask = np.ones(w.elems_c(), bool)
        mask[(np.arange(w.M)[:, None] * w.ldc + np.arange(w.N)[None, :]).ravel()] = False
        assert np.array_equal(got[mask], before[mask])
    finally:
        bg.gemm_host_destroy(handle)


def test_host_resident_gemm_refusals():
    for kw in (dict(transa=bg.OP_T), dict(batch=2), dict(flags=bg.make_flags(a_lower=True))):
        with pytest.raises(bg.GemmError) as e:
            bg.gemm_host_create(bg.make_desc(256, 256, 256, **kw))
        assert e.value.status == bg.ERR_UNSUPPORTED
    h = bg.gemm_host_create(bg.make_desc(256, 256, 64, epilogue=bg.EPI_BIAS))
    buf = torch.zeros(256 * 256, dtype=torch.float32).pin_memory()
    with pytest.raises(bg.GemmError) as e:
        bg.gemm_host_run(h, buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), 0, 1.0, 0.0)
    assert e.value.status == bg.ERR_NULL
    bg.gemm_host_destroy(h)
    bg.gemm_host_destroy(0)

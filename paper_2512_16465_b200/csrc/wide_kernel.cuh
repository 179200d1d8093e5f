// Wide paired GEMM kernel for sm_100a: a cluster of two CTAs computes a 512 x 256 output tile.
//
// Why a second dense kernel: with the tensor pipe ~93 % busy the GPU sits at its power cap, and what
// separates kernels there is energy per FLOP.  Measured on 8192^3: dropping a quarter of the L2 -> SM
// operand traffic raises the sustained clock by ~9 %.  Operand bytes received per SM and per FLOP scale
// with (A rows + local B rows) / (CTA rows x tile columns): 256 / (128 x 256) for dense_gemm_kernel<2>,
// 384 / (256 x 256) here, i.e. 25 % less.
//
// Each CTA owns 256 rows (two 128-row halves, one TMEM lane set each) x 256 columns: the accumulator
// fills all 512 TMEM columns (half h in columns [256 h, 256 h + 256)), so there is no second accumulator
// buffer.  Overlap with the next tile comes from releasing early instead: the eight epilogue warps drain half 0
// first (per thread 128 columns: read, convert and pack in registers) and hand its TMEM columns back as soon as
// they are read; the MMA issuer starts the next tile on half 0 while half 1 is still being drained.
//
// Ring stage = 64 columns of K: A 256 x 64 (32 KB) + this CTA's half of B, 128 x 64 (16 KB); per stage the
// leader issues 8 tcgen05.mma.cta_group::2 (M 256, N 256, K 16: four per half) and one multicast commit.
// Three ring stages (144 KB) and two 4 KB staging slabs per epilogue warp (64 KB).
// Roles: warp 0 producer, warp 1 MMA issuer (leader CTA) and TMEM owner, warps 4-11 epilogue (two whole
// warpgroups; warps 2-3 only take part in the CTA-wide barriers).
#pragma once
#include "dense_kernel.cuh"

namespace b200 {

constexpr int kWideCtaM = 256;      // rows per CTA (two TMEM-lane halves)
constexpr int kWideTileN = 256;     // tile columns = columns of one accumulator half
constexpr int kWideThreads = 128 + 256;  // warps 0-1: producer, MMA issuer; warps 2-3: idle; warps 4-11: epilogue

// Conversions pinned in program order (volatile): the packed values of one 64-column part must exist before the
// next part's accumulators are loaded, otherwise both parts' raw accumulators are live at once.  (A 320-thread CTA
// gets at most 168 registers per thread; the epilogue below fits without spilling, and spills here cost
// microseconds per tile because their cache lines are long gone when the next tile ends.)
__device__ __forceinline__ uint32_t pack_bf16x2_pinned(float lo, float hi) {
  uint32_t d;
  asm volatile("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ uint32_t pack_f16x2_pinned(float lo, float hi) {
  uint32_t d;
  asm volatile("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// kFp8: 8-bit float operands (128 elements of K per 128-byte slice, tcgen05 kind::f8f6f4); otherwise 16-bit.
template <bool kFp8>
__device__ __forceinline__ void wide_producer_role(const DenseParams& p, const CUtensorMap* tmA, const CUtensorMap* tmB,
                                                   uint32_t tiles_base, uint32_t full0, uint32_t empty0, uint32_t cta_rank,
                                                   int cluster_id, int num_clusters, const WaitCtx& w) {
  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const uint32_t nstages = static_cast<uint32_t>(p.stages);
  const int b_groups = p.b_rows / 64;
  uint32_t s = 0, ph = 0, it = 0;
  bool stall_pending = (p.debug_flags & 1u) != 0u;
  const uint64_t pol = l2_policy_evict_normal();
  for (int tile = cluster_id; tile < p.num_tiles; tile += num_clusters, ++it) {
    const TileCoord tc = decode_tile_div(tile, p.tiles_m, p.tiles_n, p.raster_group);
    const int m0 = tc.tm * (2 * kWideCtaM) + static_cast<int>(cta_rank) * kWideCtaM;
    const int n0 = tc.tn * kWideTileN + static_cast<int>(cta_rank) * p.b_rows;
    const bool rev = p.k_serpentine && (it & 1u);  // see dense_kernel.cuh: re-use what L2 touched last
    constexpr int kSliceK = kFp8 ? 2 * kBlockK : kBlockK;
    int k0 = rev ? (p.num_kb - 1) * kSliceK : 0;
    const int dk = rev ? -kSliceK : kSliceK;
    for (int kb = 0; kb < p.num_kb; ++kb, k0 += dk) {
      if (!mbar_wait_warp(empty0 + 8u * s, ph ^ 1u, w, (1u << 8) | s)) return;
      if (stall_pending) {  // test hook: this stage is never filled nor signalled
        stall_pending = false;
      } else {
        const uint32_t full_local = full0 + 8u * s;
        const uint32_t bar = mapa(full_local, 0);
        const uint32_t sa = tiles_base + s * stage_bytes;
        const uint32_t sb = sa + p.a_stage_bytes;
        if (elect_one()) {
          if (cta_rank == 0) mbar_arrive_expect_tx(full_local, stage_bytes * 2u);
          if (p.a_kmajor) {
            tma_load_3d_pair(sa, tmA, bar, k0, m0, tc.batch, pol);  // one 64 x 256 box
          } else {
            for (int g = 0; g < kWideCtaM / 64; ++g) tma_load_3d_pair(sa + 8192u * g, tmA, bar, m0 + 64 * g, k0, tc.batch, pol);
          }
          if (p.b_kmajor) {
            tma_load_3d_pair(sb, tmB, bar, k0, n0, tc.batch, pol);
          } else {
            for (int g = 0; g < b_groups; ++g) tma_load_3d_pair(sb + 8192u * g, tmB, bar, n0 + 64 * g, k0, tc.batch, pol);
          }
        }
        __syncwarp();
      }
      if (++s == nstages) {
        s = 0;
        ph ^= 1u;
      }
    }
  }
}

template <bool kFp8>
__device__ __forceinline__ void wide_umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if constexpr (kFp8) umma_f8<2>(tmem_d, adesc, bdesc, idesc, accumulate);
  else umma_f16<2>(tmem_d, adesc, bdesc, idesc, accumulate);
}

template <bool kFp8>
__device__ __forceinline__ void wide_mma_role(const DenseParams& p, uint32_t tiles_base, uint32_t full0, uint32_t empty0,
                                              uint32_t tfull, uint32_t tempty0, uint32_t tmem_base, int cluster_id,
                                              int num_clusters, const WaitCtx& w) {
  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const uint32_t nstages = static_cast<uint32_t>(p.stages);
  const uint32_t stage16 = stage_bytes >> 4, ak16 = p.a_kstep >> 4, bk16 = p.b_kstep >> 4;
  const uint32_t half16 = (128u * 128u) >> 4;  // second 128-row half of the A tile: 16 KB further in either layout
  const uint64_t adesc0 = smem_desc(p.a_desc_hi, tiles_base);
  const uint64_t bdesc0 = smem_desc(p.b_desc_hi, tiles_base + p.a_stage_bytes);
  const uint32_t idesc = p.idesc;
  const int num_kb = p.num_kb;
  uint32_t s = 0, ph = 0, it = 0;
  uint64_t adesc = adesc0, bdesc = bdesc0;
  // At the start of a tile half 0 is handed back first (the epilogue is still converting its values when it
  // starts on half 1), so the first `lead` stages are issued for half 0 only, without releasing their ring slots;
  // half 1 then catches up on the same stages and releases them.  From there on both halves go stage by stage.
  const int lead = min(p.stages, num_kb);
  const int tail = min(p.stages, num_kb - lead);
  auto advance = [&](uint32_t& cs, uint32_t& cph, uint64_t& ca, uint64_t& cb) {
    ca += stage16;
    cb += stage16;
    if (++cs == nstages) {
      cs = 0;
      cph ^= 1u;
      ca = adesc0;
      cb = bdesc0;
    }
  };
  for (int tile = cluster_id; tile < p.num_tiles; tile += num_clusters, ++it) {
    const uint32_t eph = (it & 1u) ^ 1u;  // both halves were handed back once per earlier tile
    {
      uint32_t s0 = s, ph0 = ph;
      uint64_t a0 = adesc, b0 = bdesc;
      if (!mbar_wait_warp(tempty0, eph, w, (2u << 8) | 0x80u)) return;
      for (int kb = 0; kb < lead; ++kb) {
        if (!mbar_wait_warp(full0 + 8u * s0, ph0, w, (2u << 8) | s0)) return;
        tc_fence_after();
        if (elect_one()) {
          wide_umma<kFp8>(tmem_base, a0, b0, idesc, static_cast<uint32_t>(kb != 0));
#pragma unroll
          for (uint32_t k = 1; k < kBlockK / kUmmaK; ++k) wide_umma<kFp8>(tmem_base, a0 + k * ak16, b0 + k * bk16, idesc, 1u);
        }
        __syncwarp();
        advance(s0, ph0, a0, b0);
      }
      if (!mbar_wait_warp(tempty0 + 8u, eph, w, (2u << 8) | 0x81u)) return;
      tc_fence_after();
      for (int kb = 0; kb < lead; ++kb) {
        if (elect_one()) {
          wide_umma<kFp8>(tmem_base + kWideTileN, adesc + half16, bdesc, idesc, static_cast<uint32_t>(kb != 0));
#pragma unroll
          for (uint32_t k = 1; k < kBlockK / kUmmaK; ++k)
            wide_umma<kFp8>(tmem_base + kWideTileN, adesc + half16 + k * ak16, bdesc + k * bk16, idesc, 1u);
          umma_commit_pair_mcast(empty0 + 8u * s, 3);  // ring slot free in both CTAs once both halves have read it
        }
        __syncwarp();
        advance(s, ph, adesc, bdesc);
      }
    }
    for (int kb = lead; kb < num_kb - tail; ++kb) {
      if (!mbar_wait_warp(full0 + 8u * s, ph, w, (2u << 8) | s)) return;
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (uint32_t k = 0; k < kBlockK / kUmmaK; ++k) wide_umma<kFp8>(tmem_base, adesc + k * ak16, bdesc + k * bk16, idesc, 1u);
#pragma unroll
        for (uint32_t k = 0; k < kBlockK / kUmmaK; ++k)
          wide_umma<kFp8>(tmem_base + kWideTileN, adesc + half16 + k * ak16, bdesc + k * bk16, idesc, 1u);
        umma_commit_pair_mcast(empty0 + 8u * s, 3);
      }
      __syncwarp();
      advance(s, ph, adesc, bdesc);
    }
    // Mirror image at the end of the tile: the last `tail` stages are issued for half 0 first, so half 0 completes
    // (and its read-out starts) while the tensor pipe is still busy with half 1's share of those stages.
    {
      uint32_t s0 = s, ph0 = ph;
      uint64_t a0 = adesc, b0 = bdesc;
      for (int kb = 0; kb < tail; ++kb) {
        if (!mbar_wait_warp(full0 + 8u * s0, ph0, w, (2u << 8) | s0)) return;
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (uint32_t k = 0; k < kBlockK / kUmmaK; ++k) wide_umma<kFp8>(tmem_base, a0 + k * ak16, b0 + k * bk16, idesc, 1u);
        }
        __syncwarp();
        advance(s0, ph0, a0, b0);
      }
      if (elect_one()) umma_commit_pair_mcast(tfull, 3);  // half 0 of the accumulator is complete
      __syncwarp();
      for (int kb = 0; kb < tail; ++kb) {
        if (elect_one()) {
#pragma unroll
          for (uint32_t k = 0; k < kBlockK / kUmmaK; ++k)
            wide_umma<kFp8>(tmem_base + kWideTileN, adesc + half16 + k * ak16, bdesc + k * bk16, idesc, 1u);
          umma_commit_pair_mcast(empty0 + 8u * s, 3);
        }
        __syncwarp();
        advance(s, ph, adesc, bdesc);
      }
      if (elect_one()) umma_commit_pair_mcast(tfull + 8u, 3);  // half 1 is complete
      __syncwarp();
    }
  }
}

__device__ __forceinline__ void wide_epilogue_role(const DenseParams& p, const CUtensorMap* tmD, uint32_t staging, uint32_t tfull,
                                                   uint32_t tempty0, uint32_t tmem_base, uint32_t cta_rank, int cluster_id,
                                                   int num_clusters, const WaitCtx& w) {
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t lane = lane_id();
  const uint32_t q = warp & 3u;          // TMEM lane quarter this warp may read
  const uint32_t ch = (warp - 4u) >> 2;  // which 128 columns of each half this warpgroup drains
  const uint32_t stg = staging + (warp - 4u) * (2u * kSlabBytes);  // two slabs per warp, used alternately
  const uint32_t sw = lane & 7u;
  uint32_t it = 0, nstore = 0;
  for (int tile = cluster_id; tile < p.num_tiles; tile += num_clusters, ++it) {
    const TileCoord tc = decode_tile_div(tile, p.tiles_m, p.tiles_n, p.raster_group);
    const int row_cta = tc.tm * (2 * kWideCtaM) + static_cast<int>(cta_rank) * kWideCtaM + static_cast<int>(q) * 32;
    const int colbase = tc.tn * kWideTileN + static_cast<int>(ch) * 128;
#pragma unroll 1
    for (uint32_t h = 0; h < 2; ++h) {
      if (!mbar_wait_warp(tfull + 8u * h, it & 1u, w, (3u << 8) | h, 64u)) return;
      tc_fence_after();
      const int row0 = row_cta + static_cast<int>(h) * 128;
      const long long row = row0 + static_cast<int>(lane);
      const uint32_t t_row = tmem_base + ((q * 32u) << 16) + h * kWideTileN + ch * 128u;
      float v[32];
      if (p.out_dtype == 2) {
        // fp32 output: 64 accumulator columns at a time; the half is handed back once its second part is read
#pragma unroll 1
        for (uint32_t part = 0; part < 2; ++part) {
          uint32_t acc0[32], acc1[32];
          tmem_ld_32x32(t_row + 64u * part, acc0);
          tmem_ld_32x32(t_row + 64u * part + 32u, acc1);
          tmem_ld_wait();
          if (part == 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa(tempty0 + 8u * h, 0));
          }
#pragma unroll
          for (int u = 0; u < 2; ++u, ++nstore) {
            const int col0 = colbase + 64 * static_cast<int>(part) + 32 * u;
            const uint32_t sbuf = stg + (nstore & 1u) * kSlabBytes;
            const uint32_t srow = sbuf + lane * 128u;
            if (lane == 0) bulk_wait_group_read<1>();  // the store that last read this slab has finished with it
            __syncwarp();
            epilogue_math<false>(v, u == 0 ? acc0 : acc1, p, row, col0, tc.batch);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              st_shared_v4(srow + ((static_cast<uint32_t>(j) ^ sw) << 4), __float_as_uint(v[4 * j]), __float_as_uint(v[4 * j + 1]),
                           __float_as_uint(v[4 * j + 2]), __float_as_uint(v[4 * j + 3]));
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (row0 < p.M && col0 < p.N) {
                if (p.l2_hint_d) tma_store_3d_hint(tmD, sbuf, col0, row0, tc.batch, l2_policy_evict_first());
                else tma_store_3d(tmD, sbuf, col0, row0, tc.batch);
              }
              bulk_commit_group();
            }
          }
        }
      } else {
        // 16-bit output: both 64-column parts are read, converted and packed (2 x 32 registers) before anything is
        // staged, so the half goes back to the MMA issuer a few hundred cycles after the accumulator is complete;
        // the two slabs are then written out without waiting on each other.
        uint32_t pk0[32], pk1[32];
        auto read_part = [&](const uint32_t part, uint32_t (&pk)[32]) {
          uint32_t acc0[32], acc1[32];
          tmem_ld_32x32(t_row + 64u * part, acc0);
          tmem_ld_32x32(t_row + 64u * part + 32u, acc1);
          tmem_ld_wait();
          if (part == 1u) {  // this thread's share of half h is in registers: hand the TMEM columns back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa(tempty0 + 8u * h, 0));
          }
          const int col64 = colbase + 64 * static_cast<int>(part);
          epilogue_math<false>(v, acc0, p, row, col64, tc.batch);
          if (p.out_dtype == 0) {
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2_pinned(v[2 * j], v[2 * j + 1]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[j] = pack_f16x2_pinned(v[2 * j], v[2 * j + 1]);
          }
          epilogue_math<false>(v, acc1, p, row, col64 + 32, tc.batch);
          if (p.out_dtype == 0) {
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[16 + j] = pack_bf16x2_pinned(v[2 * j], v[2 * j + 1]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[16 + j] = pack_f16x2_pinned(v[2 * j], v[2 * j + 1]);
          }
        };
        auto store_part = [&](const uint32_t part, const uint32_t (&pk)[32]) {
          const int col64 = colbase + 64 * static_cast<int>(part);
          const uint32_t sbuf = stg + (nstore & 1u) * kSlabBytes;
          const uint32_t srow = sbuf + lane * 128u;
          if (lane == 0) bulk_wait_group_read<1>();  // the store that last read this slab has finished with it
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            st_shared_v4(srow + ((static_cast<uint32_t>(j) ^ sw) << 4), pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (row0 < p.M && col64 < p.N) {
              if (p.l2_hint_d) tma_store_3d_hint(tmD, sbuf, col64, row0, tc.batch, l2_policy_evict_first());
              else tma_store_3d(tmD, sbuf, col64, row0, tc.batch);
            }
            bulk_commit_group();
          }
          ++nstore;
        };
        read_part(0u, pk0);
        read_part(1u, pk1);
        store_part(0u, pk0);
        store_part(1u, pk1);
      }
    }
  }
  if (lane == 0) bulk_wait_group_read<0>();
}
template <bool kFp8>
__global__ void __launch_bounds__(kWideThreads, 1)
wide_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmD, const DenseParams p) {
  extern __shared__ uint8_t smem_raw[];
  griddep_launch_dependents();  // the next kernel's set-up may overlap this one; it waits below before touching global memory
  const uint32_t raw = smem_addr(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t cta_rank = cluster_ctarank();
  const int cluster_id = static_cast<int>(blockIdx.x) / 2;
  const int num_clusters = static_cast<int>(gridDim.x) / 2;

  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const uint32_t staging_off = static_cast<uint32_t>(p.stages) * stage_bytes;
  const uint32_t bars_off = staging_off + 16u * kSlabBytes;
  const uint32_t full0 = base + bars_off;
  const uint32_t empty0 = full0 + 8u * kMaxStages;
  const uint32_t tfull = empty0 + 8u * kMaxStages;
  const uint32_t tempty0 = tfull + 16u;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + bars_off + 16u * kMaxStages + 32u);
  volatile uint32_t* s_abort = tmem_slot + 1;
  const WaitCtx w{s_abort, p.status, p.timeout_ns};

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, 1);
    }
    mbar_init(tfull, 1);          // accumulator half 0 complete
    mbar_init(tfull + 8u, 1);     // accumulator half 1 complete
    mbar_init(tempty0, 16);       // 8 epilogue warps in each CTA of the pair, per accumulator half
    mbar_init(tempty0 + 8u, 16);
    *s_abort = 0u;
    fence_mbar_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    prefetch_tensormap(&tmD);
  }
  if (warp == 1) {
    tmem_alloc<2>(smem_addr(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish<2>();
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();  // the peer's barriers must exist before anything signals them
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();  // barriers and tensor memory are set up; from here on global memory is read and written

  if (warp == 0) {
    wide_producer_role<kFp8>(p, &tmA, &tmB, base, full0, empty0, cta_rank, cluster_id, num_clusters, w);
  } else if (warp == 1) {
    if (cta_rank == 0) wide_mma_role<kFp8>(p, base, full0, empty0, tfull, tempty0, tmem_base, cluster_id, num_clusters, w);
  } else if (warp >= 4) {
    wide_epilogue_role(p, &tmD, base + staging_off, tfull, tempty0, tmem_base, cta_rank, cluster_id, num_clusters, w);
  }

  tc_fence_before();
  __syncthreads();
  cluster_arrive();  // neither CTA may free tensor memory or exit while its peer still uses the pair
  cluster_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<2>(tmem_base, 512);
  }
}

}  // namespace b200

// Skinny (memory-bound) GEMM for sm_100a: D[M x N] = act(alpha * X[M x K] * W[N x K]^T + beta * C + bias)
// with a handful of rows M.  The whole cost is streaming W from HBM once, so the kernel is built
// around the TMA stream, not around the tensor core:
//
//   * operands are swapped: a 128-row slab of W is the tcgen05.mma "A" operand (M_mma = 128), the
//     activations X, zero-padded by TMA to m_pad rows, are the "B" operand (N_mma = m_pad >= 16);
//     the accumulator is D^T: 128 TMEM lanes (output columns) x m_pad TMEM columns (output rows);
//   * stream-K: the (n-tile, k-block) work units, n-tile major, are cut into `grid` equal contiguous
//     ranges, one per CTA (one CTA per SM), so every SM streams the same number of bytes;
//   * a CTA whose range covers only part of a tile's K writes its fp32 partial to the workspace and
//     bumps the tile's arrival counter; the CTA that arrives last adds the partials in contributor
//     order (deterministic, no floating-point atomics), applies the epilogue, writes D and puts the
//     counter back to zero.  Nobody ever waits for another CTA.
//   * the counters live at the head of the caller's workspace and need no initialisation: a counter word is
//     (run tag << 16 | arrivals), the tag being unique to the run (plan identity and run number, never 0), and a
//     word that carries any other tag -- zeros, a timed-out run's leftovers, whatever the memory held before --
//     reads as "no arrivals yet".  Runs of one plan on different workspaces therefore share nothing but the
//     status word and may overlap.
//
//   * cluster mode (kCluster): when the plan gives every output tile to exactly c CTAs (c <= 8 dividing the tile's work
//     units), those c CTAs are launched as one thread-block cluster and the hand-over goes through shared memory instead:
//     each CTA parks its partial tile in its own (by then idle) ring memory, the cluster meets at a hardware barrier, and
//     every CTA finishes the 16-row chunks of the short extent that fall to its rank, adding the c partials in rank order
//     with loads from the peers' shared memory.  No workspace, no arrival word, no trip through L2; the order of the
//     additions is fixed, so results are bit-identical to the workspace path's.
//
// The same kernel serves the mirrored case, a tall output with a handful of columns (N <= 64 < M, kTall): the long
// operand A[M x K] then takes W's place and B[N x K] takes X's; only the addressing of C, D and the bias differs.
// Below, "big" is the long output extent (128 per tile, on the TMEM lanes) and "small" the short one.
//
// Roles per CTA (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and owner of the TMEM allocation
// (both warp-uniform, one elected lane issues), warps 2-5 = epilogue / fix-up.
#pragma once
#include <cuda_runtime.h>

#include <cstring>

#include "dense_kernel.cuh"
#include "launch_util.cuh"

namespace b200 {

constexpr int kSkinnyTileN = 128;   // output columns (rows of W) per tile = TMEM lanes
constexpr int kSkinnyMaxM = 64;     // largest M the skinny path takes
constexpr int kSkinnyThreads = 192;
constexpr int kSkinnyParkBytes = 80 * 128 * 4;  // 80 prefetched floats for each of the 128 epilogue threads

struct SkinnyPlan {
  int m_pad;             // small extent rounded up to a multiple of 16 (the MMA's N extent)
  int n_tiles;           // ceil(big extent / 128)
  int kblk;              // elements of K in one 128-byte slice: 64 (16-bit operands) or 128 (8-bit floats)
  int atoms;             // K slices per pipeline stage (each slice is one 128-byte swizzle atom per row)
  int kbs;               // work units per tile = ceil(K / (kblk * atoms))
  long long total_units; // n_tiles * kbs (< 2^31)
  int units_q, units_r;  // total_units = grid * units_q + units_r: the first units_r CTAs take units_q + 1 units
  int grid;              // CTAs = min(SM count, total_units)
  int stages;
  int stage_bytes;       // atoms x (16 KB of W + m_pad * 128 bytes of X)
  int smem_bytes;
  int cluster;           // > 1: CTAs per output tile, launched as one thread-block cluster (hand-over through shared memory)
  int group_tiles;       // t > 0: every t consecutive tiles are shared by t + 1 CTAs (see sk_group_begin); units_q / units_r unused
  int group_lead;        // work units by which a tile's tail is done before the CTA holding its head is
  int max_contributors;  // upper bound on CTAs touching one tile
  size_t counters_bytes; // arrival counters at the head of the workspace: n_tiles x u64, padded to 256 bytes
  size_t workspace_bytes;  // partial tiles behind them: grid * 2 slots of [m_pad][128] floats
};

// First work unit of CTA c, and the CTA that owns unit u (32-bit arithmetic: these run on the device's critical path).
__host__ __device__ inline int sk_begin(int c, int q, int r) { return c * q + (c < r ? c : r); }
__host__ __device__ inline int sk_owner(int u, int q, int r) {
  const int head = r * (q + 1);
  return u < head ? u / (q + 1) : r + (u - head) / q;
}

// Grouped ranges.  t tiles (t * kbs units) are shared by t + 1 CTAs in unit order: CTA 0 computes the head of tile 0,
// CTA i the tail of tile i - 1 and then the head of tile i, CTA t the tail of tile t - 1.  Every tile has two
// contributors, and the one holding the head finishes it from the other's partial tile, which it fetches ahead of
// time as soon as the arrival word says the partial is there (the cheap hand-over of the stream-K kernel).  That
// needs the tail to be done, published and fetched before the head is: with equal ranges it holds for every
// tile but the last, whose tail is CTA t's whole range and ends with everybody else's.  So CTA t takes
// t * (kbs - lead) / (t + 1) units, `lead` units short of an equal share plus its own head start, and the other t
// CTAs share the rest equally.  Returns the first unit, relative to the group, of CTA i (i = t + 1: the total).
__host__ __device__ inline int sk_group_begin(int kbs, int t, int lead, int i) {
  const int total = t * kbs;
  if (i > t) return total;
  const int rest = total - t * (kbs - lead) / (t + 1);
  const int q = rest / t, r = rest - q * t;
  return i * q + (i < r ? i : r);
}

// max_clusters (may be null): max_clusters[c] = clusters of c CTAs of this kernel that the device holds at once, c = 2 ... 8
// (without it: SM count / c, which real GPUs undercut for some sizes because a cluster must sit inside one GPC).
// M is the small output extent and N the big one (for a tall problem the caller passes them swapped).
inline bool skinny_make_plan(SkinnyPlan* s, int M, int N, int K, int sm_count, int forced_stages, int max_smem, int forced_atoms = 0,
                             int kblk = kBlockK, bool align = false, const int* max_clusters = nullptr, bool clusters = true) {
  if (M < 1 || M > kSkinnyMaxM) return false;
  s->m_pad = ((M + 15) / 16) * 16;
  s->n_tiles = (N + kSkinnyTileN - 1) / kSkinnyTileN;
  // Two adjacent 128-byte pieces of every weight row are requested together when K is long enough: DRAM then serves
  // both from one open row.
  s->kblk = kblk;
  const int fixed = 1024 + 16 * kMaxStages + 64 + kSkinnyParkBytes;
  const int slice_bytes = kSkinnyTileN * 128 + s->m_pad * 128;
  // ... as long as four such double stages fit (a short extent of 64 leaves room for three only: single slices, seven deep,
  // measured faster there)
  s->atoms = forced_atoms ? forced_atoms : ((K >= 16 * kblk && (max_smem - fixed) / (2 * slice_bytes) >= 4) ? 2 : 1);
  s->kbs = (K + kblk * s->atoms - 1) / (kblk * s->atoms);
  s->total_units = static_cast<long long>(s->n_tiles) * s->kbs;
  if (s->total_units > 0x7fffffffll) return false;
  s->grid = static_cast<int>(s->total_units < sm_count ? s->total_units : sm_count);
  // Grids that line up with the tiles.  The hand-over of partial tiles through the workspace costs a mid-sized problem as
  // much as the streaming itself (for a short extent of 64, 12 us of tail behind 7 us of streaming), so:
  //  (1) one whole tile per CTA, no hand-over at all, when that keeps two thirds of the SMs busy;
  //  (2) else c <= 8 CTAs per tile launched as one cluster each, the tile's units dealt to them as evenly as they go and
  //      the partial tiles added up through shared memory (about 2 us), when all clusters fit on the device at once and
  //      fill six tenths of it (any small problem: there the alternative is one CTA per unit);
  //  (3) else c > 8 CTAs per tile with c dividing the tile's units (workspace path, but no CTA contributes to two tiles),
  //      three tiles per four CTAs (grouped ranges, see sk_group_begin) when the tiles alone would keep between half
  //      and two thirds of the SMs busy, or several whole tiles per CTA;
  //  (4) else equal contiguous ranges over all SMs, straddling the tiles (the large problems, whose tail does not matter).
  // Measured against the plain rule (4) on shapes with short extents 8 ... 64: 64 x 4096 x 4096 22.3 -> 12.0 us,
  // 64 x 8192 x 8192 36.0 -> 27.7, 64 x 4096 x 14336 34.4 -> 24.3, 8 x 4096 x 4096 13.3 -> 10.7; the large ones unchanged.
  s->cluster = 1;
  s->group_tiles = 0;
  s->group_lead = 0;
  if (align) {
    int best = 0;
    const bool small_problem = s->total_units < 2ll * sm_count;
    const double streamed_mb = static_cast<double>(s->total_units) * s->atoms * (kSkinnyTileN * 128) / 1.0e6;
    if (s->total_units >= sm_count && s->n_tiles <= sm_count && s->n_tiles * 100 >= sm_count * 68) best = s->n_tiles;
    if (!best && clusters)
      for (int c = 2; c <= 8 && 2 * c <= s->kbs; ++c) {
        const int room = max_clusters ? max_clusters[c] : sm_count / c;
        if (s->n_tiles > room) continue;
        if (!small_problem && s->n_tiles * c * 10 < sm_count * 6) continue;
        if (s->n_tiles * c > best) {
          best = s->n_tiles * c;
          s->cluster = c;
        }
      }
    if (!best && s->total_units >= sm_count) {
      for (int c = clusters ? 9 : 3; c <= s->kbs; ++c)
        if (s->kbs % c == 0 && static_cast<long long>(s->n_tiles) * c <= sm_count && s->n_tiles * c * 5 >= sm_count * 4)
          best = best > s->n_tiles * c ? best : s->n_tiles * c;
      // About a hundred SMs saturate the memory system; 74 ... 100 tiles with one CTA each leave a quarter of the streaming
      // rate unused, and equal ranges over all SMs put three contributors on most tiles, all finishing at the same time
      // (the dear hand-over: publish, count, the last one fetches and adds, 8 ... 13 us at a short extent of 64).  Grouped
      // ranges use a third more CTAs than tiles and keep the cheap hand-over on every tile.  The lead (in work units) is
      // what a tail holder needs to publish its partial tile plus what the head holder needs to notice and fetch it
      // (measured 4 ... 6.5 us from 16 to 64 rows), at the rate a CTA streams: its share of some 6.5 TB/s, or what one
      // SM takes in alone (87 GB/s measured on 80 CTAs).
      if (!best && 2 * s->n_tiles >= sm_count && s->n_tiles + (s->n_tiles + 2) / 3 <= sm_count && s->kbs >= 32) {
        const int t = 3, left = s->n_tiles % t;
        const int grid = (s->n_tiles / t) * (t + 1) + (left ? left + 1 : 0);
        const double unit_w = s->atoms * (kSkinnyTileN * 128.0), unit_all = unit_w + s->atoms * (s->m_pad * 128.0);
        const double hbm = 6.5e6 / (grid * unit_w), one_sm = 87.0e3 / unit_all;  // work units per microsecond
        const double lead_us = 3.5 + 0.75 * (s->m_pad / 16);
        int lead = static_cast<int>(lead_us * (hbm < one_sm ? hbm : one_sm) + 0.999);
        lead = lead < 2 ? 2 : (lead > s->kbs / 4 ? s->kbs / 4 : lead);
        s->group_tiles = t;
        s->group_lead = lead;
        best = grid;
      }
      // (short K: whole tiles on half of the SMs, as long as the streamed operand is small; the wider the short extent, the
      // dearer the alternative)
      const double whole_tiles_up_to_mb = 160.0 + (s->m_pad > 32 ? (s->m_pad - 32) * 6.0 : 0.0);
      if (!best && s->n_tiles <= sm_count && 2 * s->n_tiles >= sm_count && streamed_mb <= whole_tiles_up_to_mb) best = s->n_tiles;
      if (!best && s->total_units / s->grid < 64)
        for (int t = 2; t <= s->n_tiles; ++t)
          if (s->n_tiles % t == 0 && s->n_tiles / t <= sm_count && (s->n_tiles / t) * 5 >= sm_count * 4) {
            best = s->n_tiles / t;
            break;
          }
    }
    if (best) s->grid = best;
  }
  s->units_q = static_cast<int>(s->total_units / s->grid);
  s->units_r = static_cast<int>(s->total_units % s->grid);
  s->stage_bytes = s->atoms * slice_bytes;
  int stages = forced_stages ? forced_stages : (max_smem - fixed) / s->stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (!forced_stages && stages * s->atoms > 8) stages = 8 / s->atoms > 3 ? 8 / s->atoms : 3;  // measured on B200: ~144 KB in flight per SM streams fastest
  if (stages < 2) return false;
  s->stages = stages;
  s->smem_bytes = fixed + stages * s->stage_bytes;
  if (s->smem_bytes > max_smem) return false;
  const int per_cta = s->units_q;  // >= 1
  s->max_contributors = s->group_tiles ? 2 : (s->kbs + per_cta - 1) / per_cta + 1;
  s->counters_bytes = (static_cast<size_t>(s->n_tiles) * 8 + 255) / 256 * 256;
  s->workspace_bytes = static_cast<size_t>(s->grid) * 2 * kSkinnyTileN * s->m_pad * 4;
  if (s->cluster > 1) s->counters_bytes = s->workspace_bytes = 0;  // nothing leaves the cluster
  // A short extent of 64 takes single slices above because four double stages do not fit.  That choice was measured with
  // every SM streaming; a grid that leaves SMs idle has fewer requests in flight and gains more from two adjacent
  // pieces per weight row than it loses with a ring of three (64 x 10240 x 8192 on 80 CTAs 41.7 -> 39.3 us,
  // 64 x 6144 x 6144 on 96 20.4 -> 19.9, 64 x 4096 x 4096 on 128 11.9 -> 11.6; on all 148 it costs 1 %).
  if (!forced_atoms && !forced_stages && s->atoms == 1 && s->grid < sm_count && K >= 16 * kblk && (max_smem - fixed) / (2 * slice_bytes) >= 3) {
    SkinnyPlan two;
    if (skinny_make_plan(&two, M, N, K, sm_count, 0, max_smem, 2, kblk, align, max_clusters, clusters) && two.grid < sm_count) *s = two;
  }
  return true;
}

// First work unit of CTA `cta` (cta = grid gives the total).  Cluster mode: the c CTAs of a cluster share out the units of
// their tile; otherwise all units are cut into `grid` equal contiguous ranges.
__host__ __device__ inline int sk_cta_begin(const SkinnyPlan& s, int cta) {
  if (s.cluster > 1) {
    const int tile = cta / s.cluster, rank = cta - tile * s.cluster;
    return tile * s.kbs + sk_begin(rank, s.kbs / s.cluster, s.kbs % s.cluster);
  }
  if (s.group_tiles > 0) {
    if (cta >= s.grid) return static_cast<int>(s.total_units);
    const int t = s.group_tiles, full = s.n_tiles / t;  // `full` whole groups, then one group of the n_tiles % t tiles left
    const int g = cta / (t + 1);
    if (g < full) return g * t * s.kbs + sk_group_begin(s.kbs, t, s.group_lead, cta - g * (t + 1));
    return full * t * s.kbs + sk_group_begin(s.kbs, s.n_tiles - full * t, s.group_lead, cta - full * (t + 1));
  }
  return sk_begin(cta, s.units_q, s.units_r);
}
// The CTA whose range holds work unit u (equal ranges or grouped ranges; not used in cluster mode).
__host__ __device__ inline int sk_unit_owner(const SkinnyPlan& s, int u) {
  if (s.group_tiles > 0) {
    const int t = s.group_tiles, full = s.n_tiles / t;
    int g = u / (t * s.kbs), tg = t;
    if (g >= full) {
      g = full;
      tg = s.n_tiles - full * t;
    }
    const int rel = u - g * t * s.kbs;
    int i = 0;
    while (i < tg && sk_group_begin(s.kbs, tg, s.group_lead, i + 1) <= rel) ++i;
    return g * (t + 1) + i;
  }
  return sk_owner(u, s.units_q, s.units_r);
}

struct SkinnyParams {
  SkinnyPlan plan;
  int M, N, K;
  uint32_t idesc;
  int out_dtype;
  int epilogue;
  int bias_per_row;       // the bias has M entries (one per output row) instead of N
  float alpha, beta;
  const float* bias;
  void* c;                // D buffer (also C_in when beta != 0), row-major M x N
  long long ldc;
  float* partials;        // workspace: slot-major, each slot [m_pad][128] floats
  unsigned long long* counters;  // one arrival word per n-tile: run tag << 16 | arrivals (any other tag reads as zero arrivals)
  unsigned long long tag;        // this run's tag (48 bits, never 0)
  uint32_t* status;
  unsigned long long timeout_ns;
  uint32_t debug_flags;   // bit 0: withhold one producer arrival (timeout test hook)
  int ab_fp8;             // operands are 8-bit floats (tcgen05 kind::f8f6f4)
  int n_full;             // columns of D covered by whole 16-byte units of a row (those leave through the copy engine; unused when tall)
};

// Count this CTA in on a tile's arrival word and return how many had arrived before it.  A word whose tag is not this
// run's counts as zero arrivals and is replaced.  Lock-free: an attempt fails only because another contributor's
// succeeded, so the loop ends after at most as many rounds as the tile has contributors; the limit is a backstop
// (0xffffffff = gave up, which the caller treats as "not the last").
__device__ __forceinline__ uint32_t sk_arrive(unsigned long long* word, unsigned long long tag) {
  unsigned long long cur = ld_relaxed_gpu_u64(word);
  for (int attempt = 0; attempt < 4096; ++attempt) {
    const bool mine = (cur >> 16) == tag;
    const unsigned long long want = mine ? cur + 1ull : ((tag << 16) | 1ull);
    const unsigned long long prev = atom_cas_acq_rel_gpu_u64(word, cur, want);
    if (prev == cur) return mine ? static_cast<uint32_t>(cur & 0xffffull) : 0u;
    cur = prev;
  }
  return 0xffffffffu;
}

// `big` is this thread's index along the long output extent, s0 the first of its 16 indices along the short one.
// D is row-major M x N: the short extent is M (rows) unless kTall.
template <bool kTall>
__device__ __forceinline__ long long sk_index(const SkinnyParams& p, int small, int big) {
  return kTall ? static_cast<long long>(big) * p.ldc + small : static_cast<long long>(small) * p.ldc + big;
}
// Fetch the 16 C_in values (zeros when beta == 0).  Kept apart from sk_values16 so that the loads can be issued
// before other long-latency loads, and before any store to the same buffer (C_in and D are one buffer: a load
// placed after a store could not be moved ahead of it and the rows would cost one round trip each).
template <bool kTall>
__device__ __forceinline__ void sk_load_cin16(const SkinnyParams& p, int s0, int big, bool big_ok, float (&cin)[16]) {
  const int small_extent = kTall ? p.N : p.M;
#pragma unroll
  for (int j = 0; j < 16; ++j) cin[j] = 0.0f;
  if (p.beta == 0.0f || !big_ok) return;
  const long long i0 = sk_index<kTall>(p, s0, big);
  const long long step = kTall ? 1 : p.ldc;
  if (p.out_dtype == 2) {  // (the type switch stays outside the loop, see sk_values16)
    const float* c = static_cast<const float*>(p.c) + i0;
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (s0 + j < small_extent) cin[j] = c[j * step];
  } else if (p.out_dtype == 0) {
    const __nv_bfloat16* c = static_cast<const __nv_bfloat16*>(p.c) + i0;
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (s0 + j < small_extent) cin[j] = __bfloat162float(c[j * step]);
  } else {
    const __half* c = static_cast<const __half*>(p.c) + i0;
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (s0 + j < small_extent) cin[j] = __half2float(c[j * step]);
  }
}
// The switches on activation and output type sit outside the loops over the 16 values: this code runs once per
// kernel, from a cold instruction cache, and a branch per value (each jumping over the inlined bodies of the other
// cases) cost hundreds of cycles per value in instruction fetches.
// sk_values16: bias, alpha / beta and the activation for 16 values along the short extent (`big_ok`: this thread's
// index along the long extent exists; otherwise nothing is read and the values are never written).
template <bool kTall>
__device__ __forceinline__ void sk_values16(const SkinnyParams& p, int s0, int big, bool big_ok, const float (&acc)[16],
                                            const float (&cin)[16], float (&v)[16]) {
  const int small_extent = kTall ? p.N : p.M;
  const bool has_bias = (p.epilogue & 1) != 0;
  // the bias runs along N (the long extent unless kTall) or, per row, along M
  const bool bias_along_big = kTall ? p.bias_per_row != 0 : p.bias_per_row == 0;
  if (has_bias && !bias_along_big) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = (s0 + j < small_extent) ? __ldg(p.bias + s0 + j) : 0.0f;
  } else {
    const float bias_big = (has_bias && big_ok) ? __ldg(p.bias + big) : 0.0f;
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = bias_big;
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) v[j] += p.alpha * acc[j] + p.beta * cin[j];
  const int act = p.epilogue >> 1;
  if (act == 1) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = fmaxf(v[j], 0.0f);
  } else if (act == 2) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = gelu_erf(v[j]);
  } else if (act == 3) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = gelu_tanh(v[j]);
  } else if (act == 4) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = silu(v[j]);
  }
}
// Plain stores of 16 finished values.  Tall: the 16 values are adjacent in a row of D (64 bytes as fp32), written as
// 16-byte pieces when all 16 exist (rows start on 16-byte boundaries, s0 is a multiple of 16).  Otherwise: one
// value per row of D.
template <bool kTall>
__device__ __forceinline__ void sk_store16(const SkinnyParams& p, int s0, int big, const float (&v)[16]) {
  const int small_extent = kTall ? p.N : p.M;
  const long long i0 = sk_index<kTall>(p, s0, big);
  const long long step = kTall ? 1 : p.ldc;  // from one of the 16 values to the next
  if (p.out_dtype == 2) {
    float* d = static_cast<float*>(p.c) + i0;
    if (kTall && s0 + 16 <= small_extent) {
#pragma unroll
      for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(d + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
      return;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (s0 + j < small_extent) d[j * step] = v[j];
  } else if (p.out_dtype == 0) {
    __nv_bfloat16* d = static_cast<__nv_bfloat16*>(p.c) + i0;
    if (kTall && s0 + 16 <= small_extent) {
      uint32_t w[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        w[j] = static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(v[2 * j]))) |
               (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(v[2 * j + 1]))) << 16);
      *reinterpret_cast<uint4*>(d) = make_uint4(w[0], w[1], w[2], w[3]);
      *reinterpret_cast<uint4*>(d + 8) = make_uint4(w[4], w[5], w[6], w[7]);
      return;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (s0 + j < small_extent) d[j * step] = __float2bfloat16_rn(v[j]);
  } else {
    __half* d = static_cast<__half*>(p.c) + i0;
    if (kTall && s0 + 16 <= small_extent) {
      uint32_t w[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        w[j] = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(v[2 * j]))) |
               (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(v[2 * j + 1]))) << 16);
      *reinterpret_cast<uint4*>(d) = make_uint4(w[0], w[1], w[2], w[3]);
      *reinterpret_cast<uint4*>(d + 8) = make_uint4(w[4], w[5], w[6], w[7]);
      return;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (s0 + j < small_extent) d[j * step] = __float2half_rn(v[j]);
  }
}
// Not tall: a warp holds 16 rows x 32 adjacent columns of D, one column per lane.  Stored from registers that is 16
// store instructions of 128 bytes each per warp, and issuing them took half a microsecond per 16 rows (measured: the
// four chunks of a 64-row tile 3.6 us with the stores, 1.6 us without).  Instead the warp writes the slab row-major
// into shared memory (`slab`, 16 x 32 elements) and one lane hands it to the copy engine as one tile store, which
// clips at the matrix bounds; the warp goes on at once.  The copy engine writes whole 16-byte units only, so the
// map ends at the last whole unit of a row (n_full) and the few columns behind it are stored from registers.
// Called by all 32 lanes together.  The slab may lie over this chunk's parked values, which every lane has read by
// the time of the first __syncwarp.
__device__ __forceinline__ void sk_stage16(const SkinnyParams& p, const CUtensorMap* tmD, uint32_t slab, uint32_t lane, int s0, int n,
                                           int col0, const float (&v)[16]) {
  __syncwarp();
  if (p.out_dtype == 2) {
#pragma unroll
    for (int j = 0; j < 16; ++j) st_shared_b32(slab + static_cast<uint32_t>(j) * 128u + lane * 4u, __float_as_uint(v[j]));
  } else if (p.out_dtype == 0) {
#pragma unroll
    for (int j = 0; j < 16; ++j) st_shared_b16(slab + static_cast<uint32_t>(j) * 64u + lane * 2u, __bfloat16_as_ushort(__float2bfloat16_rn(v[j])));
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j) st_shared_b16(slab + static_cast<uint32_t>(j) * 64u + lane * 2u, __half_as_ushort(__float2half_rn(v[j])));
  }
  fence_proxy_async_smem();
  __syncwarp();
  if (lane == 0 && col0 < p.n_full) {
    tma_store_3d(tmD, slab, col0, s0, 0);
    bulk_commit_group();
  }
  if (n >= p.n_full && n < p.N) sk_store16<false>(p, s0, n, v);
}

template <bool kTall, bool kCluster = false>
__global__ void __launch_bounds__(kSkinnyThreads, 1)
skinny_gemm_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmD,
                   const SkinnyParams p) {
  extern __shared__ uint8_t smem_raw[];
  griddep_launch_dependents();  // the next kernel's set-up may overlap this one; it waits below before touching global memory
  const uint32_t raw = smem_addr(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t lane = lane_id();
  const SkinnyPlan& sp = p.plan;
  const int small_extent = kTall ? p.N : p.M;
  const int big_extent = kTall ? p.M : p.N;

  const uint32_t bars_off = static_cast<uint32_t>(sp.stages) * sp.stage_bytes;
  const uint32_t full0 = base + bars_off;
  const uint32_t empty0 = full0 + 8u * kMaxStages;
  const uint32_t tfull0 = empty0 + 8u * kMaxStages;
  const uint32_t tempty0 = tfull0 + 16u;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + bars_off + 16u * kMaxStages + 32u);
  volatile uint32_t* s_abort = tmem_slot + 1;
  volatile uint32_t* s_last = tmem_slot + 2;
  volatile uint32_t* s_early = tmem_slot + 3;  // two words: a CTA has at most two partial segments (its first and its last)
  const WaitCtx w{s_abort, p.status, p.timeout_ns};
  // This CTA's contiguous range of work units (computed while the barriers and tensor memory are being set up).
  const int u_begin = sk_cta_begin(sp, static_cast<int>(blockIdx.x));
  const int u_end = sk_cta_begin(sp, static_cast<int>(blockIdx.x) + 1);
  const int tile0 = u_begin / sp.kbs;
  const int kb0 = u_begin - tile0 * sp.kbs;
  const int n_units = u_end - u_begin;
  const uint32_t tmem_cols = sp.m_pad * 2 <= 32 ? 32u : (sp.m_pad * 2 <= 64 ? 64u : 128u);

  if (threadIdx.x == 0) {
    for (int s = 0; s < sp.stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull0 + 8u * b, 1);
      mbar_init(tempty0 + 8u * b, 4);
    }
    *s_abort = 0u;
    fence_mbar_init();
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmX);
    if (!kTall) prefetch_tensormap(&tmD);
  }
  if (warp == 1) {
    tmem_alloc<1>(smem_addr(const_cast<uint32_t*>(tmem_slot)), tmem_cols);
    tmem_relinquish<1>();
  }
  // The producer needs the barriers (set up by its own lane 0) and nothing else: it announces them to the other
  // warps and starts streaming while those still wait for the tensor-memory allocation.
  uint32_t tmem_base = 0;
  if (warp == 0) {
    __syncwarp();
    named_barrier_arrive(3, kSkinnyThreads);
  } else {
    tc_fence_before();
    named_barrier_sync(3, kSkinnyThreads);
    tc_fence_after();
    tmem_base = *tmem_slot;
  }
  griddep_wait();  // from here on global memory is read and written
  // While the status word is set (an earlier run of this plan timed out and the host has not read the word yet) no
  // run finishes split tiles: a replay of a captured launch carries the tag of the run that may have left arrivals
  // half counted.  The load is issued here and consumed only by the fix-up, long after it has landed.
  // (Only the warps that finish tiles ask: the producer's first load must not queue behind it.)
  uint32_t stale_status = 0u;
  if (warp >= 2) stale_status = *reinterpret_cast<volatile const uint32_t*>(p.status);
  // Shared memory of the warps that finish tiles, 80 rows of 32 floats per warp (row v, lane l at + 128 v + 4 l): values
  // fetched ahead of their use are parked here, and finished 16 x 32 slabs of D are staged here for the copy engine
  // (chunk c0 in rows c0 ... c0 + 15, over the parked values of that chunk once they have been used).
  const uint32_t fin_warp = base + bars_off + 16u * kMaxStages + 64u + (warp & 3u) * (80u * 128u);
  // Finish 16 values per thread (rows m0 ... m0 + 15 of the short extent at this thread's index n along the long one)
  // and write them: through the staged tile store, or directly when tall.  Called by whole warps.
  auto emit16 = [&](int m0, int n, int col0, const float (&acc)[16], const float (&cin)[16]) {
    const bool n_ok = n < big_extent;
    float v[16];
    sk_values16<kTall>(p, m0, n, n_ok, acc, cin, v);
    if constexpr (kTall) {
      if (n_ok) sk_store16<true>(p, m0, n, v);
    } else {
      sk_stage16(p, &tmD, fin_warp + static_cast<uint32_t>(m0) * 128u, lane, m0, n, col0, v);
    }
  };

  // The producer and MMA roles run warp-uniform (one elected lane issues), with the (tile, k-block) position and
  // the ring slot advanced incrementally: the single issuing thread must sustain one 18 KB stage every few hundred
  // cycles, so there is no division and no per-lane register traffic in these loops.
  const uint32_t nstages = static_cast<uint32_t>(sp.stages);
  const uint32_t atom_bytes = kSkinnyTileN * 128u + static_cast<uint32_t>(sp.m_pad) * 128u;
  if (warp == 0) {
    const uint64_t pol_w = l2_policy_evict_first();  // weights are read exactly once
    const uint64_t pol_x = l2_policy_evict_last();   // the activation slab is re-read by every CTA
    uint32_t s = 0, ph = 0;
    int tile = tile0, kb = kb0;
    for (int i = 0; i < n_units; ++i) {
      if (!mbar_wait_warp(empty0 + 8u * s, ph ^ 1u, w, (1u << 8) | s)) break;
      const uint32_t bar = full0 + 8u * s;
      const uint32_t sw_ = base + s * sp.stage_bytes;
      if (elect_one() && !((p.debug_flags & 1u) && i == 0)) {  // test hook: the first stage is never filled nor signalled
        mbar_arrive_expect_tx(bar, sp.stage_bytes);
        for (int a = 0; a < sp.atoms; ++a) {  // slices past K are zero-filled by TMA and still count their bytes
          const int k0 = (kb * sp.atoms + a) * sp.kblk;
          tma_load_3d(sw_ + a * atom_bytes, &tmW, bar, k0, tile * kSkinnyTileN, 0, pol_w);
          tma_load_3d(sw_ + a * atom_bytes + kSkinnyTileN * 128u, &tmX, bar, k0, 0, 0, pol_x);
        }
      }
      __syncwarp();
      if (++kb == sp.kbs) {
        kb = 0;
        ++tile;
      }
      if (++s == nstages) {
        s = 0;
        ph ^= 1u;
      }
    }
  } else if (warp == 1) {
    const uint64_t desc_hi = make_smem_desc_hi(16, 1024);
    const uint32_t stage16 = static_cast<uint32_t>(sp.stage_bytes) >> 4;
    const uint64_t wdesc0 = smem_desc(desc_hi, base);
    const uint64_t xdesc0 = smem_desc(desc_hi, base + kSkinnyTileN * 128u);
    const uint32_t idesc = p.idesc;
    uint32_t s = 0, ph = 0, seg = 0;
    uint64_t wdesc = wdesc0, xdesc = xdesc0;
    int kb = kb0, done = 0;
    bool ok = true;
    while (ok && done < n_units) {
      const int seg_units = min(n_units - done, sp.kbs - kb);  // rest of this tile's K that belongs to this CTA
      const uint32_t buf = seg & 1u;
      if (!mbar_wait_warp(tempty0 + 8u * buf, ((seg >> 1) & 1u) ^ 1u, w, (2u << 8) | 0x80u | buf)) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + buf * static_cast<uint32_t>(sp.m_pad);
      for (int i = 0; i < seg_units; ++i) {
        if (!mbar_wait_warp(full0 + 8u * s, ph, w, (2u << 8) | s)) {
          ok = false;
          break;
        }
        tc_fence_after();
        if (elect_one()) {
          for (uint32_t a = 0; a < static_cast<uint32_t>(sp.atoms); ++a) {
            const uint64_t wd = wdesc + a * (atom_bytes >> 4), xd = xdesc + a * (atom_bytes >> 4);
            if (!p.ab_fp8) {
              umma_f16<1>(d_tmem, wd, xd, idesc, static_cast<uint32_t>(i != 0 || a != 0));
#pragma unroll
              for (uint32_t k = 1; k < kBlockK / kUmmaK; ++k) umma_f16<1>(d_tmem, wd + 2u * k, xd + 2u * k, idesc, 1u);
            } else {  // 8-bit floats: again four 32-byte steps per 128-byte slice
              umma_f8<1>(d_tmem, wd, xd, idesc, static_cast<uint32_t>(i != 0 || a != 0));
#pragma unroll
              for (uint32_t k = 1; k < 4; ++k) umma_f8<1>(d_tmem, wd + 2u * k, xd + 2u * k, idesc, 1u);
            }
          }
          umma_commit<1>(empty0 + 8u * s);
        }
        __syncwarp();
        wdesc += stage16;
        xdesc += stage16;
        if (++s == nstages) {
          s = 0;
          ph ^= 1u;
          wdesc = wdesc0;
          xdesc = xdesc0;
        }
      }
      if (ok && elect_one()) umma_commit<1>(tfull0 + 8u * buf);
      __syncwarp();
      done += seg_units;
      kb = 0;
      ++seg;
    }
  } else if constexpr (kCluster) {
    // This CTA's one segment: the raw accumulators go to its own ring memory (every MMA that read the ring has
    // completed once the accumulator is), laid out [short index][128 long indices] like a workspace partial.
    const uint32_t q = warp & 3u;
    const uint32_t n_local = q * 32u + lane;
    if (mbar_wait_warp(tfull0, 0u, w, (3u << 8), 64u)) {
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((q * 32u) << 16);
      for (int c0 = 0; c0 < sp.m_pad; c0 += 16) {
        uint32_t acc[16];
        tmem_ld_32x16(t_row + static_cast<uint32_t>(c0), acc);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) st_shared_b32(base + static_cast<uint32_t>(c0 + j) * (kSkinnyTileN * 4u) + n_local * 4u, acc[j]);
      }
      tc_fence_before();
    }
  } else {
    const uint32_t q = warp & 3u;
    const int n_local = static_cast<int>(q * 32u + lane);
    const bool leader = (warp == 2 && lane == 0);
    uint32_t seg = 0;
    int u = u_begin;
    while (u < u_end) {
      const int tile = u / sp.kbs;
      const int tile_u0 = tile * sp.kbs;
      const int seg_end = min(u_end, tile_u0 + sp.kbs);
      const uint32_t buf = seg & 1u;
      const int n = tile * kSkinnyTileN + n_local;
      const int col0 = tile * kSkinnyTileN + static_cast<int>(q * 32u);
      const bool n_ok = n < big_extent;
      if (seg != 0u) {  // the copy engine has read the slabs staged for the previous tile before anything else is put there
        if (lane == 0) bulk_wait_group_read<0>();
        __syncwarp();
      }
      const bool whole = (u == tile_u0) && (seg_end == tile_u0 + sp.kbs);  // this CTA owns the tile's whole K
      // contributors of a split tile: c_first reaches it at the end of its range (second slot) unless its range starts
      // exactly here; every later contributor starts inside the tile (first slot)
      const int c_first = whole ? 0 : sk_unit_owner(sp, tile_u0);
      const int c_last = whole ? 0 : sk_unit_owner(sp, tile_u0 + sp.kbs - 1);
      const int first_slot = (whole || sk_cta_begin(sp, c_first) == tile_u0) ? 0 : 1;
      auto partial_of = [&](int c) {
        return p.partials + (static_cast<size_t>(c) * 2 + (c == c_first ? first_slot : 0)) * (kSkinnyTileN * sp.m_pad);
      };
      // While the main loop of this segment runs, these warps have nothing to do.  The usual case for the CTA that
      // computes the head of a split tile is that all other contributors finish before it does; as soon as the count says so,
      // their partials (and C_in) are fetched, this CTA never publishes its own partial and the tail of the kernel
      // is one tensor-memory read, a few adds and the stores.  The fetched values are parked in shared memory: the
      // store cannot issue before its load has landed, which pins the loads to this side of the wait (left in
      // registers, the loads were scheduled after the wait, next to their use, and the tail paid their latency).
      // Room for 64 floats per thread: one chunk of 16 from up to four contributors (short extent <= 16) or up to
      // four chunks from the one other contributor; other shapes take the general path below.  Both paths add the
      // same values in the same order, so the result does not depend on which one ran.
      bool early = false;
      const bool by_chunk = sp.m_pad > 16;  // parked value 16 b + j = chunk b of the other contributor (else: chunk 0 of contributor b)
      const uint32_t park = fin_warp + lane * 4u;  // value v lives at park + 128 v
      if (!whole && (by_chunk ? c_last - c_first == 1 : c_last - c_first <= 3)) {
        // The leader looks at the arrival word again and again (about once a microsecond) until either all other
        // contributors have arrived -- for the CTA that holds the head of a tile they are always done before its own
        // range is, since their share of the tile is shorter than its whole range -- or its own accumulator is complete,
        // in which case the partial is published as usual.  (Also bounded by the plan's wait limit.)
        const unsigned long long all_others = (p.tag << 16) | static_cast<unsigned long long>(c_last - c_first);
        volatile uint32_t* answer_slot = s_early + (seg == 0 ? 0 : 1);
        const uint64_t poll_t0 = globaltimer_ns();
        uint32_t answer = 0u;  // 1: the others are all in; 2: stop looking
        while (true) {
          if (leader) {
            uint32_t v = 0u;
            if (stale_status != 0u || *s_abort != 0u) v = 2u;
            else if (ld_acquire_gpu_u64(p.counters + tile) == all_others) v = 1u;
            else if (mbar_try_wait(tfull0 + 8u * buf, (seg >> 1) & 1u) || globaltimer_ns() - poll_t0 > p.timeout_ns) v = 2u;
            *answer_slot = v;
          }
          named_barrier_sync(1, 128);
          answer = *answer_slot;
          named_barrier_sync(1, 128);  // everybody has read the answer before the leader writes the next one
          if (answer != 0u) break;
          __nanosleep(400);
        }
        early = answer == 1u;
        if (early) {
          const int other = c_first == static_cast<int>(blockIdx.x) ? c_last : c_first;
          float pre[4][16], cin0[16];
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            // (by contributor: this CTA's own slot is read too and not used; by chunk: chunks past m_pad repeat the last)
            const float* part = by_chunk ? partial_of(other) + min(b * 16, sp.m_pad - 16) * kSkinnyTileN
                                         : partial_of(min(c_first + b, c_last));
#pragma unroll
            for (int j = 0; j < 16; ++j) pre[b][j] = __ldcg(part + j * kSkinnyTileN + n_local);
          }
          sk_load_cin16<kTall>(p, 0, n, n_ok, cin0);
#pragma unroll
          for (int b = 0; b < 4; ++b) {
#pragma unroll
            for (int j = 0; j < 16; ++j) st_shared_b32(park + 128u * (16 * b + j), __float_as_uint(pre[b][j]));
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) st_shared_b32(park + 128u * (64 + j), __float_as_uint(cin0[j]));
        }
      }
      if (!mbar_wait_warp(tfull0 + 8u * buf, (seg >> 1) & 1u, w, (3u << 8) | buf, 64u)) break;
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((q * 32u) << 16) + buf * static_cast<uint32_t>(sp.m_pad);
      float* my_partial = p.partials + (static_cast<size_t>(blockIdx.x) * 2 + (seg == 0 ? 0 : 1)) * (kSkinnyTileN * sp.m_pad);
      for (int c0 = 0; c0 < sp.m_pad; c0 += 16) {
        uint32_t acc[16];
        tmem_ld_32x16(t_row + static_cast<uint32_t>(c0), acc);
        tmem_ld_wait();
        if (whole) {
          float accf[16], cin[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) accf[j] = __uint_as_float(acc[j]);
          sk_load_cin16<kTall>(p, c0, n, n_ok, cin);
          emit16(c0, n, col0, accf, cin);
        } else if (early) {
          float sum[16], cin[16];
          if (c0 == 0) {
#pragma unroll
            for (int j = 0; j < 16; ++j) cin[j] = __uint_as_float(ld_shared_b32(park + 128u * (64 + j)));
          } else {
            sk_load_cin16<kTall>(p, c0, n, n_ok, cin);
          }
          if (by_chunk) {
            // two contributors, added in their order: ((0 + first) + second), as every other path adds them
            const bool own_first = c_first == static_cast<int>(blockIdx.x);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float other_v = __uint_as_float(ld_shared_b32(park + 128u * (c0 + j)));
              const float mine = __uint_as_float(acc[j]);
              sum[j] = (0.0f + (own_first ? mine : other_v)) + (own_first ? other_v : mine);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) sum[j] = 0.0f;
#pragma unroll
            for (int b = 0; b < 4; ++b) {  // the b-th contributor's chunk 0
              const int cc = c_first + b;
              if (cc <= c_last) {
                const bool own = cc == static_cast<int>(blockIdx.x);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  const float other_v = __uint_as_float(ld_shared_b32(park + 128u * (16 * b + j)));
                  sum[j] += own ? __uint_as_float(acc[j]) : other_v;
                }
              }
            }
          }
          emit16(c0, n, col0, sum, cin);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c0 + j < small_extent) my_partial[(c0 + j) * kSkinnyTileN + n_local] = __uint_as_float(acc[j]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8u * buf);
      if (early) {
        if (leader) p.counters[tile] = 0ull;  // the others counted themselves in; a replay of this launch (same tag) must find no arrivals
      } else if (!whole) {
        // Publish the partial and count the arrival; the last contributor reduces.  The barrier orders the four
        // warps' partial stores before the leader's atomic, whose release makes them visible to whoever reads the
        // count later and whose acquire, passed on by the second barrier, lets this CTA read the earlier partials.
        named_barrier_sync(1, 128);
        if (leader) {
          const uint32_t old = stale_status == 0u ? sk_arrive(p.counters + tile, p.tag) : 0xffffffffu;
          *s_last = (old == static_cast<uint32_t>(c_last - c_first)) ? 1u : 0u;
        }
        named_barrier_sync(1, 128);
        const bool last = *s_last != 0u;
        if (last && c_last - c_first == 1 && small_extent > 16) {
          // Two contributors and several 16-row chunks (the usual case of a wide short extent on a large problem, where a
          // CTA's range is longer than a tile): the chunks are double buffered by hand -- the partials and C_in of chunk
          // i + 1 are requested before chunk i is added up and stored -- because the compiler may not move those loads
          // above the stores to D, and a chunk at a time costs one round trip to L2 plus one to HBM each (8 us for four
          // chunks, measured).  Same additions in the same order as the loop below.
          const float* q0 = partial_of(c_first) + n_local;
          const float* q1 = partial_of(c_last) + n_local;
          auto request = [&](int m0, float (&v)[2][16], float (&ci)[16]) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {  // m0 + j < m_pad
              v[0][j] = __ldcg(q0 + (m0 + j) * kSkinnyTileN);
              v[1][j] = __ldcg(q1 + (m0 + j) * kSkinnyTileN);
            }
            sk_load_cin16<kTall>(p, m0, n, n_ok, ci);
          };
          auto finish = [&](int m0, const float (&v)[2][16], const float (&ci)[16]) {
            float sum[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) sum[j] = (0.0f + v[0][j]) + v[1][j];
            emit16(m0, n, col0, sum, ci);
          };
          float va[2][16], vb[2][16], ca[16], cb[16];
          request(0, va, ca);
          for (int m0 = 0; m0 < small_extent; m0 += 32) {
            const bool second = m0 + 16 < small_extent;
            if (second) request(m0 + 16, vb, cb);
            finish(m0, va, ca);
            if (!second) break;
            if (m0 + 32 < small_extent) request(m0 + 32, va, ca);
            finish(m0 + 16, vb, cb);
          }
          if (leader) p.counters[tile] = 0ull;  // a replay of this launch (same tag) must find no arrivals
        } else if (last) {
          for (int m0 = 0; m0 < small_extent; m0 += 16) {
            float sum[16], cin[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) sum[j] = 0.0f;
            sk_load_cin16<kTall>(p, m0, n, n_ok, cin);  // in flight together with the partials
            // Contributor order, so that the result does not depend on arrival order; four contributors' loads are in
            // flight at a time.  The loads are unconditional (past the last contributor they repeat it) because loads
            // under a condition were scheduled one contributor, and one round trip to memory, after the other.
            for (int c = c_first; c <= c_last; c += 4) {
              float v[4][16];
#pragma unroll
              for (int b = 0; b < 4; ++b) {
                const float* part = partial_of(min(c + b, c_last));
#pragma unroll
                for (int j = 0; j < 16; ++j) v[b][j] = __ldcg(part + (m0 + j) * kSkinnyTileN + n_local);  // m0 + j < m_pad
              }
#pragma unroll
              for (int b = 0; b < 4; ++b)
                if (c + b <= c_last) {
#pragma unroll
                  for (int j = 0; j < 16; ++j) sum[j] += v[b][j];
                }
            }
            emit16(m0, n, col0, sum, cin);
          }
          if (leader) p.counters[tile] = 0ull;  // a replay of this launch (same tag) must find no arrivals
        }
        named_barrier_sync(1, 128);  // s_last is reused by the next segment
      }
      u = seg_end;
      ++seg;
    }
  }

  if constexpr (kCluster) {
    // Every thread of the cluster meets here (also after a timeout: the roles above fall through to this point), so
    // the partial tiles of all ranks are visible cluster-wide behind the barrier.  Rank r then finishes the 16-row
    // chunks r, r + c, ... of the short extent: the c partials are added in rank order (the order of the K ranges),
    // read from the peers' shared memory.  C_in is requested before the wait so that its latency hides behind it.
    const uint32_t crank = cluster_ctarank();
    const uint32_t csize = static_cast<uint32_t>(sp.cluster);
    const uint32_t n_local = (warp & 3u) * 32u + lane;
    const int n = tile0 * kSkinnyTileN + static_cast<int>(n_local);
    const int col0 = tile0 * kSkinnyTileN + static_cast<int>((warp & 3u) * 32u);
    const bool finisher = warp >= 2;
    const bool n_ok = n < big_extent;
    float cin[16];
    cluster_arrive();
    if (finisher && static_cast<int>(crank) * 16 < small_extent) sk_load_cin16<kTall>(p, static_cast<int>(crank) * 16, n, n_ok, cin);
    cluster_wait();
    if (finisher && *s_abort == 0u && stale_status == 0u) {
      for (int m0 = static_cast<int>(crank) * 16; m0 < small_extent; m0 += static_cast<int>(csize) * 16) {
        if (m0 != static_cast<int>(crank) * 16) sk_load_cin16<kTall>(p, m0, n, n_ok, cin);
        float sum[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) sum[j] = 0.0f;
        for (uint32_t r = 0; r < csize; ++r) {
          const uint32_t peer = mapa(base + static_cast<uint32_t>(m0) * (kSkinnyTileN * 4u) + n_local * 4u, r);
          float v[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(ld_shared_cluster_b32(peer + static_cast<uint32_t>(j) * (kSkinnyTileN * 4u)));
#pragma unroll
          for (int j = 0; j < 16; ++j) sum[j] += v[j];
        }
        emit16(m0, n, col0, sum, cin);
      }
    }
    cluster_arrive();  // nobody's shared memory may go away while a peer still reads it
    cluster_wait();
  }
  if (!kTall && warp >= 2 && lane == 0) bulk_wait_group_read<0>();  // staged slabs are read; the writes complete with the grid
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<1>(tmem_base, tmem_cols);
  }
}

// Launch.  Returns a gemm_status_t value (0 = ok, 7 = CUDA failure).
// `tall` selects the mirrored addressing (tW then maps A, tX maps B; tD, the store map of D, is then unused).
inline int skinny_launch(const SkinnyParams& p, const CUtensorMap& tW, const CUtensorMap& tX, const CUtensorMap& tD, int device, cudaStream_t stream,
                         char* err, size_t err_len, bool tall, bool early_launch) {
  const bool cluster = p.plan.cluster > 1;
  const void* kern = tall ? (cluster ? reinterpret_cast<const void*>(skinny_gemm_kernel<true, true>) : reinterpret_cast<const void*>(skinny_gemm_kernel<true, false>))
                          : (cluster ? reinterpret_cast<const void*>(skinny_gemm_kernel<false, true>) : reinterpret_cast<const void*>(skinny_gemm_kernel<false, false>));
  const KernelSlot slot = tall ? (cluster ? kSlotSkinnyTallCluster : kSlotSkinnyTall) : (cluster ? kSlotSkinnyCluster : kSlotSkinny);
  cudaError_t e = ensure_dynamic_smem(kern, slot, device, p.plan.smem_bytes);
  if (e == cudaSuccess) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(p.plan.grid, 1, 1);
    cfg.blockDim = dim3(kSkinnyThreads, 1, 1);
    cfg.dynamicSmemBytes = p.plan.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (early_launch) {
      attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up may overlap the previous kernel's tail
      attr[na].val.programmaticStreamSerializationAllowed = 1;
      ++na;
    }
    if (cluster) {
      attr[na].id = cudaLaunchAttributeClusterDimension;
      attr[na].val.clusterDim.x = p.plan.cluster;
      attr[na].val.clusterDim.y = 1;
      attr[na].val.clusterDim.z = 1;
      ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    if (tall) e = cluster ? cudaLaunchKernelEx(&cfg, skinny_gemm_kernel<true, true>, tW, tX, tD, p) : cudaLaunchKernelEx(&cfg, skinny_gemm_kernel<true, false>, tW, tX, tD, p);
    else e = cluster ? cudaLaunchKernelEx(&cfg, skinny_gemm_kernel<false, true>, tW, tX, tD, p) : cudaLaunchKernelEx(&cfg, skinny_gemm_kernel<false, false>, tW, tX, tD, p);
  }
  if (e != cudaSuccess) {
    snprintf(err, err_len, "skinny launch: %s", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return 7;
  }
  return 0;
}

}  // namespace b200

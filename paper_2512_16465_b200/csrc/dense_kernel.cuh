// Dense GEMM kernel for sm_100a: persistent, warp-specialised, TMA -> shared ring -> tcgen05.mma
// (accumulator in tensor memory, double buffered) -> epilogue warps -> swizzled staging -> TMA store.
//
// Roles inside one CTA (64 + 128 * EPI_WG threads):
//   warp 0, lane 0   TMA producer: fills the STAGES-deep ring of (A tile, B tile) k-blocks
//   warp 1, lane 0   MMA issuer: 4 x tcgen05.mma (K = 16 each) per k-block, commits free the ring slot;
//                    warp 1 also owns the tensor-memory allocation
//   warps 2..        epilogue: tcgen05.ld 32 lanes x 32 columns, alpha/beta/bias/activation in fp32,
//                    convert, write a 32-row x 128-byte swizzled slab, one TMA store per slab per warp
//
// CG = 2 runs the same code on a cluster of two CTAs that share one 256 x BN tile: each CTA loads
// its own 128 rows of A and its half of the B tile, the leader CTA (cluster rank 0) issues
// tcgen05.mma.cta_group::2 for both, and each CTA drains its own 128 accumulator rows.
//
// Everything about the problem (tile N, stage count, operand major-ness, dtypes, epilogue) is a
// run-time field of DenseParams; the only compile-time choices are CG and EPI_WG.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "ptx.cuh"

namespace b200 {

constexpr int kBlockK = 64;         // K elements per ring stage = one 128-byte swizzle row of 16-bit data
constexpr int kUmmaK = 16;          // K of one tcgen05.mma for 16-bit inputs
constexpr int kCtaM = 128;          // accumulator rows per CTA = TMEM lanes
constexpr int kMaxStages = 12;
constexpr int kSlabBytes = 32 * 128;  // epilogue staging slab of one warp: 32 rows x 128 bytes

// device status word values (also used by the skinny kernel)
constexpr uint32_t kStatusTimeout = 0x80000000u;  // | role << 8 | detail

// Division by a divisor fixed at plan time (Granlund-Montgomery): n / d for every 32-bit n in a multiply and two shifts.
// The tile scheduler divides by run-time tile counts several times per tile and role; a hardware-emulated 32-bit
// division is a chain of some twenty dependent instructions, most felt in front of a CTA's first load.
struct FastDiv {
  uint32_t mul, sh1, sh2;
};
inline FastDiv make_fastdiv(uint32_t d) {  // host; 1 <= d <= 2^31
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;
  FastDiv f;
  f.mul = static_cast<uint32_t>(((1ull << 32) * ((1ull << l) - d)) / d + 1);
  f.sh1 = l < 1 ? l : 1;
  f.sh2 = l ? l - 1 : 0;
  return f;
}
__host__ __device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv& f) {
#ifdef __CUDA_ARCH__
  const uint32_t t = __umulhi(f.mul, n);
#else
  const uint32_t t = static_cast<uint32_t>((static_cast<unsigned long long>(f.mul) * n) >> 32);
#endif
  return (t + ((n - t) >> f.sh1)) >> f.sh2;
}

struct DenseParams {
  int M, N, K, batch;
  // Columns [0, n_full) of a row are whole 16-byte units and leave through the TMA store; a bulk tensor store writes
  // whole 16-byte units, so when N * (output element size) is not a multiple of 16 the last columns [n_full, N) are
  // written element by element from the registers instead, and the bytes behind column N - 1 stay untouched.
  int n_full;
  int tiles_m, tiles_n;  // tiles per matrix; a tile is (128*CG) x bn
  int num_tiles;         // batch * tiles_m * tiles_n
  int raster_group;      // tile rows swept together (column-wise inside the group)
  // the scheduler's divisors: tiles per matrix, tiles per raster group, rows of a full group and of the last group, slots per matrix
  FastDiv fd_matrix, fd_group, fd_rows, fd_last_rows, fd_list;
  int kstep_shift;       // log2 of the K extent of a ring stage (kblk * atoms, a power of two)
  int bn;                // tile N (multiple of 64, <= 512)
  // A tile wider than 256 columns is computed by two MMAs per K step, each mma_n = bn / 2 columns wide (n_mma = 2), and
  // has no second accumulator buffer (acc_bufs = 1: 2 * bn columns would not fit the 512 of tensor memory), so such tiles
  // are planned where every CTA computes one tile.  Otherwise mma_n = bn, n_mma = 1, acc_bufs = 2.
  int mma_n, n_mma, acc_bufs;
  int b_box_rows;        // rows of one B box: this CTA's share of one MMA's columns (b_rows / n_mma)
  int stages;            // ring depth
  int num_kb;            // ring stages per tile = ceil(K / (64 * atoms))
  int atoms;             // 64-wide K slices ("swizzle atoms") per ring stage: 1 or 2
  uint32_t tmem_cols;    // power of two >= acc_bufs * bn
  uint32_t idesc;        // tcgen05 instruction descriptor
  uint32_t a_stage_bytes, b_stage_bytes;  // per CTA, per stage (all atoms)
  uint32_t a_atom_bytes, b_atom_bytes;    // per CTA, one 64-wide K slice
  int a_kmajor, b_kmajor;                 // 1: K contiguous in memory; 0: M (resp. N) contiguous
  int b_rows;                             // rows of B (N extent) this CTA loads per stage
  uint64_t a_desc_hi, b_desc_hi;          // descriptor bits above the start address
  uint32_t a_kstep, b_kstep;              // start-address advance per K = 16 slice, bytes
  int out_dtype;                          // 0 bf16, 1 f16, 2 f32
  int epilogue;                           // gemm_epilogue_t
  int bias_per_row;                       // the bias has M entries (one per output row) instead of N
  int ab_fp8;                             // operands are 8-bit floats (tcgen05 kind::f8f6f4), else 16-bit (kind::f16)
  int kblk;                               // elements of K in one 128-byte slice: 64 (16-bit operands) or 128 (8-bit)
  int a_tri;                              // structure of op(A): 0 dense, 1 lower triangular (zero for k > i), 2 upper (zero for k < i)
  int b_tri;                              // structure of op(B): 0 dense, 1 lower triangular (zero for k < j), 2 upper (zero for k > j)
  // Structured problems (one triangle of D wanted, triangular operands) come with a schedule in device memory: per
  // matrix, slot k * (CTAs or pairs) + c holds the k-th tile of CTA (pair) c as a tile id of the full tiles_m x tiles_n
  // numbering, or -1 when it has none; num_tiles then counts batch * list_len slots.
  const int* tile_list;                   // nullptr: every tile is computed, dealt round-robin
  int list_len;
  // Tail split (kernels built with kSplit): the tiles from split_first_tile on, which would leave most CTAs idle in
  // the last wave, are cut into `split` slices of K each, one work item per slice; num_items counts whole tiles + slices.
  int split, split_first_tile, num_items;
  float* partials;                        // workspace: raw fp32 accumulators of slices 1..split-1, [tile][rank][slice-1][128][bn]
  // One word per such partial at the head of the workspace: it holds this run's tag once the partial is written (any
  // other value -- zeros, another run's tag, whatever the memory held before -- means "not yet"), and the reducing CTA
  // puts it back to zero so that a replay of the same launch starts clean.  No initialisation is needed.
  unsigned long long* split_flags;
  unsigned long long split_tag;           // this run's tag (48 bits, never 0)
  float alpha, beta;
  const float* bias;
  const void* c_in;                       // = D buffer; read when beta != 0
  long long ldc, stride_c;                // elements
  uint32_t* status;                       // device status word
  unsigned long long timeout_ns;
  uint32_t debug_flags;                   // bit 0: withhold one producer arrival (timeout test hook)
  int l2_hint_a, l2_hint_b;               // L2 eviction priority of operand loads: 0 normal, 1 evict-first, 2 evict-last
  int l2_hint_d;                          // 1: output stores ask L2 to evict them first (a large D would push the operands out)
  int k_serpentine;                       // 1: every second tile of a CTA walks K from the far end back to 0
};

struct WaitCtx {
  volatile uint32_t* s_abort;  // shared: set once any thread of the CTA gave up
  uint32_t* g_status;          // global status word (also polled, so that an abort spreads between CTAs)
  unsigned long long timeout_ns;
};

// Bounded mbarrier wait.  Returns false when the wait was abandoned: either this thread ran out of
// time (it then records `code` in the status word) or another thread already aborted.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtx& w, uint32_t code) {
  const uint64_t t0 = globaltimer_ns();
  uint32_t it = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++it & 31u) == 0u) {
      if (*w.s_abort) return false;
      if (*reinterpret_cast<volatile uint32_t*>(w.g_status) != 0u) {
        *w.s_abort = 1u;
        return false;
      }
      if (globaltimer_ns() - t0 > w.timeout_ns) {
        *w.s_abort = 1u;
        atomicCAS(w.g_status, 0u, kStatusTimeout | code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& w, uint32_t code) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, w, code);
}

// Warp-uniform variant: every lane of a fully active warp polls, and all lanes leave with the same answer.
__device__ __noinline__ bool mbar_wait_warp_slow(uint32_t bar, uint32_t parity, const WaitCtx& w, uint32_t code,
                                                 uint32_t backoff_ns) {
  const uint64_t t0 = globaltimer_ns();
  uint32_t it = 0;
  while (true) {
    if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
    if (backoff_ns != 0u && it > 16u) __nanosleep(backoff_ns);  // long waits should not burn issue slots
    if ((++it & 31u) == 0u) {
      bool give_up = false;
      if (lane_id() == 0) {
        if (*w.s_abort || *reinterpret_cast<volatile uint32_t*>(w.g_status) != 0u) {
          *w.s_abort = 1u;
          give_up = true;
        } else if (globaltimer_ns() - t0 > w.timeout_ns) {
          *w.s_abort = 1u;
          atomicCAS(w.g_status, 0u, kStatusTimeout | code);
          give_up = true;
        }
      }
      if (__any_sync(0xffffffffu, give_up)) return false;
    }
  }
}
// backoff_ns > 0: the warp sleeps between polls once the wait has proved long (an epilogue warp during a main loop).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const WaitCtx& w, uint32_t code,
                                               uint32_t backoff_ns = 0u) {
  if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
  return mbar_wait_warp_slow(bar, parity, w, code, backoff_ns);
}

struct TileCoord {
  int batch, tm, tn;
};
// Linear tile id -> (batch, tile row, tile column).  Inside one matrix, tiles are visited in groups
// of `raster_group` tile rows; inside a group the row index runs fastest, so the CTAs that are
// resident together work on a compact block of the output and share A and B panels in L2.
// (The scheduling functions from here to work_item also compile for the host: gemm_plan_schedule walks a plan's
// schedule with the very code the kernels run.)
__host__ __device__ __forceinline__ TileCoord decode_tile(const DenseParams& p, int t) {
  TileCoord c;
  const int per_matrix = p.tiles_m * p.tiles_n;
  c.batch = static_cast<int>(fast_div(static_cast<uint32_t>(t), p.fd_matrix));
  const int r = t - c.batch * per_matrix;
  const int group_sz = p.raster_group * p.tiles_n;
  const int g = static_cast<int>(fast_div(static_cast<uint32_t>(r), p.fd_group));
  const int first_m = g * p.raster_group;
  const int gm = min(p.raster_group, p.tiles_m - first_m);
  const int within = r - g * group_sz;
  c.tn = static_cast<int>(fast_div(static_cast<uint32_t>(within), gm == p.raster_group ? p.fd_rows : p.fd_last_rows));
  c.tm = first_m + (within - c.tn * gm);
  return c;
}

// The same with plain divisions, for the wide pair kernel: its tiles last tens of thousands of cycles, and its register
// allocation is at the limit where any change of this code has cost spills.
__host__ __device__ __forceinline__ TileCoord decode_tile_div(int t, int tiles_m, int tiles_n, int raster_group) {
  TileCoord c;
  const int per_matrix = tiles_m * tiles_n;
  c.batch = t / per_matrix;
  const int r = t - c.batch * per_matrix;
  const int group_sz = raster_group * tiles_n;
  const int g = r / group_sz;
  const int first_m = g * raster_group;
  const int gm = min(raster_group, tiles_m - first_m);
  const int within = r - g * group_sz;
  c.tn = within / gm;
  c.tm = first_m + (within - c.tn * gm);
  return c;
}

// The ring stages [lo, hi) of K that a tile with output rows [row0, row0 + rows) and columns [col0, col0 + cols) has to
// visit.  A triangular op(A) or op(B) (zero beyond the diagonal by the caller's word) makes every stage that lies
// wholly in a zero part a no-op, so it is skipped; the stages that a diagonal crosses are computed in full.  At least
// one stage is always kept so that the accumulator gets written (when nothing is left, any stage yields the zeros).
struct KRange {
  int lo, hi;
};
__host__ __device__ __forceinline__ KRange k_range(const DenseParams& p, int row0, int rows, int col0, int cols) {
  KRange r{0, p.num_kb};
  const int ks = p.kstep_shift;
  if (p.a_tri == 1) r.hi = min(r.hi, ((min(row0 + rows, p.M) - 1) >> ks) + 1);       // k <= last row
  else if (p.a_tri == 2) r.lo = max(r.lo, row0 >> ks);                                // k >= first row
  if (p.b_tri == 1) r.lo = max(r.lo, col0 >> ks);                                     // k >= first column
  else if (p.b_tri == 2) r.hi = min(r.hi, ((min(col0 + cols, p.N) - 1) >> ks) + 1);   // k <= last column
  if (r.lo >= r.hi) {
    r.lo = min(r.lo, p.num_kb - 1);
    r.hi = r.lo + 1;
  }
  return r;
}

// A work item of a CTA (pair): a whole tile (slice = -1) or one K slice of a split tile, with the ring stages it covers.
struct WorkItem {
  int tile, slice;
  KRange kr;
};
template <bool kSplit>
__host__ __device__ __forceinline__ int item_tile(const DenseParams& p, int item) {
  if (p.tile_list != nullptr) {  // (never together with a tail split); < 0: an empty slot
    const int b = static_cast<int>(fast_div(static_cast<uint32_t>(item), p.fd_list));
#ifdef __CUDA_ARCH__
    const int t = __ldg(p.tile_list + (item - b * p.list_len));
#else
    const int t = p.tile_list[item - b * p.list_len];  // (the host walks the plan's host copy of the list)
#endif
    return t < 0 ? -1 : b * (p.tiles_m * p.tiles_n) + t;
  }
  if (!kSplit || item < p.split_first_tile) return item;
  return p.split_first_tile + (item - p.split_first_tile) / p.split;
}
template <bool kSplit>
__host__ __device__ __forceinline__ WorkItem work_item(const DenseParams& p, int item, int tile, int row0, int rows, int col0) {
  WorkItem wi{tile, -1, k_range(p, row0, rows, col0, p.bn)};
  if (kSplit && item >= p.split_first_tile) {
    wi.slice = (item - p.split_first_tile) - (tile - p.split_first_tile) * p.split;
    wi.kr.lo = wi.slice * p.num_kb / p.split;
    wi.kr.hi = (wi.slice + 1) * p.num_kb / p.split;
  }
  return wi;
}
// Bounded wait for up to 32 consecutive flag words that other CTAs of this launch set to `tag` (all CTAs of these
// persistent kernels are resident, and a CTA that sets a flag never waits for anybody).  Lane l looks at word l, so the
// wait costs one round trip to memory however many words there are (one wait after the other cost a round trip each:
// 4 us for the seven slices of 256 x 256 x 32768).  Warp-uniform; false = gave up (timeout or abort elsewhere).
__device__ __noinline__ bool flags_wait_warp(const unsigned long long* flags, int n, unsigned long long tag, const WaitCtx& w, uint32_t code) {
  const uint64_t t0 = globaltimer_ns();
  const int l = static_cast<int>(lane_id());
  uint32_t it = 0;
  while (true) {
    const bool hit = l >= n || ld_acquire_gpu_u64(flags + l) == tag;
    if (__all_sync(0xffffffffu, hit)) {
      __syncwarp();  // (orders every lane's later loads after the acquiring loads of the others)
      return true;
    }
    __nanosleep(64);
    if ((++it & 31u) == 0u) {
      bool give_up = false;
      if (l == 0) {
        if (*w.s_abort || *reinterpret_cast<volatile uint32_t*>(w.g_status) != 0u) {
          *w.s_abort = 1u;
          give_up = true;
        } else if (globaltimer_ns() - t0 > w.timeout_ns) {
          *w.s_abort = 1u;
          atomicCAS(w.g_status, 0u, kStatusTimeout | code);
          give_up = true;
        }
      }
      if (__any_sync(0xffffffffu, give_up)) return false;
    }
  }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
// GELU with the exact error function, t * Phi(t) = 0.5 t (1 + erf(x)), x = t / sqrt(2), evaluated without branches:
// g = erfc(|x|) = 2^p(z) with one degree-9 polynomial in z = |x| / 2 - 1 on |x| <= 4 (zero beyond: erfc(4) = 1.5e-8),
// then 1 + erf(x) = g for x < 0 (no cancellation in the negative tail) and 2 - g otherwise.  Coefficients, their
// derivation and the fp32 error report (max |error| 2.1e-7, relative error of erfc 3e-6) come from fit_gelu_poly.py
// beside this file.  About half the instructions of erff(), which matters because the epilogue shares the power budget
// with the tensor pipe.
__device__ __forceinline__ float gelu_erf(float t) {
  const float ar = fabsf(t) * 0.70710678118654752f;
  const float ax = fminf(ar, 4.0f);
  const float z = fmaf(ax, 0.5f, -1.0f);
  float p = 0.0007019337f;
  p = fmaf(p, z, -0.00019923763f);
  p = fmaf(p, z, -0.004372892f);
  p = fmaf(p, z, 0.0133363f);
  p = fmaf(p, z, -0.033581443f);
  p = fmaf(p, z, 0.08212937f);
  p = fmaf(p, z, -0.19007199f);
  p = fmaf(p, z, -5.330728f);
  p = fmaf(p, z, -12.748116f);
  p = fmaf(p, z, -7.739975f);
  float g;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(g) : "f"(p));
  g = ar > 4.0f ? 0.0f : g;  // beyond the fitted range erfc is 1.5e-8 and less: the tail goes to -0 (and to t), not to t * 7.7e-9
  return 0.5f * t * (t < 0.0f ? g : 2.0f - g);
}

// Two fp32 values in one 64-bit register and the packed arithmetic of sm_100 on them (one instruction, two results;
// each half rounds exactly like the scalar instruction).
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
// gelu_erf on two values at once: the same operations in the same order (bit-identical results), with the polynomial
// -- half of the instructions -- evaluated by packed FMAs.  The epilogue shares the power budget with the tensor pipe,
// so instructions saved here are clock gained there.
__device__ __forceinline__ void gelu_erf_pair(float& t0, float& t1) {
  const float ar0 = fabsf(t0) * 0.70710678118654752f, ar1 = fabsf(t1) * 0.70710678118654752f;
  const unsigned long long z = fma_f32x2(pack_f32x2(fminf(ar0, 4.0f), fminf(ar1, 4.0f)), pack_f32x2(0.5f, 0.5f), pack_f32x2(-1.0f, -1.0f));
  unsigned long long p = pack_f32x2(0.0007019337f, 0.0007019337f);
  p = fma_f32x2(p, z, pack_f32x2(-0.00019923763f, -0.00019923763f));
  p = fma_f32x2(p, z, pack_f32x2(-0.004372892f, -0.004372892f));
  p = fma_f32x2(p, z, pack_f32x2(0.0133363f, 0.0133363f));
  p = fma_f32x2(p, z, pack_f32x2(-0.033581443f, -0.033581443f));
  p = fma_f32x2(p, z, pack_f32x2(0.08212937f, 0.08212937f));
  p = fma_f32x2(p, z, pack_f32x2(-0.19007199f, -0.19007199f));
  p = fma_f32x2(p, z, pack_f32x2(-5.330728f, -5.330728f));
  p = fma_f32x2(p, z, pack_f32x2(-12.748116f, -12.748116f));
  p = fma_f32x2(p, z, pack_f32x2(-7.739975f, -7.739975f));
  float p0, p1, g0, g1;
  unpack_f32x2(p, p0, p1);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(g0) : "f"(p0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(g1) : "f"(p1));
  g0 = ar0 > 4.0f ? 0.0f : g0;
  g1 = ar1 > 4.0f ? 0.0f : g1;
  t0 = 0.5f * t0 * (t0 < 0.0f ? g0 : 2.0f - g0);
  t1 = 0.5f * t1 * (t1 < 0.0f ? g1 : 2.0f - g1);
}

// x * logistic(x): one ex2 and one reciprocal.  Far in the negative tail e^-x overflows to +inf, the reciprocal is 0
// and the result -0, the limit.
__device__ __forceinline__ float silu(float t) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-1.4426950408889634f * t));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return t * r;
}
// GELU, tanh form: 0.5 t (1 + tanh u) = t * logistic(2u), u = sqrt(2/pi) (t + 0.044715 t^3).  The constants are
// 2 sqrt(2/pi) log2(e) and that times 0.044715.
__device__ __forceinline__ float gelu_tanh(float t) {
  const float a = t * fmaf(0.10294324f * t, t, 2.3022082f);
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-a));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return t * r;
}
// The activation of gemm_epilogue_t value `epilogue` (value >> 1: none, ReLU, erf GELU, tanh GELU, SiLU).
__device__ __forceinline__ float activate(float v, int act) {
  if (act == 1) return fmaxf(v, 0.0f);
  if (act == 2) return gelu_erf(v);
  if (act == 3) return gelu_tanh(v);
  if (act == 4) return silu(v);
  return v;
}

// alpha/beta/bias/activation on 32 consecutive columns of one output row, in fp32.  kAll = false is the wide pair
// kernel's subset (bias per column, ReLU, erf GELU): its epilogue runs at the 168-register ceiling, and of the code
// shapes tried only this one, with erf GELU through erff(), was allocated without spills (the polynomial GELU, the
// further activations, and even no GELU at all spilled 16 to 48 bytes).  The plan never picks that kernel for a
// transcendental epilogue, so the slower erff() is not on any automatic path.
template <bool kAll = true>
__device__ __forceinline__ void epilogue_math(float (&v)[32], const uint32_t (&acc)[32], const DenseParams& p, long long row,
                                              int col0, int batch) {
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = p.alpha * __uint_as_float(acc[j]);
  if (p.beta != 0.0f && row < p.M) {
    const long long off = static_cast<long long>(batch) * p.stride_c + row * p.ldc + col0;
    if (col0 + 32 <= p.N) {
      if (p.out_dtype == 2) {
        const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(p.c_in) + off);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float4 c = src[j];
          v[4 * j + 0] += p.beta * c.x;
          v[4 * j + 1] += p.beta * c.y;
          v[4 * j + 2] += p.beta * c.z;
          v[4 * j + 3] += p.beta * c.w;
        }
      } else {
        const uint4* src = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(p.c_in) + off);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 c = src[j];
          const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float lo, hi;
            if (p.out_dtype == 0) {
              lo = __uint_as_float(w[e] << 16);
              hi = __uint_as_float(w[e] & 0xFFFF0000u);
            } else {
              const __half2 h = *reinterpret_cast<const __half2*>(&w[e]);
              lo = __low2float(h);
              hi = __high2float(h);
            }
            v[8 * j + 2 * e + 0] += p.beta * lo;
            v[8 * j + 2 * e + 1] += p.beta * hi;
          }
        }
      }
    } else {
      for (int j = 0; j < 32; ++j) {
        if (col0 + j < p.N) {
          float c;
          if (p.out_dtype == 2) c = static_cast<const float*>(p.c_in)[off + j];
          else if (p.out_dtype == 0) c = __bfloat162float(static_cast<const __nv_bfloat16*>(p.c_in)[off + j]);
          else c = __half2float(static_cast<const __half*>(p.c_in)[off + j]);
          v[j] += p.beta * c;
        }
      }
    }
  }
  if (kAll && (p.epilogue & 1) && p.bias_per_row) {  // bias variants are the odd enum values
    const float b = row < p.M ? __ldg(p.bias + row) : 0.0f;
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] += b;
  } else if (p.epilogue & 1) {
    if (col0 + 32 <= p.N) {
      const float4* b4 = reinterpret_cast<const float4*>(p.bias + col0);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float4 b = __ldg(b4 + j);
        v[4 * j + 0] += b.x;
        v[4 * j + 1] += b.y;
        v[4 * j + 2] += b.z;
        v[4 * j + 3] += b.w;
      }
    } else {
      for (int j = 0; j < 32; ++j)
        if (col0 + j < p.N) v[j] += __ldg(p.bias + col0 + j);
    }
  }
  const int act = p.epilogue >> 1;
  if (p.epilogue == 2 || p.epilogue == 3) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.0f);
  } else if (!kAll && p.epilogue >= 4) {  // (only erf GELU reaches the wide kernel)
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = 0.5f * v[j] * (1.0f + erff(v[j] * 0.70710678118654752f));
  } else if (kAll && act == 2) {
#pragma unroll
    for (int j = 0; j < 32; j += 2) gelu_erf_pair(v[j], v[j + 1]);
  } else if (kAll && act == 3) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = gelu_tanh(v[j]);
  } else if (kAll && act == 4) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = silu(v[j]);
  }
}

// The last columns of a row when they do not fill a 16-byte unit (see DenseParams::n_full): v holds the finished values
// of columns col0 .. col0 + 31 of row `row`; rounding as in the packed path.
__device__ __forceinline__ void store_ragged_columns(const DenseParams& p, const float (&v)[32], long long row, int col0, int batch) {
  if (p.n_full == p.N || col0 + 32 <= p.n_full || col0 >= p.N || row >= p.M) return;
  const long long off = static_cast<long long>(batch) * p.stride_c + row * p.ldc;
  void* d = const_cast<void*>(p.c_in);  // (C and D share the buffer)
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int c = col0 + j;
    if (c >= p.n_full && c < p.N) {
      if (p.out_dtype == 2) static_cast<float*>(d)[off + c] = v[j];
      else static_cast<uint16_t*>(d)[off + c] = static_cast<uint16_t>(p.out_dtype == 0 ? pack_bf16x2(v[j], 0.0f) : pack_f16x2(v[j], 0.0f));
    }
  }
}

// Both single-issuer roles are run by a whole warp in uniform control flow; only the instructions that
// must be issued once (TMA, tcgen05.mma, commits, barrier arrivals) sit under elect_one().  That keeps
// addresses, descriptors and coordinates in uniform registers, which is what those instructions read.
// kJoinSetup (pairs): the warp enters before the CTA-wide end of set-up and joins it itself -- the block barrier and
// the cluster barrier the other warps execute in the kernel body -- once it has worked out its first tile, so that
// work overlaps the tensor-memory allocation and the wait for the peer CTA instead of following them.
template <int CG, bool kSplit = false, bool kJoinSetup = false>
__device__ __forceinline__ void producer_role(const DenseParams& p, const CUtensorMap* tmA, const CUtensorMap* tmB,
                                              uint32_t tiles_base, uint32_t full0, uint32_t empty0, uint32_t cta_rank,
                                              int cluster_id, int num_clusters, const WaitCtx& w) {
  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const uint32_t nstages = static_cast<uint32_t>(p.stages);
  const bool expects = (CG == 1) || (cta_rank == 0);  // in a pair only the leader's barrier counts bytes
  const int b_groups = p.b_rows / 64;
  uint32_t s = 0, ph = 0;                             // ring slot and its phase, advanced incrementally
  bool stall_pending = (p.debug_flags & 1u) != 0u;
  const uint64_t pol_a = p.l2_hint_a == 2 ? l2_policy_evict_last() : (p.l2_hint_a == 1 ? l2_policy_evict_first() : l2_policy_evict_normal());
  const uint64_t pol_b = p.l2_hint_b == 2 ? l2_policy_evict_last() : (p.l2_hint_b == 1 ? l2_policy_evict_first() : l2_policy_evict_normal());
  const int kstep = p.kblk * p.atoms;
  uint32_t it = 0;
  bool waited = false;
  const int n_items = kSplit ? p.num_items : p.num_tiles;
  for (int item = cluster_id; item < n_items; item += num_clusters, ++it) {
    const int tile = item_tile<kSplit>(p, item);
    if (tile < 0) {  // an empty slot of a dealt schedule: every role skips it alike, and it does not count as a tile
      --it;          // (the loop header adds the one back: buffer and phase bookkeeping follow the tiles actually computed)
      continue;
    }
    const TileCoord tc = decode_tile(p, tile);
    const int m0 = tc.tm * (kCtaM * CG) + static_cast<int>(cta_rank) * kCtaM;
    // first column of this CTA's share of MMA group 0 (group g starts mma_n columns further; in a pair each CTA holds
    // b_box_rows of every group's columns)
    const int n0 = tc.tn * p.bn + (CG == 2 ? static_cast<int>(cta_rank) * p.b_box_rows : 0);
    // Serpentine K: all CTAs advance through K roughly in step, so the K range a wave touched last is what L2
    // still holds when the next wave starts; walking it backwards re-uses those lines of the shared A band.
    const bool rev = p.k_serpentine && (it & 1u);
    const KRange kr = work_item<kSplit>(p, item, tile, tc.tm * (kCtaM * CG), kCtaM * CG, tc.tn * p.bn).kr;
    // Everything above needs only the kernel's parameters (and the plan's own tile schedule), so it runs while the
    // previous kernel of the stream is still finishing; its memory is touched from here on.
    if (!waited) {
      if constexpr (kJoinSetup) {
        tc_fence_before();
        __syncthreads();
        cluster_arrive();  // the peer's barriers must exist before anything signals them
        cluster_wait();
        tc_fence_after();
      }
      griddep_wait();
      waited = true;
    }
    int k0 = rev ? (kr.hi - 1) * kstep : kr.lo * kstep;
    const int dk = rev ? -kstep : kstep;
    for (int kb = kr.lo; kb < kr.hi; ++kb, k0 += dk) {
      if (!mbar_wait_warp(empty0 + 8u * s, ph ^ 1u, w, (1u << 8) | s)) return;
      if (stall_pending) {  // test hook: this stage is never filled nor signalled
        stall_pending = false;
      } else {
        const uint32_t full_local = full0 + 8u * s;
        const uint32_t bar = (CG == 1) ? full_local : mapa(full_local, 0);
        const uint32_t sa = tiles_base + s * stage_bytes;
        const uint32_t sb = sa + p.a_stage_bytes;
        if (elect_one()) {
          if (expects) mbar_arrive_expect_tx(full_local, stage_bytes * CG);
          auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t pol) {
            if constexpr (CG == 1) tma_load_3d(dst, map, bar, x, y, tc.batch, pol);
            else tma_load_3d_pair(dst, map, bar, x, y, tc.batch, pol);
          };
          for (int a = 0; a < p.atoms; ++a) {  // slices past K are zero-filled by the copy engine
            const int ka = k0 + a * p.kblk;
            const uint32_t saa = sa + a * p.a_atom_bytes, sba = sb + a * p.b_atom_bytes;
            if (p.a_kmajor) {
              load(saa, tmA, ka, m0, pol_a);
            } else {
              load(saa, tmA, m0, ka, pol_a);
              load(saa + 8192u, tmA, m0 + 64, ka, pol_a);
            }
            if (p.b_kmajor) {
              for (int g = 0; g < p.n_mma; ++g) load(sba + static_cast<uint32_t>(g * p.b_box_rows) * 128u, tmB, ka, n0 + g * p.mma_n, pol_b);
            } else {
              for (int g = 0; g < b_groups; ++g) load(sba + 8192u * g, tmB, n0 + 64 * g, ka, pol_b);
            }
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
  if (kJoinSetup && !waited) {  // no tile at all: the others still wait for this warp at the end of set-up
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
  }
}

template <int CG, bool kSplit = false>
__device__ __forceinline__ void mma_role(const DenseParams& p, uint32_t tiles_base, uint32_t full0, uint32_t empty0,
                                         uint32_t tfull0, uint32_t tempty0, uint32_t tmem_base, int cluster_id,
                                         int num_clusters, const WaitCtx& w) {
  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const uint32_t nstages = static_cast<uint32_t>(p.stages);
  const uint32_t stage16 = stage_bytes >> 4, ak16 = p.a_kstep >> 4, bk16 = p.b_kstep >> 4;
  const uint64_t adesc0 = smem_desc(p.a_desc_hi, tiles_base);
  const uint64_t bdesc0 = smem_desc(p.b_desc_hi, tiles_base + p.a_stage_bytes);
  const uint32_t idesc = p.idesc;
  const int num_kb = p.num_kb;
  const uint32_t aatom16 = p.a_atom_bytes >> 4, batom16 = p.b_atom_bytes >> 4;
  // atoms of the last stage that still hold part of K (the rest is zero fill and is skipped)
  const int last_atoms = (p.K - (num_kb - 1) * p.kblk * p.atoms + p.kblk - 1) / p.kblk;
  uint32_t s = 0, ph = 0, it = 0;
  uint64_t adesc = adesc0, bdesc = bdesc0;
  const int n_items = kSplit ? p.num_items : p.num_tiles;
  for (int item = cluster_id; item < n_items; item += num_clusters, ++it) {
    const int tile = item_tile<kSplit>(p, item);
    if (tile < 0) {  // an empty slot of a dealt schedule: every role skips it alike, and it does not count as a tile
      --it;          // (the loop header adds the one back: buffer and phase bookkeeping follow the tiles actually computed)
      continue;
    }
    const uint32_t buf = p.acc_bufs == 2 ? (it & 1u) : 0u;
    const uint32_t aph = p.acc_bufs == 2 ? ((it >> 1) & 1u) : (it & 1u);
    if (!mbar_wait_warp(tempty0 + 8u * buf, aph ^ 1u, w, (2u << 8) | 0x80u | buf)) return;
    tc_fence_after();
    const uint32_t d_tmem = tmem_base + buf * static_cast<uint32_t>(p.bn);
    const bool rev = p.k_serpentine && (it & 1u);
    KRange kr{0, num_kb};
    if ((p.a_tri | p.b_tri) != 0 || (kSplit && item >= p.split_first_tile)) {
      const TileCoord tc = decode_tile(p, tile);
      kr = work_item<kSplit>(p, item, tile, tc.tm * (kCtaM * CG), kCtaM * CG, tc.tn * p.bn).kr;
    }
    const int n_kb = kr.hi - kr.lo;
    for (int kb = 0; kb < n_kb; ++kb) {
      if (!mbar_wait_warp(full0 + 8u * s, ph, w, (2u << 8) | s)) return;
      tc_fence_after();
      const uint32_t empty_bar = empty0 + 8u * s;
      const bool ragged_stage = (rev ? kr.hi - 1 - kb : kr.lo + kb) == num_kb - 1;  // the stage that holds the end of K
      const bool two = (p.atoms == 2) && (!ragged_stage || last_atoms == 2);
      if (p.n_mma == 2) {
        // two column groups per K step: group g reads this CTA's rows [g * b_box_rows, ...) of the B tile and
        // accumulates into tensor-memory columns [g * mma_n, ...)
        if (elect_one()) {
          const uint32_t g16 = (static_cast<uint32_t>(p.b_box_rows) * 128u) >> 4, dn = static_cast<uint32_t>(p.mma_n);
          const int n_atoms = two ? 2 : 1;
          for (int a = 0; a < n_atoms; ++a) {
            const uint64_t ad = adesc + a * aatom16, bd = bdesc + a * batom16;
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) {
              const uint32_t acc_on = static_cast<uint32_t>(kb != 0 || a != 0 || k != 0);
              if (!p.ab_fp8) {
                umma_f16<CG>(d_tmem, ad + k * ak16, bd + k * bk16, idesc, acc_on);
                umma_f16<CG>(d_tmem + dn, ad + k * ak16, bd + g16 + k * bk16, idesc, acc_on);
              } else {
                umma_f8<CG>(d_tmem, ad + k * ak16, bd + k * bk16, idesc, acc_on);
                umma_f8<CG>(d_tmem + dn, ad + k * ak16, bd + g16 + k * bk16, idesc, acc_on);
              }
            }
          }
          if constexpr (CG == 1) umma_commit<1>(empty_bar);
          else umma_commit_pair_mcast(empty_bar, 3);
        }
      } else if (elect_one()) {
        if (!p.ab_fp8) {
          umma_f16<CG>(d_tmem, adesc, bdesc, idesc, static_cast<uint32_t>(kb != 0));
#pragma unroll
          for (uint32_t k = 1; k < kBlockK / kUmmaK; ++k) umma_f16<CG>(d_tmem, adesc + k * ak16, bdesc + k * bk16, idesc, 1u);
          if (two) {
#pragma unroll
            for (uint32_t k = 0; k < kBlockK / kUmmaK; ++k)
              umma_f16<CG>(d_tmem, adesc + aatom16 + k * ak16, bdesc + batom16 + k * bk16, idesc, 1u);
          }
        } else {  // four 32-byte steps per 128-byte slice, as above
          umma_f8<CG>(d_tmem, adesc, bdesc, idesc, static_cast<uint32_t>(kb != 0));
#pragma unroll
          for (uint32_t k = 1; k < 4; ++k) umma_f8<CG>(d_tmem, adesc + k * ak16, bdesc + k * bk16, idesc, 1u);
          if (two) {
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) umma_f8<CG>(d_tmem, adesc + aatom16 + k * ak16, bdesc + batom16 + k * bk16, idesc, 1u);
          }
        }
        // ring slot reusable once these MMAs have read it (both CTAs of a pair are told at once)
        if constexpr (CG == 1) umma_commit<1>(empty_bar);
        else umma_commit_pair_mcast(empty_bar, 3);
      }
      __syncwarp();
      adesc += stage16;
      bdesc += stage16;
      if (++s == nstages) {
        s = 0;
        ph ^= 1u;
        adesc = adesc0;
        bdesc = bdesc0;
      }
    }
    if (elect_one()) {  // accumulator complete
      if constexpr (CG == 1) umma_commit<1>(tfull0 + 8u * buf);
      else umma_commit_pair_mcast(tfull0 + 8u * buf, 3);
    }
    __syncwarp();
  }
}

// Partial tiles travel through the workspace in the order the epilogue threads hold them, not row-major: the 32
// accumulator columns of TMEM lane quarter q, column group g are eight 512-byte rows, one float4 per lane, so that
// every warp-wide store and load is one contiguous 512-byte access.  Offset (in float4) of row j of group (q, g):
__device__ __forceinline__ size_t partial_f4(uint32_t q, int g, int groups, int j) {
  return (static_cast<size_t>(q) * groups + g) * 256 + static_cast<size_t>(j) * 32;
}
// Fetch the eight float4 of one (q, g) group of one partial tile (issued together: one round trip to L2).
__device__ __forceinline__ void load_partial(float4 (&v)[8], const float4* tile, uint32_t q, int g, int groups, uint32_t lane) {
#pragma unroll
  for (int j = 0; j < 8; ++j) v[j] = __ldcg(tile + partial_f4(q, g, groups, j) + lane);
}
__device__ __forceinline__ void add_partial(uint32_t (&acc)[32], const float4 (&v)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    acc[4 * j + 0] = __float_as_uint(__uint_as_float(acc[4 * j + 0]) + v[j].x);
    acc[4 * j + 1] = __float_as_uint(__uint_as_float(acc[4 * j + 1]) + v[j].y);
    acc[4 * j + 2] = __float_as_uint(__uint_as_float(acc[4 * j + 2]) + v[j].z);
    acc[4 * j + 3] = __float_as_uint(__uint_as_float(acc[4 * j + 3]) + v[j].w);
  }
}

template <int CG, int EPI_WG, bool kSplit = false>
__device__ __forceinline__ void epilogue_role(const DenseParams& p, const CUtensorMap* tmD, uint32_t staging, uint32_t tfull0,
                                              uint32_t tempty0, uint32_t tmem_base, uint32_t cta_rank, int cluster_id,
                                              int num_clusters, const WaitCtx& w) {
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t lane = lane_id();
  const uint32_t q = warp & 3u;            // TMEM lane quarter this warp may read
  const uint32_t ew = warp - 2u;           // epilogue warp index
  const uint32_t wg = ew >> 2;             // epilogue warpgroup: takes every EPI_WG-th slab
  const uint32_t stg = staging + ew * (2u * kSlabBytes);
  const int slab_cols = (p.out_dtype == 2) ? 32 : 64;
  const int nslabs = p.bn / slab_cols;
  uint32_t it = 0, nstore = 0;
  const int n_items = kSplit ? p.num_items : p.num_tiles;
  const size_t partial_elems = static_cast<size_t>(kCtaM) * p.bn;
  for (int item = cluster_id; item < n_items; item += num_clusters, ++it) {
    const int tile = item_tile<kSplit>(p, item);
    if (tile < 0) {  // an empty slot of a dealt schedule: every role skips it alike, and it does not count as a tile
      --it;          // (the loop header adds the one back: buffer and phase bookkeeping follow the tiles actually computed)
      continue;
    }
    const TileCoord tc = decode_tile(p, tile);
    const uint32_t buf = p.acc_bufs == 2 ? (it & 1u) : 0u;
    const uint32_t ph = p.acc_bufs == 2 ? ((it >> 1) & 1u) : (it & 1u);
    if (!mbar_wait_warp(tfull0 + 8u * buf, ph, w, (3u << 8) | buf, 64u)) return;  // whole warp leaves the wait together
    tc_fence_after();
    // split tile: slice `slice` of `p.split`; the partials of slices 1.. live at part0, flags at flag0
    int slice = -1;
    float* part0 = nullptr;
    unsigned long long* flag0 = nullptr;
    if (kSplit && item >= p.split_first_tile) {
      slice = (item - p.split_first_tile) - (tile - p.split_first_tile) * p.split;
      const size_t first = (static_cast<size_t>(tile - p.split_first_tile) * CG + cta_rank) * (p.split - 1);
      part0 = p.partials + first * partial_elems;
      flag0 = p.split_flags + first;
    }
    if (kSplit && slice > 0) {
      // contributor: the raw accumulators go to the workspace, 32 columns at a time, then the flag is raised
      const uint32_t t_rowc = tmem_base + ((q * 32u) << 16) + buf * static_cast<uint32_t>(p.bn);
      float4* dst = reinterpret_cast<float4*>(part0 + static_cast<size_t>(slice - 1) * partial_elems);
      const int groups = p.bn / 32;
      for (int g = static_cast<int>(wg); g < p.bn / 32; g += EPI_WG) {
        uint32_t acc[32];
        tmem_ld_32x32(t_rowc + static_cast<uint32_t>(g * 32), acc);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          __stcg(dst + partial_f4(q, g, groups, j) + lane, make_float4(__uint_as_float(acc[4 * j]), __uint_as_float(acc[4 * j + 1]), __uint_as_float(acc[4 * j + 2]),
                                     __uint_as_float(acc[4 * j + 3])));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if constexpr (CG == 1) mbar_arrive(tempty0 + 8u * buf);
        else mbar_arrive_cluster(mapa(tempty0 + 8u * buf, 0));
      }
      // the barrier orders every epilogue warp's stores before the one releasing store of the flag
      named_barrier_sync(2, 128 * EPI_WG);
      if (ew == 0 && lane == 0) st_release_gpu_u64(flag0 + (slice - 1), p.split_tag);
      continue;
    }
    if (kSplit && slice == 0) {  // reducer: the other slices of this tile run in the same wave; wait for their partials
      if (!flags_wait_warp(flag0, p.split - 1, p.split_tag, w, (3u << 8) | 0x40u)) return;  // (at most 16 slices)
    }
    const int row0 = tc.tm * (kCtaM * CG) + static_cast<int>(cta_rank) * kCtaM + static_cast<int>(q) * 32;
    const long long row = row0 + static_cast<int>(lane);
    const uint32_t t_row = tmem_base + ((q * 32u) << 16) + buf * static_cast<uint32_t>(p.bn);
    for (int sl = static_cast<int>(wg); sl < nslabs; sl += EPI_WG, ++nstore) {
      const int col0 = tc.tn * p.bn + sl * slab_cols;
      const uint32_t sbuf = stg + (nstore & 1u) * kSlabBytes;
      if (lane == 0) bulk_wait_group_read<1>();  // the store that last read this slab buffer is done
      __syncwarp();
      const uint32_t srow = sbuf + lane * 128u;
      const uint32_t sw = lane & 7u;
      uint32_t acc[32];
      float v[32];
      if (p.out_dtype == 2) {
        tmem_ld_32x32(t_row + static_cast<uint32_t>(sl * 32), acc);
        if (kSplit && slice == 0) {
          // The partials are requested while the tensor-memory read is in flight, and two slices' loads are kept in
          // flight: one after the other, every slice cost a round trip to L2 (about 0.5 us each on 256 x 256 x 32768
          // with 16 slices).  Added in slice order all the same.
          // (with two epilogue warpgroups the register limit is 168 and there is nothing to spare: one slice at a time)
          const int n = p.split - 1;
          const int groups = p.bn / 32;
          float4 pa[8];
          load_partial(pa, reinterpret_cast<const float4*>(part0), q, sl, groups, lane);
          if constexpr (EPI_WG == 1) {
            float4 pb[8];
            if (n > 1) load_partial(pb, reinterpret_cast<const float4*>(part0 + partial_elems), q, sl, groups, lane);
            tmem_ld_wait();
            for (int sidx = 0; sidx < n; sidx += 2) {
              add_partial(acc, pa);
              if (sidx + 2 < n) load_partial(pa, reinterpret_cast<const float4*>(part0 + (sidx + 2) * partial_elems), q, sl, groups, lane);
              if (sidx + 1 < n) {
                add_partial(acc, pb);
                if (sidx + 3 < n) load_partial(pb, reinterpret_cast<const float4*>(part0 + (sidx + 3) * partial_elems), q, sl, groups, lane);
              }
            }
          } else {
            tmem_ld_wait();
            add_partial(acc, pa);
            for (int sidx = 1; sidx < n; ++sidx) {  // further slices, in slice order
              load_partial(pa, reinterpret_cast<const float4*>(part0 + sidx * partial_elems), q, sl, groups, lane);
              add_partial(acc, pa);
            }
          }
        } else {
          tmem_ld_wait();
        }
        epilogue_math(v, acc, p, row, col0, tc.batch);
        store_ragged_columns(p, v, row, col0, tc.batch);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          st_shared_v4(srow + ((static_cast<uint32_t>(j) ^ sw) << 4), __float_as_uint(v[4 * j]), __float_as_uint(v[4 * j + 1]),
                       __float_as_uint(v[4 * j + 2]), __float_as_uint(v[4 * j + 3]));
      } else {
        // both halves of the 64-column slab are requested before the single wait, so their TMEM latencies overlap
        uint32_t acc1[32];
        tmem_ld_32x32(t_row + static_cast<uint32_t>(sl * 64), acc);
        tmem_ld_32x32(t_row + static_cast<uint32_t>(sl * 64 + 32), acc1);
        if (kSplit && slice == 0) {
          const int n = p.split - 1;
          const int groups = p.bn / 32;
          if constexpr (EPI_WG == 1) {  // (registers to spare: two slices' loads in flight, as above)
            float4 pa[8], pa1[8], pb[8], pb1[8];
            load_partial(pa, reinterpret_cast<const float4*>(part0), q, 2 * sl, groups, lane);
            load_partial(pa1, reinterpret_cast<const float4*>(part0), q, 2 * sl + 1, groups, lane);
            if (n > 1) {
              load_partial(pb, reinterpret_cast<const float4*>(part0 + partial_elems), q, 2 * sl, groups, lane);
              load_partial(pb1, reinterpret_cast<const float4*>(part0 + partial_elems), q, 2 * sl + 1, groups, lane);
            }
            tmem_ld_wait();
            for (int sidx = 0; sidx < n; sidx += 2) {
              add_partial(acc, pa);
              add_partial(acc1, pa1);
              if (sidx + 2 < n) {
                load_partial(pa, reinterpret_cast<const float4*>(part0 + (sidx + 2) * partial_elems), q, 2 * sl, groups, lane);
                load_partial(pa1, reinterpret_cast<const float4*>(part0 + (sidx + 2) * partial_elems), q, 2 * sl + 1, groups, lane);
              }
              if (sidx + 1 < n) {
                add_partial(acc, pb);
                add_partial(acc1, pb1);
                if (sidx + 3 < n) {
                  load_partial(pb, reinterpret_cast<const float4*>(part0 + (sidx + 3) * partial_elems), q, 2 * sl, groups, lane);
                  load_partial(pb1, reinterpret_cast<const float4*>(part0 + (sidx + 3) * partial_elems), q, 2 * sl + 1, groups, lane);
                }
              }
            }
          } else {
            float4 pv[8], pv1[8];
            load_partial(pv, reinterpret_cast<const float4*>(part0), q, 2 * sl, groups, lane);
            load_partial(pv1, reinterpret_cast<const float4*>(part0), q, 2 * sl + 1, groups, lane);
            tmem_ld_wait();
            add_partial(acc, pv);
            add_partial(acc1, pv1);
            for (int sidx = 1; sidx < n; ++sidx) {
              load_partial(pv, reinterpret_cast<const float4*>(part0 + sidx * partial_elems), q, 2 * sl, groups, lane);
              load_partial(pv1, reinterpret_cast<const float4*>(part0 + sidx * partial_elems), q, 2 * sl + 1, groups, lane);
              add_partial(acc, pv);
              add_partial(acc1, pv1);
            }
          }
        } else {
          tmem_ld_wait();
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          epilogue_math(v, h == 0 ? acc : acc1, p, row, col0 + h * 32, tc.batch);
          store_ragged_columns(p, v, row, col0 + h * 32, tc.batch);
          uint32_t pk[16];
          if (p.out_dtype == 0) {
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(v[2 * j], v[2 * j + 1]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[j] = pack_f16x2(v[2 * j], v[2 * j + 1]);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j)
            st_shared_v4(srow + ((static_cast<uint32_t>(4 * h + j) ^ sw) << 4), pk[4 * j], pk[4 * j + 1], pk[4 * j + 2],
                         pk[4 * j + 3]);
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        if (row0 < p.M && col0 < p.n_full) {
          if (p.l2_hint_d) tma_store_3d_hint(tmD, sbuf, col0, row0, tc.batch, l2_policy_evict_first());
          else tma_store_3d(tmD, sbuf, col0, row0, tc.batch);
        }
        bulk_commit_group();
      }
    }
    // every tcgen05.ld of this accumulator buffer has completed: hand it back to the MMA issuer
    tc_fence_before();
    __syncwarp();
    if (lane == 0) {
      if constexpr (CG == 1) mbar_arrive(tempty0 + 8u * buf);
      else mbar_arrive_cluster(mapa(tempty0 + 8u * buf, 0));
    }
    if (kSplit && slice == 0) {  // every epilogue warp has read the partials: lower the flags for the next launch
      named_barrier_sync(2, 128 * EPI_WG);
      if (ew == 0 && lane == 0)
        for (int sidx = 0; sidx < p.split - 1; ++sidx) flag0[sidx] = 0ull;
    }
  }
  if (lane == 0) bulk_wait_group_read<0>();  // staging may be released; the writes themselves complete with the grid
}

template <int CG, int EPI_WG, bool kSplit = false>
__global__ void __launch_bounds__(64 + 128 * EPI_WG, 1)
dense_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmD, const DenseParams p) {
  extern __shared__ uint8_t smem_raw[];
  griddep_launch_dependents();  // the next kernel's set-up may overlap this one; it waits below before touching global memory
  const uint32_t raw = smem_addr(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte swizzle atoms need 1024-byte alignment
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t cta_rank = (CG == 2) ? cluster_ctarank() : 0u;
  const int cluster_id = static_cast<int>(blockIdx.x) / CG;
  const int num_clusters = static_cast<int>(gridDim.x) / CG;

  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const uint32_t staging_off = static_cast<uint32_t>(p.stages) * stage_bytes;
  const uint32_t bars_off = staging_off + 4u * EPI_WG * 2u * kSlabBytes;
  const uint32_t full0 = base + bars_off;
  const uint32_t empty0 = full0 + 8u * kMaxStages;
  const uint32_t tfull0 = empty0 + 8u * kMaxStages;
  const uint32_t tempty0 = tfull0 + 16u;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + bars_off + 16u * kMaxStages + 32u);
  volatile uint32_t* s_abort = tmem_slot + 1;
  const WaitCtx w{s_abort, p.status, p.timeout_ns};

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull0 + 8u * b, 1);
      mbar_init(tempty0 + 8u * b, 4u * EPI_WG * CG);
    }
    *s_abort = 0u;
    fence_mbar_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    prefetch_tensormap(&tmD);
  }
  if (warp == 1) {
    tmem_alloc<CG>(smem_addr(const_cast<uint32_t*>(tmem_slot)), p.tmem_cols);
    tmem_relinquish<CG>();
  }
  uint32_t tmem_base = 0;
  if (CG == 1 && warp == 0) {
    // A single CTA's producer needs the barriers (set up by its own lane 0) and nothing else: it announces them to
    // the other warps and starts the loads while those are still waiting for the tensor-memory allocation.
    __syncwarp();
    named_barrier_arrive(3, blockDim.x);
    producer_role<CG, kSplit>(p, &tmA, &tmB, base, full0, empty0, cta_rank, cluster_id, num_clusters, w);
  } else if (CG == 2 && warp == 0) {
    __syncwarp();  // (lane 0 set the barriers up)
    producer_role<CG, kSplit, true>(p, &tmA, &tmB, base, full0, empty0, cta_rank, cluster_id, num_clusters, w);
  } else {
    tc_fence_before();
    if constexpr (CG == 1) {
      named_barrier_sync(3, blockDim.x);
    } else {
      __syncthreads();
      cluster_arrive();  // the peer's barriers must exist before anything signals them
      cluster_wait();
    }
    tc_fence_after();
    tmem_base = *tmem_slot;
    // barriers and tensor memory are set up; from here on global memory is read and written (the producer warp makes
    // this wait itself, once it has worked out its first tile)
    if (warp != 0) griddep_wait();
  }

  if (warp == 0) {
    // (ran above)
  } else if (warp == 1) {
    if (cta_rank == 0) mma_role<CG, kSplit>(p, base, full0, empty0, tfull0, tempty0, tmem_base, cluster_id, num_clusters, w);
  } else {
    epilogue_role<CG, EPI_WG, kSplit>(p, &tmD, base + staging_off, tfull0, tempty0, tmem_base, cta_rank, cluster_id, num_clusters, w);
  }

  tc_fence_before();
  __syncthreads();
  if constexpr (CG == 2) {  // neither CTA may free tensor memory or exit while its peer still uses the pair
    cluster_arrive();
    cluster_wait();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<CG>(tmem_base, p.tmem_cols);
  }
}

}  // namespace b200

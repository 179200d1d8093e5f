// Host side of the b200 GEMM library: the C ABI of include/gemm.h.
//   gemm_plan  : validation, roofline classification, variant / tile / stage / raster choice (host only)
//   gemm_run   : tensor-map encoding and the kernel launch (asynchronous)
// No cuBLAS / CUTLASS, no fallback path: an unsupported request is an error code.
#include "../../include/gemm.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <queue>
#include <random>
#include <utility>
#include <vector>

#include "dense_kernel.cuh"
#include "mirror_kernel.cuh"
#include "skinny_kernel.cuh"
#include "tune_cache.h"
#include "wide_kernel.cuh"

using namespace b200;

namespace {

constexpr int kDefaultSmCount = 148;        // B200
constexpr int kMaxSmemOptin = 232448;       // 227 KB dynamic shared memory per CTA on sm_100
// Machine ridges for the plan-time roofline class (FLOP per byte): tensor-core ridge and CUDA-core ridge
// from the public B200 figures (2250 TFLOP/s dense 16-bit, about 75 TFLOP/s fp32 FMA, 8 TB/s HBM3e).
constexpr double kRidgeTensor = 2250.0e12 / 8.0e12;
constexpr double kRidgeCudaCore = 75.0e12 / 8.0e12;

thread_local char g_last_cuda_error[160] = "";

void note_cuda_error(const char* what, const char* name) {
  snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "%s: %s", what, name ? name : "?");
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode_fn() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
  });
  return fn;
}

bool is_fp8(int dtype) { return dtype == GEMM_FP8_E4M3 || dtype == GEMM_FP8_E5M2; }
int elem_bytes(int dtype) { return dtype == GEMM_F32 ? 4 : (is_fp8(dtype) ? 1 : 2); }
// elements of K in one 128-byte swizzle row of an operand
int kblk_of(int ab_dtype) { return is_fp8(ab_dtype) ? 2 * kBlockK : kBlockK; }
// format code of the instruction descriptor: kind::f16 0 = f16, 1 = bf16; kind::f8f6f4 0 = E4M3, 1 = E5M2
int ab_format(int ab_dtype) { return (ab_dtype == GEMM_BF16 || ab_dtype == GEMM_FP8_E5M2) ? 1 : 0; }

CUtensorMapDataType tm_dtype(int dtype) {
  if (is_fp8(dtype)) return CU_TENSOR_MAP_DATA_TYPE_UINT8;  // the copy engine only moves the bytes
  return dtype == GEMM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                            : (dtype == GEMM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32);
}

// 3-D tiled map over a row-major matrix batch: dim0 = contiguous extent, dim1 = rows, dim2 = batch.
// 128-byte swizzle (or, for a store from a plain row-major staging buffer, none), out-of-bounds elements read as zero /
// are not written.
bool encode_map(CUtensorMap* m, int dtype, const void* base, uint64_t inner, uint64_t rows, uint64_t batch, uint64_t ld,
                uint64_t batch_stride, uint32_t box_inner, uint32_t box_rows, bool swizzle = true) {
  EncodeFn fn = get_encode_fn();
  if (!fn) {
    note_cuda_error("cuTensorMapEncodeTiled", "driver entry point not found");
    return false;
  }
  const uint64_t eb = static_cast<uint64_t>(elem_bytes(dtype));
  cuuint64_t dims[3] = {inner, rows, batch};
  cuuint64_t strides[2] = {ld * eb, (batch > 1 ? batch_stride : rows * ld) * eb};
  cuuint32_t box[3] = {box_inner, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  // L2 fetches in 256-byte units only when the rows start on 128-byte lines: with any other pitch seven of eight box
  // rows straddle two lines, and promoting each straddled piece to 256 bytes over-fetches (measured on
  // 4100 x 4104 x 4104: 164 -> 144 us without promotion; no difference on aligned pitches)
  const CUtensorMapL2promotion promotion = (ld * eb) % 128 == 0 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE;
  CUresult r = fn(m, tm_dtype(dtype), 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, promotion, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char buf[64];
    snprintf(buf, sizeof buf, "CUresult %d", static_cast<int>(r));
    note_cuda_error("cuTensorMapEncodeTiled", buf);
    return false;
  }
  return true;
}

int ceil_div(long long a, long long b) { return static_cast<int>((a + b - 1) / b); }

}  // namespace

namespace {

// Tensor maps a plan has already encoded, by operand address.  Everything else a map depends on (extents, pitches,
// box, element type) is fixed by the plan, so the base address alone identifies it.  One table per operand (A, B, D): a
// caller that keeps its weights and changes its activations still finds two of the three.  256 entries each, eight
// probes from a hash of the address, the oldest of the eight replaced on a miss (a loop over 126 buffer sets, the
// benchmark's small configuration, then never misses; with 128 entries and four probes it re-encoded about every third
// map).  Several host threads may run one plan, hence the lock (held for a 128-byte copy).
struct MapCache {
  static constexpr int kEntries = 256, kProbes = 8;
  struct alignas(64) Entry {
    CUtensorMap map;
    const void* key;
    uint64_t stamp;  // 0 = empty
  };
  Entry table[3][kEntries];
  uint64_t clock = 0;
  std::atomic_flag lock = ATOMIC_FLAG_INIT;
  MapCache() { memset(table, 0, sizeof table); }
  static int slot_of(const void* key) {
    uint64_t h = reinterpret_cast<uintptr_t>(key) >> 4;  // (operands are 16-byte aligned)
    h *= 0x9E3779B97F4A7C15ull;
    return static_cast<int>(h >> 56);  // 8 bits
  }
  // True and *out filled when `key` is known for operand `which`.
  bool find(int which, const void* key, CUtensorMap* out) {
    const int s0 = slot_of(key);
    bool hit = false;
    while (lock.test_and_set(std::memory_order_acquire)) {
    }
    for (int i = 0; i < kProbes; ++i) {
      Entry& e = table[which][(s0 + i) & (kEntries - 1)];
      if (e.stamp != 0 && e.key == key) {
        *out = e.map;
        e.stamp = ++clock;
        hit = true;
        break;
      }
    }
    lock.clear(std::memory_order_release);
    return hit;
  }
  void insert(int which, const void* key, const CUtensorMap& m) {
    const int s0 = slot_of(key);
    while (lock.test_and_set(std::memory_order_acquire)) {
    }
    Entry* victim = &table[which][s0];
    for (int i = 0; i < kProbes; ++i) {
      Entry& e = table[which][(s0 + i) & (kEntries - 1)];
      if (e.stamp != 0 && e.key == key) {  // (another thread got there first)
        victim = &e;
        break;
      }
      if (e.stamp < victim->stamp) victim = &e;
    }
    victim->map = m;
    victim->key = key;
    victim->stamp = ++clock;
    lock.clear(std::memory_order_release);
  }
};

}  // namespace

struct gemm_plan_s {
  gemm_desc_t d;
  gemm_info_t info;
  int variant;     // gemm_variant_t
  int cg;          // CTAs per tile (dense)
  int epi_wg;      // epilogue warpgroups (dense)
  int bn;          // tile N (dense)
  int stages;
  int raster_group;
  int grid;
  int smem_bytes;
  int sm_count;
  int device;            // CUDA device the plan was made on (-1: none); runs must use the same one
  bool has_device;
  bool arch_ok;
  uint32_t* d_status;       // device: 16-byte status word
  uint32_t* h_status = nullptr;  // page-locked host copy written by gemm_plan_status_async (made on first use)
  uint64_t tag_base = 0;        // plan identity, bits 24-47 of every run's tag (see run_tag)
  MapCache* maps = nullptr;     // tensor maps already encoded for this plan, by operand address (made on first run)
  int split = 1;                // tail split factor of a dense plan
  int d_tri = 0;                // one triangle of D wanted: 1 lower, 2 upper (dense variants)
  int* d_tile_list = nullptr;   // device: the dealt tile schedule of one matrix (structured problems)
  int* h_tile_list = nullptr;   // host copy (uploaded at plan time; gemm_plan_schedule walks it)
  ~gemm_plan_s() {
    free(h_tile_list);
    delete maps;
  }
  size_t split_flag_bytes = 0;  // head of a tail-split plan's workspace: one 64-bit flag word per partial tile
  unsigned long long runs = 0;  // launches so far (the timeout test hook acts on the first one only)
  uint32_t timeout_ms;
  DenseParams dense;     // filled at plan time except pointers / scalars
  SkinnyPlan skinny;     // stream-K decomposition of the skinny variant
  bool skinny_tall = false;  // the short output extent is N (A is the streamed operand), not M
};

namespace {

bool has_bias(int epi) { return (epi & 1) != 0; }  // the odd gemm_epilogue_t values

gemm_status_t validate(const gemm_desc_t* d) {
  if (d->struct_size != sizeof(gemm_desc_t)) return GEMM_ERR_INVALID_ARG;
  if (d->M < 1 || d->N < 1 || d->K < 1 || d->batch_count < 1) return GEMM_ERR_INVALID_ARG;
  if (d->M > 0x7FFFFFFFll || d->N > 0x7FFFFFFFll || d->K > 0x7FFFFFFFll) return GEMM_ERR_INVALID_ARG;
  if ((d->transa != GEMM_OP_N && d->transa != GEMM_OP_T) || (d->transb != GEMM_OP_N && d->transb != GEMM_OP_T))
    return GEMM_ERR_INVALID_ARG;
  if (d->ab_dtype < GEMM_BF16 || d->ab_dtype > GEMM_FP8_E5M2 || d->c_dtype < GEMM_BF16 || d->c_dtype > GEMM_F32)
    return GEMM_ERR_INVALID_ARG;
  if (d->epilogue < GEMM_EPI_NONE || d->epilogue > GEMM_EPI_BIAS_SILU) return GEMM_ERR_INVALID_ARG;
  if ((d->flags & GEMM_FLAG_A_LOWER) && (d->flags & GEMM_FLAG_A_UPPER)) return GEMM_ERR_INVALID_ARG;
  if ((d->flags & GEMM_FLAG_D_LOWER) && (d->flags & GEMM_FLAG_D_UPPER)) return GEMM_ERR_INVALID_ARG;
  if ((d->structure & ~(GEMM_STRUCT_B_LOWER | GEMM_STRUCT_B_UPPER | GEMM_STRUCT_D_MIRROR)) || (d->options & ~GEMM_OPT_STREAMK_WORKSPACE)) return GEMM_ERR_INVALID_ARG;
  if ((d->structure & GEMM_STRUCT_D_MIRROR) && (!(d->flags & (GEMM_FLAG_D_LOWER | GEMM_FLAG_D_UPPER)) || d->M != d->N || d->batch_count > 65535))
    return GEMM_ERR_INVALID_ARG;  // a triangle to copy from, and a square D
  if ((d->structure & GEMM_STRUCT_B_LOWER) && (d->structure & GEMM_STRUCT_B_UPPER)) return GEMM_ERR_INVALID_ARG;
  if (d->ab_dtype == GEMM_F32) return GEMM_ERR_UNSUPPORTED;
  // 8-bit operands: K-contiguous storage only (A stored M x K, B stored N x K)
  if (is_fp8(d->ab_dtype) && (d->transa != GEMM_OP_N || d->transb != GEMM_OP_T)) return GEMM_ERR_UNSUPPORTED;
  const int64_t a_row = d->transa == GEMM_OP_N ? d->K : d->M;
  const int64_t b_row = d->transb == GEMM_OP_N ? d->N : d->K;
  if (d->lda < a_row || d->ldb < b_row || d->ldc < d->N) return GEMM_ERR_INVALID_ARG;
  const int64_t a_rows = d->transa == GEMM_OP_N ? d->M : d->K;
  const int64_t b_rows = d->transb == GEMM_OP_N ? d->K : d->N;
  if (d->batch_count > 1) {
    if (d->stride_a < 0 || d->stride_b < 0 || d->stride_c < 0) return GEMM_ERR_INVALID_ARG;
    if (d->stride_c < (d->M - 1) * d->ldc + d->N) return GEMM_ERR_INVALID_ARG;  // outputs would overlap
    if (d->stride_a == 0 || d->stride_b == 0) return GEMM_ERR_UNSUPPORTED;      // operand broadcast
    (void)a_rows;
    (void)b_rows;
  }
  const int eab = elem_bytes(d->ab_dtype), ec = elem_bytes(d->c_dtype);
  if ((d->lda * eab) % 16 || (d->ldb * eab) % 16 || (d->ldc * ec) % 16) return GEMM_ERR_ALIGNMENT;
  if (d->batch_count > 1 && ((d->stride_a * eab) % 16 || (d->stride_b * eab) % 16 || (d->stride_c * ec) % 16))
    return GEMM_ERR_ALIGNMENT;
  return GEMM_OK;
}

int dense_smem_bytes(int stages, int a_stage, int b_stage, int epi_wg) {  // a_stage, b_stage: all atoms of a stage
  return 1024 /*alignment slack*/ + stages * (a_stage + b_stage) + 4 * epi_wg * 2 * kSlabBytes + 16 * kMaxStages + 64;
}

int d_tri_of(const gemm_desc_t& d) { return (d.flags & GEMM_FLAG_D_LOWER) ? 1 : ((d.flags & GEMM_FLAG_D_UPPER) ? 2 : 0); }

// Tile columns [*j0, *j1] of tile row i that touch the wanted triangle of D (empty when *j0 > *j1).
// Lower (row >= column): the tile's last row must reach its first column; upper: its first row must not pass its last column.
void tri_columns(int d_tri, long long i, int tile_m, int bn, long long M, long long N, int tiles_n, int* j0, int* j1) {
  *j0 = 0;
  *j1 = tiles_n - 1;
  if (d_tri == 1) {
    const long long last_row = std::min<long long>((i + 1) * tile_m, M) - 1;
    *j1 = static_cast<int>(std::min<long long>(tiles_n - 1, last_row / bn));
  } else if (d_tri == 2) {
    const long long first_row = i * tile_m;
    *j0 = first_row > N - 1 ? tiles_n : static_cast<int>(first_row / bn);
  }
}
long long tri_tile_count(int d_tri, int tile_m, int bn, long long M, long long N) {
  const int tiles_m = ceil_div(M, tile_m), tiles_n = ceil_div(N, bn);
  if (d_tri == 0) return static_cast<long long>(tiles_m) * tiles_n;
  long long n = 0;
  for (int i = 0; i < tiles_m; ++i) {
    int j0, j1;
    tri_columns(d_tri, i, tile_m, bn, M, N, tiles_n, &j0, &j1);
    if (j1 >= j0) n += j1 - j0 + 1;
  }
  return n;
}
// The schedule of a structured problem (one triangle of D wanted, triangular op(A) or op(B)): the tiles of one matrix
// that are computed at all, dealt out to `units` CTAs (pairs) ahead of time.  The tiles are taken in the order the
// scheduler visits the full grid (groups of `raster` tile rows, inside a group column by column with the row running
// fastest, so that tiles in flight together share their A band and B panels) and each goes to the CTA with the least
// work so far -- the K range of a tile under a triangular operand varies from one ring stage to all of K, and a
// round-robin deal would leave the CTAs unevenly loaded.  Slot k * units + c holds the k-th tile of CTA c (tile id
// of the full tiles_m x tiles_n numbering), -1 where that CTA has none; the kernels walk their slots in order.
struct TileSchedule {
  std::vector<int> slots;
  int units = 0;        // CTAs (pairs) dealt to
  long long tiles = 0;  // real tiles
};
// `batches` > 1: the tiles of all matrices are dealt together (the list then holds tile ids of the whole batch).
TileSchedule deal_tiles(const gemm_desc_t& d, int tile_m, int bn, int raster, int kstep, int num_kb, int max_units, int batches = 1) {
  const int d_tri = d_tri_of(d);
  const int a_tri = (d.flags & GEMM_FLAG_A_LOWER) ? 1 : ((d.flags & GEMM_FLAG_A_UPPER) ? 2 : 0);
  const int b_tri = (d.structure & GEMM_STRUCT_B_LOWER) ? 1 : ((d.structure & GEMM_STRUCT_B_UPPER) ? 2 : 0);
  const int tiles_m = ceil_div(d.M, tile_m), tiles_n = ceil_div(d.N, bn);
  struct Item {
    int tile;
    long long work;
  };
  std::vector<Item> order;
  for (int b = 0; b < batches; ++b) {
  int t = b * tiles_m * tiles_n;
  for (int first = 0; first < tiles_m; first += raster) {
    const int gm = std::min(raster, tiles_m - first);
    for (int tn = 0; tn < tiles_n; ++tn)
      for (int r = 0; r < gm; ++r, ++t) {
        const long long tm = first + r;
        int j0, j1;
        tri_columns(d_tri, tm, tile_m, bn, d.M, d.N, tiles_n, &j0, &j1);
        if (tn < j0 || tn > j1) continue;
        // ring stages this tile visits (the kernel's k_range) -> tensor-pipe cycles, plus what a tile costs besides
        long long lo = 0, hi = num_kb;
        const long long row0 = tm * tile_m, col0 = static_cast<long long>(tn) * bn;
        if (a_tri == 1) hi = std::min<long long>(hi, (std::min<long long>(row0 + tile_m, d.M) - 1) / kstep + 1);
        else if (a_tri == 2) lo = std::max<long long>(lo, row0 / kstep);
        if (b_tri == 1) lo = std::max<long long>(lo, col0 / kstep);
        else if (b_tri == 2) hi = std::min<long long>(hi, (std::min<long long>(col0 + bn, d.N) - 1) / kstep + 1);
        const long long stages = std::max<long long>(1, hi - lo);
        order.push_back(Item{t, stages * (kstep / 64) * 2 * bn + 1000});
      }
  }
  }
  TileSchedule sch;
  sch.tiles = static_cast<long long>(order.size());
  sch.units = static_cast<int>(std::max<long long>(1, std::min<long long>(max_units, sch.tiles)));
  std::vector<std::vector<int>> mine(sch.units);
  using Load = std::pair<long long, int>;  // (work so far, CTA): the least loaded CTA, the lowest index among equals
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
  for (int c = 0; c < sch.units; ++c) heap.push(Load(0, c));
  for (const Item& it : order) {
    Load l = heap.top();
    heap.pop();
    mine[l.second].push_back(it.tile);
    heap.push(Load(l.first + it.work, l.second));
  }
  size_t rounds = 1;
  for (const auto& v : mine) rounds = std::max(rounds, v.size());
  sch.slots.assign(rounds * sch.units, -1);
  for (int c = 0; c < sch.units; ++c)
    for (size_t k = 0; k < mine[c].size(); ++k) sch.slots[k * sch.units + c] = mine[c][k];
  return sch;
}

// The tile scheduler's plan-time divisors (see FastDiv).  False if a division came out wrong (it cannot; checked on
// the values the scheduler will actually meet at the ends of each range, so that a mistake here fails at plan time).
bool set_scheduler_divisors(DenseParams& p) {
  const uint32_t per_matrix = static_cast<uint32_t>(p.tiles_m) * p.tiles_n;
  const uint32_t group = static_cast<uint32_t>(p.raster_group) * p.tiles_n;
  const uint32_t last_rows = p.tiles_m % p.raster_group ? p.tiles_m % p.raster_group : p.raster_group;
  const uint32_t list = p.list_len > 0 ? p.list_len : 1;
  p.fd_matrix = make_fastdiv(per_matrix);
  p.fd_group = make_fastdiv(group);
  p.fd_rows = make_fastdiv(p.raster_group);
  p.fd_last_rows = make_fastdiv(last_rows);
  p.fd_list = make_fastdiv(list);
  const int kstep = p.kblk * p.atoms;
  p.kstep_shift = 0;
  while ((1 << p.kstep_shift) < kstep) ++p.kstep_shift;
  if ((1 << p.kstep_shift) != kstep) return false;
  const struct {
    const FastDiv* f;
    uint32_t d;
  } all[] = {{&p.fd_matrix, per_matrix}, {&p.fd_group, group}, {&p.fd_rows, static_cast<uint32_t>(p.raster_group)},
             {&p.fd_last_rows, last_rows}, {&p.fd_list, list}};
  for (const auto& e : all)
    for (uint32_t n : {0u, 1u, e.d - 1, e.d, e.d + 1, 2 * e.d - 1, 2 * e.d, 1000003u, 0x7FFFFFFEu, 0x7FFFFFFFu, 0xFFFFFFFFu})
      if (fast_div(n, *e.f) != n / e.d) return false;
  return true;
}

// Tail split of the double-buffered dense kernels (on request, GEMM_FLAG_TAIL_SPLIT): when the tiles left over after the
// full waves occupy at most half of the CTAs (pairs), each of them is cut into this many K slices, one per CTA (pair); the slice that
// starts at K = 0 adds the others' raw accumulators from the workspace and finishes the tile.  1 = no split.
int tail_split(long long tiles, int units, int num_kb, const gemm_desc_t& d, int bn, int cg, int atoms) {
  if (bn > 256) return 1;  // (the partial-tile layout and the flag protocol are written for two accumulator buffers)
  if ((d.flags & (GEMM_FLAG_A_LOWER | GEMM_FLAG_A_UPPER | GEMM_FLAG_D_LOWER | GEMM_FLAG_D_UPPER)) || d.structure) return 1;
  const long long rem = tiles % units;
  if (rem == 0 || rem * 2 > units) return 1;
  if (tiles / units >= 8) return 1;  // many full waves: the last one is a few per cent at most; keep the plain kernel
  // s slices shorten a tile's main loop to 1 / s of its T cycles and make the reducing CTA read s - 1 partial tiles of
  // R cycles each (128 x bn floats at the 58 B/clk one SM takes from L2; the flags of all slices are polled together):
  // T / s + (s - 1) R is least at s = sqrt(T / R).  T per 128-byte K slice: the operand feed at the same rate or the
  // tensor pipe, whichever is slower.  (Measured, us at the old rule's count -> at this one's: 384 x 384 x 8192 18.0 at 3
  // -> 14.8 at 6, 256 x 512 x 8192 18.1 at 3 -> 14.5 at 9, 256 x 256 x 32768 27.0 at 7 -> 21.7 at 16; the old rule
  // charged 5000 cycles per partial tile, from before the flags were polled together.)
  const double width = bn > 0 ? bn : 128;
  const double per_slice = std::max((128.0 + width / cg) * 128.0 / 58.0, 4.0 * (width / 2.0) / 0.8);
  const double read_partial = 128.0 * width * 4.0 / 58.0;
  int by_length = static_cast<int>(std::lround(std::sqrt(static_cast<double>(num_kb) * atoms * per_slice / read_partial)));
  by_length = std::max(2, std::min(by_length, 16));
  int split = static_cast<int>(std::min<long long>(units / rem, by_length));
  split = std::min(split, num_kb / 4);  // a slice of fewer than four ring stages is all pipeline fill
  split = std::max(split, 1);
  // Without the flag only the extreme case splits by itself: a handful of tiles (no full wave) whose K is long enough for
  // three or more slices each, where whole tiles would leave most of the GPU idle for the whole run -- or for two slices
  // when K has 48 or more 128-byte slices (measured with two slices allowed: 1024 x 1024 x 4096 20.6 -> 17.8 us,
  // 2048 x 512 x 4096 20.8 -> 17.9, 1024 x 1024 x 8192 27.2 -> 25.5, but 1280 x 1280 x 2560 15.8 -> 18.5).
  if (!(d.flags & GEMM_FLAG_TAIL_SPLIT) && !(tiles < units && (split >= 3 || (split == 2 && num_kb * atoms >= 48)))) return 1;
  return split;
}

// Plan-time roofline estimate (Section 4.3 applied per kernel candidate): cycles one SM spends on its share of the
// problem with a given kernel family and tile width.  Per tile the slowest of three resources decides -- the tensor
// pipe (with the family's measured streaming efficiency), the L2 -> SM operand feed and the HBM write share -- plus
// what the family leaves exposed per tile; tiles are dealt out in waves over the SMs (or SM pairs).
struct DenseCandidate {
  int variant;
  int bn;
  double cycles;
};
double estimate_dense_cycles(const gemm_desc_t& d, int sm_count, int variant, int bn) {
  const bool wide = variant == GEMM_VARIANT_DENSE_2CTA_WIDE;
  const int cg = variant == GEMM_VARIANT_DENSE_1CTA ? 1 : 2;
  const int rows_cta = wide ? kWideCtaM : kCtaM;
  const int rows_tile = rows_cta * cg;
  const int units = std::max(1, sm_count / cg);
  const long long tiles = tri_tile_count(d_tri_of(d), rows_tile, bn, d.M, d.N) * d.batch_count;
  const double kblocks = static_cast<double>(ceil_div(d.K, kblk_of(d.ab_dtype)));  // 128-byte slices: same pipe time for either width
  double waves = static_cast<double>((tiles + units - 1) / units);
  double handover = 0.0;
  if (!wide) {  // a thinly filled last wave is split along K (two slices per stage assumed, as plan_dense will choose for long K)
    const int split = tail_split(tiles, units, static_cast<int>(kblocks) / 2, d, bn, cg, 2);
    if (split > 1) {
      waves += 1.0 / split - 1.0;
      handover = (split - 1) * (128.0 * bn * 4.0 / 58.0) + 2500.0;  // the reducing CTA reads the other slices' accumulators
    }
  }
  // tensor pipe: one 128 x bn x 16 MMA per CTA takes bn / 2 cycles; four per k-block and 128-row half
  static const double eff1[4] = {0.45, 0.68, 0.76, 0.82}, eff2[4] = {0.55, 0.80, 0.88, 0.938};  // bn = 64, 128, 192, 256 (measured: 8192^3, and K = 512 ... 4096; 192 in between)
  const int mma_n = bn > 256 ? bn / 2 : bn;  // (a tile wider than 256 columns is two MMAs side by side)
  const int bi = mma_n <= 64 ? 0 : (mma_n <= 128 ? 1 : (mma_n <= 192 ? 2 : 3));
  const double eff = wide ? 1.0 : (cg == 1 ? eff1[bi] : eff2[bi]);
  const double mma = kblocks * 4.0 * (bn / 2.0) * (rows_cta / 128.0) / eff;
  // operand feed: bytes this SM receives per k-block at ~90 B/clk (fitted on multi-wave problems; at the start of a
  // kernel, when 144-148 SMs fill their rings at once, traces show 55-58 B/clk per SM -- about 17 TB/s out of L2 in
  // total -- which is what bounds the one- and two-tile-per-CTA problems)
  // ... and half that rate when an operand's row pitch is not a multiple of 128 bytes: every row of a TMA box then
  // straddles two memory lines (measured: the families rank by loads per FLOP there, wide > pair > single CTA)
  const bool straddling = (d.lda * elem_bytes(d.ab_dtype)) % 128 != 0 || (d.ldb * elem_bytes(d.ab_dtype)) % 128 != 0;
  const double feed = kblocks * (rows_cta + static_cast<double>(bn) / cg) * 128.0 / (straddling ? 45.0 : 90.0);
  // output: this SM's share of the HBM write bandwidth is ~16 B/clk
  const double out = static_cast<double>(rows_cta) * bn * elem_bytes(d.c_dtype) / 16.0;
  const bool gelu = d.epilogue >= GEMM_EPI_GELU_ERF;  // any transcendental activation
  double exposed = 900.0;                       // barrier round trips per tile that nothing hides (fitted at K = 512, 1024)
  // no second accumulator: read-out (and bias fetch, conversion) of half 0; fitted, like the pair efficiency above, to
  // measured pair-vs-wide time ratios at K = 4096 ... 16384 on 8192 x 8192 and 16384 x 14336 outputs
  if (wide) exposed = (gelu ? 13000.0 : 5100.0) + (has_bias(d.epilogue) ? 1300.0 : 0.0);
  else if (cg == 2) exposed = 1000.0;           // pair hand-shakes cross the SM-to-SM network
  // a tile wider than 256 columns has a single accumulator buffer: its whole read-out (eight warps, about 900 cycles per
  // 64-column slab and warp) stands between two tiles; and at the end of the kernel it is longer than a narrow tile's
  if (!wide && bn > 256) exposed += (bn / 64) / 2.0 * 900.0;
  // what is exposed stalls the tensor pipe, so it adds to the compute side; an output-bound tile instead pays a small
  // switch-over per tile (measured on the batched short-K shape: fewer, larger tiles win)
  const double per_tile = std::max(std::max(mma, feed) + exposed, out + 300.0);
  // (fitted: against a second, partly filled wave of narrower tiles the one wave of wide tiles does about 8 % better than
  // this estimate says -- measured 2304^3 23.0 us against 27.0, 2560^3 27.6 / 30.5, 3072^3 42.2 / 42.8, 2816^3 37.9 / 36.9)
  const double fitted = (!wide && bn > 256) ? 0.92 : 1.0;
  return (waves * per_tile + 3000.0 + handover) * fitted;  // + pipeline fill and drain
}

// Fill plan->dense and the launch geometry for a dense variant.
gemm_status_t plan_dense(gemm_plan_s* pl, int cg, int forced_bn, int forced_raster, int forced_stages, int forced_atoms) {
  const gemm_desc_t& d = pl->d;
  const int a_kmajor = d.transa == GEMM_OP_N;
  const int b_kmajor = d.transb == GEMM_OP_T;
  const int tile_m = kCtaM * cg;
  const int tiles_m = ceil_div(d.M, tile_m);
  // tile N: the widest tile that still gives every SM (pair) work; B tiles with N contiguous are loaded in
  // 64-column boxes per CTA, so a pair needs bn % 128 == 0 there
  const int bn_step = (!b_kmajor && cg == 2) ? 128 : 64;
  int bn = forced_bn;
  if (bn == 0) {
    const int units = pl->sm_count / cg;
    bn = 256;
    while (bn > bn_step) {
      const long long tiles = tri_tile_count(d_tri_of(d), tile_m, bn, d.M, d.N) * d.batch_count;
      if (tiles >= units && d.N > bn / 2) break;
      bn -= bn_step;  // 256 -> 192 -> 128 -> 64
      if (bn == 192) bn = 128;
    }
  }
  if (bn < bn_step || bn > 512 || bn % bn_step) return GEMM_ERR_UNSUPPORTED;
  // wider than 256 columns: two MMAs per K step, one accumulator buffer (see DenseParams::mma_n); B with K contiguous only
  // (the loader for N-contiguous B moves 64-column boxes and has no notion of the two column groups)
  const bool wide_n = bn > 256;
  if (wide_n && !b_kmajor) return GEMM_ERR_UNSUPPORTED;
  const int tiles_n = ceil_div(d.N, bn);
  const int b_rows = bn / cg;
  const int a_atom = kCtaM * kBlockK * 2;
  const int b_atom = b_rows * kBlockK * 2;
  // Each ring stage ends with one tcgen05.commit, which costs tensor-pipe time; a stage of two 64-wide K slices
  // halves that cost.  Worth it when the ring still has at least three such stages (pairs; narrow 1-CTA tiles).
  const int units = pl->sm_count / cg;
  const int d_tri = d_tri_of(d);
  const long long tiles_total = tri_tile_count(d_tri, tile_m, bn, d.M, d.N) * d.batch_count;  // tiles that are computed
  const bool single_wave = tiles_total <= units;  // every CTA (pair) computes at most one tile: pure latency
  // A tile's main loop lasts about 512 cycles per 64 columns of K (at tile N = 256); draining 128 x 256 accumulators
  // with four warps takes several thousand.  Short-K (output-bound) problems with several tiles per CTA get a second
  // epilogue warpgroup (measured: a gain only up to K = 512 at tile N = 256; 7-14 % slower beyond).  A problem of one
  // 256-wide tile per CTA has nothing to hide its epilogue behind: there too eight warps drain the accumulator
  // (2048^3: 19.6 -> 18.0 us; narrower tiles measured slower with them).
  const int kblk = kblk_of(d.ab_dtype);
  const int epi_wg = ((!single_wave && static_cast<long long>(ceil_div(d.K, kblk)) * 2 * bn <= 4096) || (single_wave && bn >= 256) || wide_n) ? 2 : 1;
  int atoms = forced_atoms;
  if (atoms == 0) {
    const bool fits3 = 3 * 2 * (a_atom + b_atom) + dense_smem_bytes(0, 0, 0, epi_wg) <= kMaxSmemOptin;
    atoms = (d.K > 2 * kblk && fits3) ? 2 : 1;  // (measured by gemm_tune: also faster for one-tile-per-CTA problems)
  }
  if (atoms < 1 || atoms > 2) return GEMM_ERR_UNSUPPORTED;
  const int a_stage = atoms * a_atom;
  const int b_stage = atoms * b_atom;
  int stages = forced_stages;
  if (stages == 0) {
    stages = (kMaxSmemOptin - dense_smem_bytes(0, a_stage, b_stage, epi_wg)) / (a_stage + b_stage);
    stages = std::min(stages, 8);
  }
  if (stages < 2 || stages > kMaxStages) return GEMM_ERR_UNSUPPORTED;
  const int smem = dense_smem_bytes(stages, a_stage, b_stage, epi_wg);
  if (smem > kMaxSmemOptin) return GEMM_ERR_UNSUPPORTED;
  if (static_cast<long long>(tiles_m) * tiles_n * d.batch_count > 0x7FFFFFFFll) return GEMM_ERR_UNSUPPORTED;
  const long long num_tiles = tiles_total;
  // raster group height G: the resident tiles cover G tile rows x (units / G) tile columns; operand traffic from L2
  // is smallest when that block is square in elements, G * tile_m ~ (units / G) * bn
  int raster = forced_raster;
  if (raster == 0) {
    const double units = static_cast<double>(pl->sm_count / cg);
    raster = static_cast<int>(std::lround(1.4 * std::sqrt(units * bn / tile_m)));  // a little taller than square: the A band stays in L2 across waves (measured +1 %)
    raster = std::max(1, raster);
  }
  raster = std::max(1, std::min(raster, tiles_m));

  DenseParams& p = pl->dense;
  memset(&p, 0, sizeof p);
  p.M = static_cast<int>(d.M);
  p.N = static_cast<int>(d.N);
  p.n_full = static_cast<int>(d.N - d.N % (16 / elem_bytes(d.c_dtype)));
  p.K = static_cast<int>(d.K);
  p.batch = d.batch_count;
  p.tiles_m = tiles_m;
  p.tiles_n = tiles_n;
  p.num_tiles = static_cast<int>(num_tiles);
  p.raster_group = raster;
  p.bn = bn;
  p.stages = stages;
  p.num_kb = ceil_div(d.K, kblk * atoms);
  p.atoms = atoms;
  p.kblk = kblk;
  p.ab_fp8 = is_fp8(d.ab_dtype) ? 1 : 0;
  p.a_atom_bytes = a_atom;
  p.b_atom_bytes = b_atom;
  p.n_mma = wide_n ? 2 : 1;
  p.mma_n = bn / p.n_mma;
  p.acc_bufs = wide_n ? 1 : 2;
  p.b_box_rows = b_rows / p.n_mma;
  uint32_t cols = 32;
  while (cols < static_cast<uint32_t>(p.acc_bufs * bn)) cols <<= 1;
  p.tmem_cols = cols;
  p.idesc = make_idesc(ab_format(d.ab_dtype), !a_kmajor, !b_kmajor, tile_m, p.mma_n);
  p.a_stage_bytes = a_stage;
  p.b_stage_bytes = b_stage;
  p.a_kmajor = a_kmajor;
  p.b_kmajor = b_kmajor;
  p.b_rows = b_rows;
  // K-major tile: rows of 128 bytes, 8-row swizzle atoms 1024 bytes apart (stride offset); the leading offset is unused.
  // MN-major tile: 64-element (128-byte) runs along M/N, k rows 128 bytes apart, 8-k-row atoms 1024 bytes apart
  // (stride offset) and the next 64-element run group one whole 64 x 64 box = 8192 bytes further (leading offset).
  p.a_desc_hi = a_kmajor ? make_smem_desc_hi(16, 1024) : make_smem_desc_hi(8192, 1024);
  p.b_desc_hi = b_kmajor ? make_smem_desc_hi(16, 1024) : make_smem_desc_hi(8192, 1024);
  p.a_kstep = a_kmajor ? kUmmaK * 2 : kUmmaK * 128;
  p.b_kstep = b_kmajor ? kUmmaK * 2 : kUmmaK * 128;
  p.out_dtype = d.c_dtype;
  p.epilogue = d.epilogue;
  p.bias_per_row = (d.flags & GEMM_FLAG_BIAS_PER_ROW) ? 1 : 0;
  // an output much larger than half the L2 is written with evict-first priority so that it does not push the operands
  // out (measured: +0.5 to +2.5 % on the 470 MB output of the projection shape, neutral on 134 MB)
  p.l2_hint_d = static_cast<double>(d.M) * d.N * d.batch_count * elem_bytes(d.c_dtype) > 64.0e6 ? 1 : 0;
  p.a_tri = (d.flags & GEMM_FLAG_A_LOWER) ? 1 : ((d.flags & GEMM_FLAG_A_UPPER) ? 2 : 0);
  p.b_tri = (d.structure & GEMM_STRUCT_B_LOWER) ? 1 : ((d.structure & GEMM_STRUCT_B_UPPER) ? 2 : 0);
  p.tile_list = nullptr;  // the device copy of the schedule is made by gemm_plan
  p.list_len = 0;
  pl->d_tri = d_tri;
  int dealt_units = 0;
  if (d_tri || p.a_tri || p.b_tri) {  // structured problem: tiles left out and / or unequal K ranges -> dealt ahead of time
    // A batch is dealt as a whole (one list over all its matrices) unless that list would be very long; then the deal of
    // one matrix is repeated for every matrix, which loads the CTAs less evenly: who gets the heavy tiles gets them every time.
    const bool whole_batch = d.batch_count > 1 && static_cast<long long>(tiles_m) * tiles_n * d.batch_count <= (1ll << 22);
    const TileSchedule sch = deal_tiles(d, tile_m, bn, raster, kblk * atoms, p.num_kb, units, whole_batch ? static_cast<int>(d.batch_count) : 1);
    if (static_cast<long long>(sch.slots.size()) * (whole_batch ? 1 : d.batch_count) > 0x7FFFFFFFll) return GEMM_ERR_UNSUPPORTED;
    free(pl->h_tile_list);
    pl->h_tile_list = static_cast<int*>(malloc(sch.slots.size() * sizeof(int)));
    if (!pl->h_tile_list) return GEMM_ERR_CUDA;
    memcpy(pl->h_tile_list, sch.slots.data(), sch.slots.size() * sizeof(int));
    p.list_len = static_cast<int>(sch.slots.size());
    p.num_tiles = whole_batch ? p.list_len : p.list_len * static_cast<int>(d.batch_count);  // slots, the empty ones included
    dealt_units = sch.units;
  }
  if (!set_scheduler_divisors(p)) return GEMM_ERR_UNSUPPORTED;
  p.ldc = d.ldc;
  p.stride_c = d.batch_count > 1 ? d.stride_c : 0;
  p.debug_flags = 0u;  // set per run
  // The scheduler keeps a band of `raster` tile rows of A live across several waves while B panels stream past;
  // on request, L2 is asked to hold on to A and to let B go first (measured neutral on 8192^3, so off by default).
  const bool hints = (d.flags & GEMM_FLAG_L2_HINTS) != 0;
  p.k_serpentine = ((d.flags & GEMM_FLAG_NO_K_SERPENTINE) || p.num_kb < 4) ? 0 : 1;  // pointless for a couple of stages
  p.l2_hint_a = hints ? 2 : 0;
  p.l2_hint_b = hints ? 1 : 0;

  pl->cg = cg;
  pl->epi_wg = epi_wg;
  pl->bn = bn;
  pl->stages = stages;
  pl->raster_group = raster;
  pl->smem_bytes = smem;
  pl->grid = (dealt_units ? dealt_units : static_cast<int>(std::min<long long>(num_tiles, units))) * cg;
  pl->variant = cg == 2 ? GEMM_VARIANT_DENSE_2CTA : GEMM_VARIANT_DENSE_1CTA;

  gemm_info_t& info = pl->info;
  info.variant = pl->variant;
  info.tile_m = tile_m;
  info.tile_n = bn;
  info.tile_k = kblk * atoms;
  info.stages = stages;
  info.cluster_size = cg;
  info.grid = pl->grid;
  info.raster_group = raster;
  const int units_i = pl->sm_count / cg;
  const int split = tail_split(num_tiles, units_i, p.num_kb, d, bn, cg, atoms);
  const long long rem = num_tiles % units_i;
  p.split = split;
  p.split_first_tile = static_cast<int>(split > 1 ? num_tiles - rem : num_tiles);
  p.num_items = static_cast<int>(split > 1 ? num_tiles - rem + rem * split : num_tiles);
  pl->split = split;
  pl->split_flag_bytes = split > 1 ? (static_cast<size_t>(rem) * cg * (split - 1) * 8 + 255) / 256 * 256 : 0;
  if (split > 1) pl->grid = static_cast<int>(std::min<long long>(p.num_items, units_i)) * cg;
  info.grid = pl->grid;
  info.split = split;
  info.smem_bytes = smem;
  info.num_tiles = num_tiles;
  info.workspace_bytes = split > 1 ? pl->split_flag_bytes + static_cast<size_t>(rem) * cg * (split - 1) * kCtaM * bn * 4 : 0;
  return GEMM_OK;
}

// Wide pair variant: 512 x 256 cluster tiles, one 64-wide K slice per stage, 3-deep ring, 8 epilogue warps.
gemm_status_t plan_wide(gemm_plan_s* pl, int forced_raster, int forced_stages) {
  const gemm_desc_t& d = pl->d;
  // its epilogue covers the bias per column, ReLU and erf GELU only; its MMA schedule has no K-range skipping
  if (d.epilogue > GEMM_EPI_BIAS_GELU_ERF || (d.flags & (GEMM_FLAG_BIAS_PER_ROW | GEMM_FLAG_A_LOWER | GEMM_FLAG_A_UPPER))) return GEMM_ERR_UNSUPPORTED;
  if (d_tri_of(d) || d.structure) return GEMM_ERR_UNSUPPORTED;  // its scheduler has no tile list, its MMA schedule no K ranges
  if ((d.N * elem_bytes(d.c_dtype)) % 16) return GEMM_ERR_UNSUPPORTED;  // its epilogue has no element-wise path for a partly filled last 16-byte unit of a row
  const int a_kmajor = d.transa == GEMM_OP_N;
  const int b_kmajor = d.transb == GEMM_OP_T;
  const int tile_m = 2 * kWideCtaM, bn = kWideTileN;
  const int tiles_m = ceil_div(d.M, tile_m), tiles_n = ceil_div(d.N, bn);
  const int a_stage = kWideCtaM * kBlockK * 2, b_stage = (bn / 2) * kBlockK * 2;
  const int fixed = 1024 + 16 * kSlabBytes + 16 * kMaxStages + 64;
  int stages = forced_stages ? forced_stages : std::min(3, (kMaxSmemOptin - fixed) / (a_stage + b_stage));
  if (stages < 2 || stages > kMaxStages) return GEMM_ERR_UNSUPPORTED;
  const int smem = fixed + stages * (a_stage + b_stage);
  if (smem > kMaxSmemOptin) return GEMM_ERR_UNSUPPORTED;
  const long long num_tiles = static_cast<long long>(tiles_m) * tiles_n * d.batch_count;
  if (num_tiles > 0x7FFFFFFFll) return GEMM_ERR_UNSUPPORTED;
  const int units = pl->sm_count / 2;
  int raster = forced_raster;
  if (raster == 0) raster = std::max(1, static_cast<int>(std::lround(1.4 * std::sqrt(static_cast<double>(units) * bn / tile_m))));
  raster = std::max(1, std::min(raster, tiles_m));

  DenseParams& p = pl->dense;
  memset(&p, 0, sizeof p);
  p.M = static_cast<int>(d.M);
  p.N = static_cast<int>(d.N);
  p.n_full = static_cast<int>(d.N - d.N % (16 / elem_bytes(d.c_dtype)));
  p.K = static_cast<int>(d.K);
  p.batch = d.batch_count;
  p.tiles_m = tiles_m;
  p.tiles_n = tiles_n;
  p.num_tiles = static_cast<int>(num_tiles);
  p.raster_group = raster;
  p.bn = bn;
  p.stages = stages;
  p.num_kb = ceil_div(d.K, kblk_of(d.ab_dtype));
  p.kblk = kblk_of(d.ab_dtype);
  p.ab_fp8 = is_fp8(d.ab_dtype) ? 1 : 0;
  p.atoms = 1;
  p.tmem_cols = 512;
  p.n_mma = 1;
  p.mma_n = bn;
  p.acc_bufs = 1;
  p.b_box_rows = bn / 2;
  p.idesc = make_idesc(ab_format(d.ab_dtype), !a_kmajor, !b_kmajor, 256, bn);
  p.a_stage_bytes = a_stage;
  p.b_stage_bytes = b_stage;
  p.a_atom_bytes = a_stage;
  p.b_atom_bytes = b_stage;
  p.a_kmajor = a_kmajor;
  p.b_kmajor = b_kmajor;
  p.b_rows = bn / 2;
  p.a_desc_hi = a_kmajor ? make_smem_desc_hi(16, 1024) : make_smem_desc_hi(8192, 1024);
  p.b_desc_hi = b_kmajor ? make_smem_desc_hi(16, 1024) : make_smem_desc_hi(8192, 1024);
  p.a_kstep = a_kmajor ? kUmmaK * 2 : kUmmaK * 128;
  p.b_kstep = b_kmajor ? kUmmaK * 2 : kUmmaK * 128;
  if (!set_scheduler_divisors(p)) return GEMM_ERR_UNSUPPORTED;
  p.out_dtype = d.c_dtype;
  p.epilogue = d.epilogue;
  p.bias_per_row = (d.flags & GEMM_FLAG_BIAS_PER_ROW) ? 1 : 0;
  // an output much larger than half the L2 is written with evict-first priority so that it does not push the operands
  // out (measured: +0.5 to +2.5 % on the 470 MB output of the projection shape, neutral on 134 MB)
  p.l2_hint_d = static_cast<double>(d.M) * d.N * d.batch_count * elem_bytes(d.c_dtype) > 64.0e6 ? 1 : 0;
  p.a_tri = (d.flags & GEMM_FLAG_A_LOWER) ? 1 : ((d.flags & GEMM_FLAG_A_UPPER) ? 2 : 0);
  p.ldc = d.ldc;
  p.stride_c = d.batch_count > 1 ? d.stride_c : 0;
  p.debug_flags = 0u;  // set per run
  p.k_serpentine = ((d.flags & GEMM_FLAG_NO_K_SERPENTINE) || p.num_kb < 4) ? 0 : 1;

  pl->cg = 2;
  pl->epi_wg = 2;
  pl->bn = bn;
  pl->stages = stages;
  pl->raster_group = raster;
  pl->smem_bytes = smem;
  pl->grid = static_cast<int>(std::min<long long>(num_tiles, units)) * 2;
  pl->variant = GEMM_VARIANT_DENSE_2CTA_WIDE;
  gemm_info_t& info = pl->info;
  info.variant = pl->variant;
  info.tile_m = tile_m;
  info.tile_n = bn;
  info.tile_k = kblk_of(d.ab_dtype);
  info.stages = stages;
  info.cluster_size = 2;
  info.grid = pl->grid;
  info.raster_group = raster;
  info.split = 1;
  info.smem_bytes = smem;
  info.num_tiles = num_tiles;
  info.workspace_bytes = 0;
  return GEMM_OK;
}

// How many clusters of c = 2 ... 8 CTAs of the stream-K kernel (one CTA per SM: it takes nearly all shared memory) the
// device holds at once, asked of the occupancy calculator once per device.  A cluster must fit inside one GPC, so for
// some sizes this is fewer than SM count / c, and a plan whose clusters do not all fit would run in two waves.
const int* skinny_cluster_room(int device) {
  static int room[kMaxDevices][9];
  static bool known[kMaxDevices];
  static std::mutex mu;
  if (device < 0 || device >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[device]) {
    const void* kern = reinterpret_cast<const void*>(skinny_gemm_kernel<false, true>);
    if (ensure_dynamic_smem(kern, kSlotSkinnyCluster, device, kMaxSmemOptin) != cudaSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    for (int c = 2; c <= 8; ++c) {
      cudaLaunchConfig_t cfg;
      memset(&cfg, 0, sizeof cfg);
      cfg.gridDim = dim3(c * 16, 1, 1);
      cfg.blockDim = dim3(kSkinnyThreads, 1, 1);
      cfg.dynamicSmemBytes = kMaxSmemOptin;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = c;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, skinny_gemm_kernel<false, true>, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        n = 0;  // unknown: no clusters of this size
      }
      room[device][c] = n;
    }
    known[device] = true;
    if (getenv("B200GEMM_LOG"))
      fprintf(stderr, "[b200gemm] stream-K clusters that fit at once, sizes 2..8: %d %d %d %d %d %d %d\n", room[device][2], room[device][3],
              room[device][4], room[device][5], room[device][6], room[device][7], room[device][8]);
  }
  return room[device];
}

gemm_status_t plan_skinny(gemm_plan_s* pl, int forced_stages, int forced_atoms) {
  const gemm_desc_t& d = pl->d;
  if (d.transa != GEMM_OP_N || d.transb != GEMM_OP_T) return GEMM_ERR_UNSUPPORTED;  // both operands K-contiguous
  if ((d.M > kSkinnyMaxM && d.N > kSkinnyMaxM) || d.batch_count != 1) return GEMM_ERR_UNSUPPORTED;
  if (d.flags & (GEMM_FLAG_A_LOWER | GEMM_FLAG_A_UPPER)) return GEMM_ERR_UNSUPPORTED;  // no K-range skipping in stream-K
  if (d_tri_of(d) || d.structure) return GEMM_ERR_UNSUPPORTED;  // a short extent of 64 has a single tile row or column: nothing to leave out
  SkinnyPlan& s = pl->skinny;
  pl->skinny_tall = d.M > kSkinnyMaxM;  // the short extent is N: A is streamed, B is the resident slab
  const int small_extent = static_cast<int>(pl->skinny_tall ? d.N : d.M), big_extent = static_cast<int>(pl->skinny_tall ? d.M : d.N);
  if (forced_atoms > 3) return GEMM_ERR_UNSUPPORTED;
  if (!skinny_make_plan(&s, small_extent, big_extent, static_cast<int>(d.K), pl->sm_count, forced_stages, kMaxSmemOptin, forced_atoms,
                        kblk_of(d.ab_dtype), /*align=*/true, (pl->has_device && pl->arch_ok) ? skinny_cluster_room(pl->device) : nullptr,
                        /*clusters=*/!(d.options & GEMM_OPT_STREAMK_WORKSPACE)))
    return GEMM_ERR_UNSUPPORTED;
  pl->variant = GEMM_VARIANT_SKINNY_STREAMK;
  pl->cg = 1;
  pl->stages = s.stages;
  pl->grid = s.grid;
  pl->smem_bytes = s.smem_bytes;
  gemm_info_t& info = pl->info;
  info.variant = pl->variant;
  // 128 rows of the streamed operand per tile; the short extent padded to a multiple of 16
  info.tile_m = kSkinnyTileN;
  info.tile_n = s.m_pad;
  info.tile_k = s.kblk * s.atoms;
  info.stages = s.stages;
  info.cluster_size = s.cluster;  // > 1: the CTAs of one output tile form a cluster and hand over through shared memory
  info.grid = s.grid;
  info.raster_group = 1;
  info.split = s.max_contributors;
  info.smem_bytes = s.smem_bytes;
  info.num_tiles = s.total_units;
  info.workspace_bytes = s.counters_bytes + s.workspace_bytes;  // arrival words, then the partial tiles
  return GEMM_OK;
}

}  // namespace

namespace {

// Identity of a plan (or of one allocation-free call), 24 bits, never 0: together with the run number it forms the tag
// that marks a run's hand-shake words in a workspace, so that words left by anything else read as "nothing yet".
uint64_t next_plan_identity() {
  static std::atomic<uint64_t> counter{0};
  uint64_t id;
  do id = (counter.fetch_add(1, std::memory_order_relaxed) + 1) & 0xFFFFFFull;
  while (id == 0);
  return id;
}
// Tag of run number `run` of a plan: 48 bits, never 0.  The pair (identity, run number) is unique, but as a bit pattern
// it is a small number next to zeros, and so is much of what a recycled workspace holds: 16-bit floats of small integer
// value between zeros read, as a 64-bit word, exactly like "identity 0x5b, run 0, count x" (found by a randomised
// sweep: one tile of one problem in 240 was never finished because a stale word passed for this run's arrival
// word).  So the pair goes through a bijection of the 48-bit numbers that spreads it over all bits -- distinct pairs
// still give distinct tags -- after an exclusive-or with a per-process random number, so that words left by another
// process that used this library do not repeat this process's tags either.  What remains is the chance that arbitrary
// stale data equals one given 48-bit value.
uint64_t tag_salt() {
  static const uint64_t salt = [] {
    uint64_t s = 0x9E3779B97F4A7C15ull ^ static_cast<uint64_t>(std::chrono::steady_clock::now().time_since_epoch().count());
    s ^= static_cast<uint64_t>(std::chrono::system_clock::now().time_since_epoch().count()) << 17;
    s ^= reinterpret_cast<uintptr_t>(&s) << 7;
    try {
      std::random_device rd;
      s ^= (static_cast<uint64_t>(rd()) << 32) ^ rd();
    } catch (...) {
    }
    return s & 0xFFFFFFFFFFFFull;
  }();
  return salt;
}
uint64_t run_tag(uint64_t tag_base, unsigned long long run) {
  const uint64_t mask = 0xFFFFFFFFFFFFull;
  uint64_t x = ((tag_base | (run & 0xFFFFFFull)) ^ tag_salt()) & mask;
  // every step is a bijection of the 48-bit numbers (exclusive-or with a right shift; multiplication by an odd number)
  x ^= x >> 23;
  x = (x * 0x2127599BF4325ull) & mask;
  x ^= x >> 19;
  x = (x * 0x880355F21E6D1ull) & mask;
  x ^= x >> 25;
  return x ? x : 0x5DEECE66Dull;  // (the one pair that maps to 0 shares this tag with one other pair)
}

// gemm_plan proper.  use_cache: take the tuning fields gemm_tune remembered for this shape (when the caller set none);
// *cache_used tells whether that happened.
gemm_status_t plan_impl(const gemm_desc_t* desc, gemm_plan_t* out_plan, bool use_cache, bool* cache_used) {
  *cache_used = false;
  if (!desc || !out_plan) return GEMM_ERR_NULL;
  *out_plan = nullptr;
  gemm_status_t st = validate(desc);
  if (st != GEMM_OK) return st;
  gemm_plan_s* pl = new (std::nothrow) gemm_plan_s();
  if (!pl) return GEMM_ERR_CUDA;
  memset(pl, 0, sizeof *pl);
  pl->d = *desc;
  if (pl->d.batch_count == 1) pl->d.stride_a = pl->d.stride_b = pl->d.stride_c = 0;
  pl->timeout_ms = 2000;
  pl->sm_count = kDefaultSmCount;
  int dev = -1;
  pl->device = -1;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) == cudaSuccess) {
      pl->device = dev;
      pl->has_device = true;
      pl->arch_ok = prop.major == 10;
      if (pl->arch_ok) pl->sm_count = prop.multiProcessorCount;
    }
  }
  (void)cudaGetLastError();
  if (use_cache && pl->has_device && (pl->d.flags & kTuningFlagMask) == 0) {  // a measured choice for this shape, if gemm_tune made one
    uint32_t tuned = 0;
    if (tune_cache_lookup(pl->d, pl->device, &tuned) && tuned != 0) {
      pl->d.flags |= tuned;
      *cache_used = true;
    }
  }

  // roofline class (Section 4.3): compulsory traffic vs. work
  const gemm_desc_t& d = pl->d;
  const double eb = elem_bytes(d.ab_dtype), ec = elem_bytes(d.c_dtype);
  // elements of D that are wanted: all of it, or one triangle (diagonal included)
  double d_elems = static_cast<double>(d.M) * d.N;
  if (d_tri_of(d)) {
    const double s = static_cast<double>(std::min(d.M, d.N));  // the square part holds s (s + 1) / 2; what lies beside it is whole or empty
    const double beside = d_tri_of(d) == 1 ? static_cast<double>(std::max<int64_t>(d.M - d.N, 0)) * d.N
                                           : static_cast<double>(std::max<int64_t>(d.N - d.M, 0)) * d.M;
    d_elems = s * (s + 1.0) / 2.0 + beside;
  }
  const double flops = 2.0 * d_elems * d.K * d.batch_count;
  double bytes = d.batch_count * (static_cast<double>(d.M) * d.K + static_cast<double>(d.K) * d.N) * eb +
                 d.batch_count * d_elems * ec;
  if (has_bias(d.epilogue)) bytes += 4.0 * ((d.flags & GEMM_FLAG_BIAS_PER_ROW) ? d.M : d.N);
  gemm_info_t& info = pl->info;
  info.struct_size = sizeof(gemm_info_t);
  info.flops = flops;
  info.min_bytes = bytes;  // beta is a run-time scalar: the C read is not counted here
  info.intensity = flops / bytes;
  info.regime = info.intensity < kRidgeCudaCore ? GEMM_REGIME_MEMORY
                                                : (info.intensity < kRidgeTensor ? GEMM_REGIME_MIDDLE : GEMM_REGIME_COMPUTE);

  const int forced_variant = (d.flags & GEMM_FLAG_VARIANT_MASK) >> GEMM_FLAG_VARIANT_SHIFT;
  // (field values up to 16 count sixteenths of 256 columns; 17 ... 20 are the wide tiles 320, 384, 448 and 512)
  const int tile_field = static_cast<int>((d.flags & GEMM_FLAG_TILE_N_MASK) >> GEMM_FLAG_TILE_N_SHIFT);
  if (tile_field > 20) {
    delete pl;
    return GEMM_ERR_INVALID_ARG;
  }
  const int forced_bn = tile_field <= 16 ? tile_field * 16 : 256 + (tile_field - 16) * 64;
  const int forced_raster = (d.flags & GEMM_FLAG_RASTER_MASK) >> GEMM_FLAG_RASTER_SHIFT;
  const int forced_stages = (d.flags & GEMM_FLAG_STAGES_MASK) >> GEMM_FLAG_STAGES_SHIFT;
  const int forced_atoms = (d.flags & GEMM_FLAG_KSLICES_MASK) >> GEMM_FLAG_KSLICES_SHIFT;
  int variant = forced_variant;
  int auto_bn = 0;  // tile width chosen together with the variant
  if (variant == 0) {
    // memory-bound problems with a handful of rows stream the weight matrix once: stream-K path;
    // everything else is a dense tiled GEMM, paired CTAs when there are at least two tile rows
    const bool skinny_ok = (d.M <= kSkinnyMaxM || d.N <= kSkinnyMaxM) && d.batch_count == 1 && d.transa == GEMM_OP_N &&
                           d.transb == GEMM_OP_T && !(d.flags & (GEMM_FLAG_A_LOWER | GEMM_FLAG_A_UPPER)) && !d_tri_of(d) && !d.structure;
    if (skinny_ok && info.intensity < 7.0 * kRidgeCudaCore) {
      variant = GEMM_VARIANT_SKINNY_STREAMK;  // measured: level with the dense kernels at a short extent of 64 on the largest shapes, far ahead elsewhere
    } else {
      // score every dense family and tile width with the roofline estimate and take the cheapest
      const bool b_kmajor = d.transb == GEMM_OP_T;
      DenseCandidate best{GEMM_VARIANT_DENSE_1CTA, 64, 1e300};
      for (int v : {GEMM_VARIANT_DENSE_1CTA, GEMM_VARIANT_DENSE_2CTA, GEMM_VARIANT_DENSE_2CTA_WIDE}) {
        for (int bn : {512, 448, 384, 320, 256, 192, 128, 64}) {
          if (v == GEMM_VARIANT_DENSE_2CTA_WIDE && bn != kWideTileN) continue;
          if (bn > 256) {
            // wide single-buffered tiles: K-contiguous B, and only where they give every CTA (pair) at most one tile --
            // their purpose is to turn "a little more than one wave" into one wave (2304^3: 108 tiles of 256 x 192 on 74
            // pairs become 72 of 256 x 320) and to cut the operand traffic per FLOP on the way
            const int rows_tile = v == GEMM_VARIANT_DENSE_1CTA ? kCtaM : 2 * kCtaM;
            const long long tiles = tri_tile_count(d_tri_of(d), rows_tile, bn, d.M, d.N) * d.batch_count;
            if (!b_kmajor || tiles > pl->sm_count / (v == GEMM_VARIANT_DENSE_1CTA ? 1 : 2) || (d.flags & GEMM_FLAG_TAIL_SPLIT)) continue;
          }
          if (v == GEMM_VARIANT_DENSE_2CTA_WIDE &&
              (d.epilogue > GEMM_EPI_BIAS_GELU_ERF || d_tri_of(d) || d.structure || (d.N * elem_bytes(d.c_dtype)) % 16 ||
               (d.flags & (GEMM_FLAG_BIAS_PER_ROW | GEMM_FLAG_A_LOWER | GEMM_FLAG_A_UPPER))))
            continue;
          if (v == GEMM_VARIANT_DENSE_2CTA && !b_kmajor && bn % 128) continue;  // 64-column boxes per CTA
          if (v != GEMM_VARIANT_DENSE_1CTA && d.M <= kCtaM) continue;           // a pair needs two tile rows
          if (forced_bn && bn != forced_bn) continue;
          const double c = estimate_dense_cycles(d, pl->sm_count, v, bn);
          if (c < best.cycles * 0.995) best = DenseCandidate{v, bn, c};          // ties go to the earlier, simpler one
        }
      }
      variant = best.variant;
      auto_bn = best.bn;
    }
  }
  if (variant == GEMM_VARIANT_DENSE_1CTA) st = plan_dense(pl, 1, forced_bn ? forced_bn : auto_bn, forced_raster, forced_stages, forced_atoms);
  else if (variant == GEMM_VARIANT_DENSE_2CTA) st = plan_dense(pl, 2, forced_bn ? forced_bn : auto_bn, forced_raster, forced_stages, forced_atoms);
  else if (variant == GEMM_VARIANT_SKINNY_STREAMK) st = plan_skinny(pl, forced_stages, forced_atoms);
  else if (variant == GEMM_VARIANT_DENSE_2CTA_WIDE) st = plan_wide(pl, forced_raster, forced_stages);
  else st = GEMM_ERR_INVALID_ARG;
  if (st != GEMM_OK) {
    delete pl;
    return st;
  }
  pl->tag_base = next_plan_identity() << 24;
  if (pl->has_device && pl->arch_ok) {
    pl->maps = new (std::nothrow) MapCache();
    if (!pl->maps || cudaMalloc(&pl->d_status, 16) != cudaSuccess || cudaMemset(pl->d_status, 0, 16) != cudaSuccess) {
      note_cuda_error("cudaMalloc(status word)", cudaGetErrorName(cudaGetLastError()));
      if (pl->d_status) cudaFree(pl->d_status);
      delete pl;
      return GEMM_ERR_CUDA;
    }
  }
  if (pl->has_device && pl->arch_ok && pl->h_tile_list) {
    const size_t bytes = static_cast<size_t>(pl->dense.list_len) * sizeof(int);
    if (cudaMalloc(&pl->d_tile_list, bytes) != cudaSuccess ||
        cudaMemcpy(pl->d_tile_list, pl->h_tile_list, bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
      note_cuda_error("cudaMalloc(tile schedule)", cudaGetErrorName(cudaGetLastError()));
      if (pl->d_tile_list) cudaFree(pl->d_tile_list);
      cudaFree(pl->d_status);
      delete pl;
      return GEMM_ERR_CUDA;
    }
    pl->dense.tile_list = pl->d_tile_list;  // (the host copy stays with the plan for gemm_plan_schedule)
  }
  if (getenv("B200GEMM_LOG")) {
    fprintf(stderr,
            "[b200gemm] M=%lld N=%lld K=%lld batch=%d AI=%.1f regime=%d variant=%d tile=%dx%dx%d stages=%d cluster=%d "
            "grid=%d raster=%d split=%d smem=%d ws=%zu\n",
            (long long)d.M, (long long)d.N, (long long)d.K, d.batch_count, info.intensity, info.regime, info.variant,
            info.tile_m, info.tile_n, info.tile_k, info.stages, info.cluster_size, info.grid, info.raster_group, info.split,
            info.smem_bytes, info.workspace_bytes);
  }
  *out_plan = pl;
  return GEMM_OK;
}

}  // namespace

namespace {
// Take the status word: what a timed-out run left there goes to the plan's page-locked host word (read by
// gemm_plan_status_result once the stream has got this far) and the device word is cleared in the same atomic step,
// so a run on another stream that gives up at this very moment is not lost.
__global__ void status_take_kernel(uint32_t* status, uint32_t* host_word) {
  const uint32_t v = atomicExch(status, 0u);
  if (v != 0u) *reinterpret_cast<volatile uint32_t*>(host_word) = v;
}
}  // namespace

extern "C" {

gemm_status_t gemm_plan(const gemm_desc_t* desc, gemm_plan_t* out_plan) {
  bool cache_used = false;
  gemm_status_t st = plan_impl(desc, out_plan, true, &cache_used);
  // remembered tuning fields that do not plan (a file from another version of the library) must not break the problem
  if (st != GEMM_OK && cache_used) st = plan_impl(desc, out_plan, false, &cache_used);
  return st;
}

size_t gemm_workspace_bytes(gemm_plan_t plan) { return plan ? plan->info.workspace_bytes : 0; }

gemm_status_t gemm_plan_info(gemm_plan_t plan, gemm_info_t* out) {
  if (!plan || !out) return GEMM_ERR_NULL;
  if (out->struct_size != sizeof(gemm_info_t)) return GEMM_ERR_INVALID_ARG;
  *out = plan->info;
  return GEMM_OK;
}

gemm_status_t gemm_plan_set_timeout_ms(gemm_plan_t plan, uint32_t ms) {
  if (!plan) return GEMM_ERR_NULL;
  plan->timeout_ms = std::max(1u, ms);
  return GEMM_OK;
}

gemm_status_t gemm_plan_status_async(gemm_plan_t plan, gemm_stream_t stream) {
  if (!plan) return GEMM_ERR_NULL;
  if (!plan->d_status) return GEMM_ERR_ARCH;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess || cur != plan->device) return GEMM_ERR_INVALID_ARG;
  cudaError_t e = cudaSuccess;
  {
    static std::mutex mu;  // first use only: the page-locked word the device writes the status into
    std::lock_guard<std::mutex> lock(mu);
    if (!plan->h_status) {
      void* h = nullptr;
      e = cudaHostAlloc(&h, 16, cudaHostAllocMapped | cudaHostAllocPortable);
      if (e == cudaSuccess) {
        memset(h, 0, 16);
        plan->h_status = static_cast<uint32_t*>(h);
      }
    }
  }
  uint32_t* dev_view = nullptr;
  if (e == cudaSuccess) e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&dev_view), plan->h_status, 0);
  if (e == cudaSuccess) {
    status_take_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(plan->d_status, dev_view);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    note_cuda_error("gemm_plan_status_async", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  return GEMM_OK;
}

gemm_status_t gemm_plan_status_result(gemm_plan_t plan) {
  if (!plan) return GEMM_ERR_NULL;
  if (!plan->h_status) return GEMM_OK;  // nothing was ever fetched
  const uint32_t word = __atomic_exchange_n(plan->h_status, 0u, __ATOMIC_ACQUIRE);
  if (word & kStatusTimeout) {
    snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "device wait expired: role %u detail 0x%02x", (word >> 8) & 0xFF,
             word & 0xFF);
    return GEMM_ERR_TIMEOUT;
  }
  return GEMM_OK;
}

gemm_status_t gemm_plan_status_stream(gemm_plan_t plan, gemm_stream_t stream) {
  gemm_status_t st = gemm_plan_status_async(plan, stream);
  if (st != GEMM_OK) return st;
  const cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    note_cuda_error("gemm_plan_status_stream", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  return gemm_plan_status_result(plan);
}

gemm_status_t gemm_plan_status(gemm_plan_t plan) {
  if (!plan) return GEMM_ERR_NULL;
  if (!plan->d_status) return GEMM_ERR_ARCH;
  const cudaError_t e = cudaDeviceSynchronize();  // the plan does not know which streams ran it: wait for all of them
  if (e != cudaSuccess) {
    note_cuda_error("gemm_plan_status", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  return gemm_plan_status_stream(plan, nullptr);
}

gemm_status_t gemm_plan_schedule(gemm_plan_t plan, gemm_work_item_t* items, size_t capacity, size_t* count) {
  if (!plan || !count || (capacity > 0 && !items)) return GEMM_ERR_NULL;
  size_t n = 0;
  auto emit = [&](int cta, int batch, int row, int col, int k0, int k1, int slice) {
    if (n < capacity) items[n] = gemm_work_item_t{cta, batch, row, col, k0, k1, slice, 0};
    ++n;
  };
  if (plan->variant == GEMM_VARIANT_SKINNY_STREAMK) {
    const SkinnyPlan& s = plan->skinny;
    for (int c = 0; c < s.grid; ++c) {
      const int u_end = sk_cta_begin(s, c + 1);
      for (int u = sk_cta_begin(s, c); u < u_end;) {  // one item per tile this CTA's range touches
        const int tile = u / s.kbs, tile_u0 = tile * s.kbs;
        const int seg_end = std::min(u_end, tile_u0 + s.kbs);
        const bool whole = u == tile_u0 && seg_end == tile_u0 + s.kbs;
        // position among the tile's contributors (cluster mode: the rank in the cluster)
        const int slice = whole ? -1 : (s.cluster > 1 ? c % s.cluster : c - sk_unit_owner(s, tile_u0));
        emit(c, 0, plan->skinny_tall ? tile : 0, plan->skinny_tall ? 0 : tile, u - tile_u0, seg_end - tile_u0, slice);
        u = seg_end;
      }
    }
  } else {
    DenseParams p = plan->dense;
    p.tile_list = plan->h_tile_list;  // (nullptr for an unstructured problem)
    const int cg = plan->cg, clusters = plan->grid / cg;
    const bool wide = plan->variant == GEMM_VARIANT_DENSE_2CTA_WIDE;
    const int tile_rows = (wide ? kWideCtaM : kCtaM) * cg;
    for (int c = 0; c < clusters; ++c) {
      if (wide) {
        for (int tile = c; tile < p.num_tiles; tile += clusters) {
          const TileCoord tc = decode_tile_div(tile, p.tiles_m, p.tiles_n, p.raster_group);
          emit(c, tc.batch, tc.tm, tc.tn, 0, p.num_kb, -1);
        }
        continue;
      }
      const bool split = plan->split > 1;
      const int n_items = split ? p.num_items : p.num_tiles;
      for (int item = c; item < n_items; item += clusters) {
        const int tile = split ? item_tile<true>(p, item) : item_tile<false>(p, item);
        if (tile < 0) continue;
        const TileCoord tc = decode_tile(p, tile);
        const WorkItem wi = split ? work_item<true>(p, item, tile, tc.tm * tile_rows, tile_rows, tc.tn * p.bn)
                                  : work_item<false>(p, item, tile, tc.tm * tile_rows, tile_rows, tc.tn * p.bn);
        emit(c, tc.batch, tc.tm, tc.tn, wi.kr.lo, wi.kr.hi, wi.slice);
      }
    }
  }
  *count = n;
  return GEMM_OK;
}

gemm_status_t gemm_destroy(gemm_plan_t plan) {
  if (!plan) return GEMM_OK;
  gemm_status_t st = GEMM_OK;
  if (plan->d_tile_list && cudaFree(plan->d_tile_list) != cudaSuccess) {
    note_cuda_error("cudaFree", cudaGetErrorName(cudaGetLastError()));
    st = GEMM_ERR_CUDA;
  }
  if (plan->d_status && cudaFree(plan->d_status) != cudaSuccess) {
    note_cuda_error("cudaFree", cudaGetErrorName(cudaGetLastError()));
    st = GEMM_ERR_CUDA;
  }
  if (plan->h_status && cudaFreeHost(plan->h_status) != cudaSuccess) {
    note_cuda_error("cudaFreeHost", cudaGetErrorName(cudaGetLastError()));
    st = GEMM_ERR_CUDA;
  }
  delete plan;
  return st;
}

const char* gemm_status_string(gemm_status_t s) {
  switch (s) {
    case GEMM_OK: return "GEMM_OK";
    case GEMM_ERR_NULL: return "GEMM_ERR_NULL";
    case GEMM_ERR_INVALID_ARG: return "GEMM_ERR_INVALID_ARG";
    case GEMM_ERR_UNSUPPORTED: return "GEMM_ERR_UNSUPPORTED";
    case GEMM_ERR_ALIGNMENT: return "GEMM_ERR_ALIGNMENT";
    case GEMM_ERR_WORKSPACE: return "GEMM_ERR_WORKSPACE";
    case GEMM_ERR_ARCH: return "GEMM_ERR_ARCH";
    case GEMM_ERR_CUDA: return "GEMM_ERR_CUDA";
    case GEMM_ERR_TIMEOUT: return "GEMM_ERR_TIMEOUT";
  }
  return "GEMM_ERR_UNKNOWN";
}

const char* gemm_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"

namespace {

template <int CG, int EPI_WG, bool kSplit>
gemm_status_t launch_dense(const gemm_plan_s* pl, const CUtensorMap& tA, const CUtensorMap& tB, const CUtensorMap& tD,
                           const DenseParams& p, cudaStream_t stream) {
  auto kern = dense_gemm_kernel<CG, EPI_WG, kSplit>;
  constexpr KernelSlot slot = static_cast<KernelSlot>((CG == 1 ? (EPI_WG == 1 ? kSlotDense11 : kSlotDense12) : (EPI_WG == 1 ? kSlotDense21 : kSlotDense22)) +
                                                      (kSplit ? kSlotDenseSplit11 - kSlotDense11 : 0));
  if (ensure_dynamic_smem(reinterpret_cast<const void*>(kern), slot, pl->device, pl->smem_bytes) != cudaSuccess) {
    note_cuda_error("cudaFuncSetAttribute", cudaGetErrorName(cudaGetLastError()));
    return GEMM_ERR_CUDA;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(pl->grid, 1, 1);
  cfg.blockDim = dim3(64 + 128 * EPI_WG, 1, 1);
  cfg.dynamicSmemBytes = pl->smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up may overlap the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (pl->d.flags & GEMM_FLAG_NO_EARLY_LAUNCH) ? 1 : 2;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tA, tB, tD, p);
  if (e != cudaSuccess) {
    note_cuda_error("cudaLaunchKernelEx(dense)", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  return GEMM_OK;
}

gemm_status_t launch_wide(const gemm_plan_s* pl, const CUtensorMap& tA, const CUtensorMap& tB, const CUtensorMap& tD,
                          const DenseParams& p, cudaStream_t stream) {
  const bool fp8 = is_fp8(pl->d.ab_dtype);
  const void* kern = fp8 ? reinterpret_cast<const void*>(wide_gemm_kernel<true>) : reinterpret_cast<const void*>(wide_gemm_kernel<false>);
  if (ensure_dynamic_smem(kern, fp8 ? kSlotWideFp8 : kSlotWide, pl->device, pl->smem_bytes) != cudaSuccess) {
    note_cuda_error("cudaFuncSetAttribute", cudaGetErrorName(cudaGetLastError()));
    return GEMM_ERR_CUDA;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(pl->grid, 1, 1);
  cfg.blockDim = dim3(kWideThreads, 1, 1);
  cfg.dynamicSmemBytes = pl->smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up may overlap the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (pl->d.flags & GEMM_FLAG_NO_EARLY_LAUNCH) ? 1 : 2;
  cudaError_t e = fp8 ? cudaLaunchKernelEx(&cfg, wide_gemm_kernel<true>, tA, tB, tD, p) : cudaLaunchKernelEx(&cfg, wide_gemm_kernel<false>, tA, tB, tD, p);
  if (e != cudaSuccess) {
    note_cuda_error("cudaLaunchKernelEx(wide)", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  return GEMM_OK;
}

gemm_status_t run_dense(gemm_plan_s* pl, const void* A, const void* B, void* C, const float* bias, float alpha, float beta,
                        void* workspace, cudaStream_t stream, bool stall, unsigned long long run_index) {
  const gemm_desc_t& d = pl->d;
  DenseParams p = pl->dense;
  CUtensorMap tA, tB, tD;
  const uint64_t batch = d.batch_count;
  // Each map is encoded the first time its operand address is seen and fetched from the plan's table afterwards
  // (an encoding costs the host about a microsecond, three of them more than the launch itself).
  // A: K-major -> rows are M, inner K, box 64 x 128; M-major (stored K x M) -> rows are K, inner M, box 64 x 64
  const uint32_t a_box_rows = pl->variant == GEMM_VARIANT_DENSE_2CTA_WIDE ? kWideCtaM : kCtaM;
  bool ok = true;
  if (!pl->maps->find(0, A, &tA)) {
    ok = p.a_kmajor ? encode_map(&tA, d.ab_dtype, A, d.K, d.M, batch, d.lda, d.stride_a, p.kblk, a_box_rows)
                    : encode_map(&tA, d.ab_dtype, A, d.M, d.K, batch, d.lda, d.stride_a, 64, kBlockK);
    if (ok) pl->maps->insert(0, A, tA);
  }
  if (ok && !pl->maps->find(1, B, &tB)) {
    ok = p.b_kmajor ? encode_map(&tB, d.ab_dtype, B, d.K, d.N, batch, d.ldb, d.stride_b, p.kblk, p.b_box_rows)
                    : encode_map(&tB, d.ab_dtype, B, d.N, d.K, batch, d.ldb, d.stride_b, 64, kBlockK);
    if (ok) pl->maps->insert(1, B, tB);
  }
  if (ok && !pl->maps->find(2, C, &tD)) {
    const uint32_t slab_cols = d.c_dtype == GEMM_F32 ? 32 : 64;
    // (whole 16-byte units of a row only: the store engine writes whole units, see DenseParams::n_full)
    const uint64_t d_cols = std::max<uint64_t>(p.n_full, 16 / elem_bytes(d.c_dtype));
    ok = encode_map(&tD, d.c_dtype, C, d_cols, d.M, batch, d.ldc, d.stride_c, slab_cols, 32);
    if (ok) pl->maps->insert(2, C, tD);
  }
  if (!ok) return GEMM_ERR_CUDA;
  p.alpha = alpha;
  p.beta = beta;
  p.bias = bias;
  p.c_in = C;
  p.debug_flags = stall ? 1u : 0u;
  p.status = pl->d_status;
  p.timeout_ns = static_cast<unsigned long long>(pl->timeout_ms) * 1000000ull;
  if (pl->variant == GEMM_VARIANT_DENSE_2CTA_WIDE) return launch_wide(pl, tA, tB, tD, p, stream);
  gemm_status_t st;
  if (pl->split > 1) {
    // head of the workspace: the flag words (tagged per run, no initialisation needed); behind them the partial tiles
    p.split_flags = static_cast<unsigned long long*>(workspace);
    p.partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + pl->split_flag_bytes);
    p.split_tag = run_tag(pl->tag_base, run_index);
    if (pl->cg == 1) st = pl->epi_wg == 2 ? launch_dense<1, 2, true>(pl, tA, tB, tD, p, stream) : launch_dense<1, 1, true>(pl, tA, tB, tD, p, stream);
    else st = pl->epi_wg == 2 ? launch_dense<2, 2, true>(pl, tA, tB, tD, p, stream) : launch_dense<2, 1, true>(pl, tA, tB, tD, p, stream);
  } else if (pl->cg == 1) {
    st = pl->epi_wg == 2 ? launch_dense<1, 2, false>(pl, tA, tB, tD, p, stream) : launch_dense<1, 1, false>(pl, tA, tB, tD, p, stream);
  } else {
    st = pl->epi_wg == 2 ? launch_dense<2, 2, false>(pl, tA, tB, tD, p, stream) : launch_dense<2, 1, false>(pl, tA, tB, tD, p, stream);
  }
  if (st == GEMM_OK && (d.structure & GEMM_STRUCT_D_MIRROR)) {  // symmetric result: copy the computed triangle into the other one
    MirrorParams mp;
    mp.d = C;
    mp.ldc = d.ldc;
    mp.stride = d.batch_count > 1 ? d.stride_c : 0;
    mp.n = static_cast<int>(d.M);
    mp.blocks = ceil_div(d.M, 32);
    mp.upper_source = (d.flags & GEMM_FLAG_D_UPPER) ? 1 : 0;
    const cudaError_t e = mirror_launch(mp, elem_bytes(d.c_dtype), d.batch_count, stream);
    if (e != cudaSuccess) {
      note_cuda_error("mirror kernel launch", cudaGetErrorName(e));
      return GEMM_ERR_CUDA;
    }
  }
  return st;
}

gemm_status_t run_skinny(gemm_plan_s* pl, const void* A, const void* B, void* C, const float* bias, float alpha, float beta,
                         void* workspace, cudaStream_t stream, bool stall, unsigned long long run_index) {
  const gemm_desc_t& d = pl->d;
  const SkinnyPlan& s = pl->skinny;
  CUtensorMap tW, tX, tD;
  // weights W = B stored N x K (K contiguous): box 64 x 128; activations X = A stored M x K: box 64 x m_pad;
  // a tall problem streams A in W's place and keeps B as the slab.  Maps are remembered by operand address.
  // D (unless tall): plain row-major boxes of 16 rows x 32 columns over the whole 16-byte units of each row.
  const void* w_ptr = pl->skinny_tall ? A : B;
  const void* x_ptr = pl->skinny_tall ? B : A;
  const int64_t w_rows = pl->skinny_tall ? d.M : d.N, w_ld = pl->skinny_tall ? d.lda : d.ldb;
  const int64_t x_rows = pl->skinny_tall ? d.N : d.M, x_ld = pl->skinny_tall ? d.ldb : d.lda;
  bool ok = true;
  if (!pl->maps->find(0, w_ptr, &tW)) {
    ok = encode_map(&tW, d.ab_dtype, w_ptr, d.K, w_rows, 1, w_ld, 0, s.kblk, kSkinnyTileN);
    if (ok) pl->maps->insert(0, w_ptr, tW);
  }
  if (ok && !pl->maps->find(1, x_ptr, &tX)) {
    ok = encode_map(&tX, d.ab_dtype, x_ptr, d.K, x_rows, 1, x_ld, 0, s.kblk, s.m_pad);
    if (ok) pl->maps->insert(1, x_ptr, tX);
  }
  const int64_t per16 = 16 / elem_bytes(d.c_dtype);
  const int n_full = pl->skinny_tall ? 0 : static_cast<int>(d.N / per16 * per16);
  if (n_full == 0) {
    tD = tW;  // never used
  } else if (ok && !pl->maps->find(2, C, &tD)) {
    ok = encode_map(&tD, d.c_dtype, C, n_full, d.M, 1, d.ldc, 0, 32, 16, /*swizzle=*/false);
    if (ok) pl->maps->insert(2, C, tD);
  }
  if (!ok) return GEMM_ERR_CUDA;
  SkinnyParams p;
  memset(&p, 0, sizeof p);
  p.plan = s;
  p.n_full = n_full;
  p.M = static_cast<int>(d.M);
  p.N = static_cast<int>(d.N);
  p.K = static_cast<int>(d.K);
  p.idesc = make_idesc(ab_format(d.ab_dtype), 0, 0, kSkinnyTileN, s.m_pad);
  p.ab_fp8 = is_fp8(d.ab_dtype) ? 1 : 0;
  p.out_dtype = d.c_dtype;
  p.epilogue = d.epilogue;
  p.bias_per_row = (d.flags & GEMM_FLAG_BIAS_PER_ROW) ? 1 : 0;
  p.alpha = alpha;
  p.beta = beta;
  p.bias = bias;
  p.c = C;
  p.ldc = d.ldc;
  // head of the workspace: the arrival words (tagged per run, no initialisation needed); behind them the partial tiles
  p.counters = static_cast<unsigned long long*>(workspace);
  p.partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + s.counters_bytes);
  p.tag = run_tag(pl->tag_base, run_index);
  p.debug_flags = stall ? 1u : 0u;
  p.status = pl->d_status;
  p.timeout_ns = static_cast<unsigned long long>(pl->timeout_ms) * 1000000ull;
  return static_cast<gemm_status_t>(
      skinny_launch(p, tW, tX, tD, pl->device, stream, g_last_cuda_error, sizeof g_last_cuda_error, pl->skinny_tall,
                    /*early_launch=*/!(d.flags & GEMM_FLAG_NO_EARLY_LAUNCH)));
}

}  // namespace

extern "C" gemm_status_t gemm_run(gemm_plan_t plan, const void* A, const void* B, void* C, const float* bias, float alpha,
                                  float beta, void* workspace, size_t workspace_bytes, gemm_stream_t stream) {
  if (!plan || !A || !B || !C) return GEMM_ERR_NULL;
  if (has_bias(plan->d.epilogue) && !bias) return GEMM_ERR_NULL;
  auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (misaligned(A) || misaligned(B) || misaligned(C) || (bias && misaligned(bias))) return GEMM_ERR_ALIGNMENT;
  const size_t need = plan->info.workspace_bytes;
  if (need > 0) {
    if (!workspace || workspace_bytes < need) return GEMM_ERR_WORKSPACE;
    if (misaligned(workspace)) return GEMM_ERR_ALIGNMENT;
  }
  if (!plan->has_device || !plan->arch_ok || !plan->d_status) return GEMM_ERR_ARCH;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess || cur != plan->device) return GEMM_ERR_INVALID_ARG;  // plan belongs to another device
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // (atomic: a plan may be run from several host threads at once)
  const unsigned long long run_index = __atomic_fetch_add(&plan->runs, 1ull, __ATOMIC_RELAXED);
  const bool stall = (plan->d.flags & GEMM_FLAG_DEBUG_STALL) && run_index == 0;  // test hook: the plan's first run only
  if (plan->variant == GEMM_VARIANT_SKINNY_STREAMK) return run_skinny(plan, A, B, C, bias, alpha, beta, workspace, s, stall, run_index);
  return run_dense(plan, A, B, C, bias, alpha, beta, workspace, s, stall, run_index);
}

// ---------------------------------------------------------------------------------------------------------
// Allocation-free entry point (no counterpart in the paper).
//
// Some callers may not allocate device memory once they are running: a serving process that handed the whole
// GPU to its own memory pool at start-up (a later cudaMalloc fails or fragments the pool), a latency-critical
// loop that cannot afford cudaMalloc's implicit device-wide synchronisation, or code running under a rule that
// forbids allocator calls after initialisation.  gemm_plan allocates (the plan object and a status word) and the
// stream-K kernel wants a caller-provided workspace, so neither fits such a caller.  gemm_skinny_run_noalloc runs
// the same stream-K kernel with its scratch (status word, arrival counters, partial tiles) in the fixed array
// below and builds its plan on the stack.
namespace {

constexpr size_t kNoAllocScratchBytes = 4u << 20;  // held by every GPU that loads the library, until exit
constexpr size_t kNoAllocHeaderBytes = 256;        // status word of the bounded device waits
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kNoAllocMaxDevices = 64;
struct NoAllocDevice {
  unsigned char* scratch;  // device address of g_noalloc_scratch on this device
  int sm_count;
  bool arch_ok;
  bool ready;
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mu;

// Once per device, with that device current: resolve the device address of the scratch array.  In host code the
// name g_noalloc_scratch is only a handle for the symbol, never a pointer a kernel could use.
gemm_status_t noalloc_device(int dev, NoAllocDevice* out) {
  if (dev < 0 || dev >= kNoAllocMaxDevices) return GEMM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  NoAllocDevice& d = g_noalloc_dev[dev];
  if (!d.ready) {
    int major = 0, sms = 0;
    void* ptr = nullptr;
    cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess && major == 10) e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) {
      note_cuda_error("gemm_skinny_run_noalloc set-up", cudaGetErrorName(e));
      (void)cudaGetLastError();
      return GEMM_ERR_CUDA;
    }
    d.scratch = static_cast<unsigned char*>(ptr);
    d.sm_count = sms;
    d.arch_ok = (major == 10) && ptr != nullptr;
    d.ready = true;
  }
  *out = d;
  return GEMM_OK;
}

}  // namespace

extern "C" gemm_status_t gemm_skinny_run_noalloc(const gemm_desc_t* desc, const void* A, const void* B, void* C,
                                                 const float* bias, float alpha, float beta, gemm_stream_t stream,
                                                 int sync_and_check) {
  if (!desc || !A || !B || !C) return GEMM_ERR_NULL;
  gemm_status_t st = validate(desc);
  if (st != GEMM_OK) return st;
  if (has_bias(desc->epilogue) && !bias) return GEMM_ERR_NULL;
  // what the stream-K plans refuse is refused here too: every structure promise (this kernel skips nothing, so it would
  // multiply a triangle the caller declared as not stored) and the per-row bias this entry point has no field for
  if (desc->transa != GEMM_OP_N || desc->transb != GEMM_OP_T || desc->batch_count != 1 || desc->M > kSkinnyMaxM || is_fp8(desc->ab_dtype) ||
      desc->structure != 0 ||
      (desc->flags & (GEMM_FLAG_A_LOWER | GEMM_FLAG_A_UPPER | GEMM_FLAG_D_LOWER | GEMM_FLAG_D_UPPER | GEMM_FLAG_BIAS_PER_ROW)))
    return GEMM_ERR_UNSUPPORTED;
  auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (misaligned(A) || misaligned(B) || misaligned(C) || (bias && misaligned(bias))) return GEMM_ERR_ALIGNMENT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return GEMM_ERR_ARCH;
  }
  NoAllocDevice nd;
  st = noalloc_device(dev, &nd);
  if (st != GEMM_OK) return st;
  if (!nd.arch_ok) return GEMM_ERR_ARCH;

  SkinnyPlan sp;  // on the stack: nothing is allocated
  if (!skinny_make_plan(&sp, static_cast<int>(desc->M), static_cast<int>(desc->N), static_cast<int>(desc->K), nd.sm_count, 0,
                        kMaxSmemOptin))
    return GEMM_ERR_UNSUPPORTED;
  const size_t need = kNoAllocHeaderBytes + sp.counters_bytes + sp.workspace_bytes;
  if (need > kNoAllocScratchBytes) {
    snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "problem needs %zu bytes of scratch, the built-in array has %zu", need,
             kNoAllocScratchBytes);
    return GEMM_ERR_WORKSPACE;
  }
  CUtensorMap tW, tX, tD;
  if (!encode_map(&tW, desc->ab_dtype, B, desc->K, desc->N, 1, desc->ldb, 0, kBlockK, kSkinnyTileN) ||
      !encode_map(&tX, desc->ab_dtype, A, desc->K, desc->M, 1, desc->lda, 0, kBlockK, sp.m_pad))
    return GEMM_ERR_CUDA;
  const int64_t per16 = 16 / elem_bytes(desc->c_dtype);
  const int n_full = static_cast<int>(desc->N / per16 * per16);  // D leaves through the copy engine in whole 16-byte units
  if (n_full == 0) tD = tW;                                      // (never used)
  else if (!encode_map(&tD, desc->c_dtype, C, n_full, desc->M, 1, desc->ldc, 0, 32, 16, /*swizzle=*/false))
    return GEMM_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left: the status word must start at zero (the arrival words carry a
  // tag that is new with every call, so the previous call's read as empty; the partial tiles are fully written
  // before they are read).
  cudaError_t e = cudaMemsetAsync(nd.scratch, 0, kNoAllocHeaderBytes, s);
  if (e != cudaSuccess) {
    note_cuda_error("cudaMemsetAsync(status)", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  SkinnyParams p;
  memset(&p, 0, sizeof p);
  p.plan = sp;
  p.M = static_cast<int>(desc->M);
  p.N = static_cast<int>(desc->N);
  p.K = static_cast<int>(desc->K);
  p.idesc = make_idesc(desc->ab_dtype == GEMM_BF16, 0, 0, kSkinnyTileN, sp.m_pad);
  p.out_dtype = desc->c_dtype;
  p.n_full = n_full;
  p.epilogue = desc->epilogue;
  p.bias_per_row = 0;  // (refused above; the tuning fields of desc->flags are ignored)
  p.alpha = alpha;
  p.beta = beta;
  p.bias = bias;
  p.c = C;
  p.ldc = desc->ldc;
  p.status = reinterpret_cast<uint32_t*>(nd.scratch);
  p.counters = reinterpret_cast<unsigned long long*>(nd.scratch + kNoAllocHeaderBytes);
  p.partials = reinterpret_cast<float*>(nd.scratch + kNoAllocHeaderBytes + sp.counters_bytes);
  p.tag = run_tag(next_plan_identity() << 24, 0);
  p.timeout_ns = 2000ull * 1000000ull;
  st = static_cast<gemm_status_t>(
      skinny_launch(p, tW, tX, tD, dev, s, g_last_cuda_error, sizeof g_last_cuda_error, /*tall=*/false, /*early_launch=*/false));
  if (st != GEMM_OK || !sync_and_check) return st;
  uint32_t word = 0;
  e = cudaStreamSynchronize(s);
  if (e == cudaSuccess) e = cudaMemcpy(&word, nd.scratch, sizeof word, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) {
    note_cuda_error("gemm_skinny_run_noalloc check", cudaGetErrorName(e));
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  if (word & kStatusTimeout) {
    snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "device wait expired: role %u detail 0x%02x", (word >> 8) & 0xFF,
             word & 0xFF);
    return GEMM_ERR_TIMEOUT;
  }
  return GEMM_OK;
}

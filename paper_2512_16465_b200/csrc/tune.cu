// Measured plan selection (gemm_tune) on top of the library's own public calls: candidates are ordinary plans with
// forced tuning fields, timed with CUDA events on the caller's buffers.  Which candidates are worth trying follows
// from the problem's roofline class (Section 4.3 of the paper: memory-bound kernels are tuned for streaming, compute-
// bound ones for tensor-pipe occupancy); the winner is remembered per device and shape.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>
#include <vector>

#include "../../include/gemm.h"
#include "tune_cache.h"

namespace b200 {
namespace {

using Key = std::tuple<int, int64_t, int64_t, int64_t, int32_t, int32_t, int32_t, int32_t, int64_t, int64_t, int64_t, int32_t, int32_t,
                       int64_t, int64_t, int64_t, uint32_t, uint32_t>;

Key key_of(const gemm_desc_t& d, int device) {
  const bool batched = d.batch_count > 1;
  return Key(device, d.M, d.N, d.K, d.transa, d.transb, d.ab_dtype, d.c_dtype, d.lda, d.ldb, d.ldc, d.batch_count, d.epilogue,
             batched ? d.stride_a : 0, batched ? d.stride_b : 0, batched ? d.stride_c : 0, d.flags & ~kTuningFlagMask, d.structure);
}

std::mutex g_mu;
std::map<Key, uint32_t>& cache() {
  static std::map<Key, uint32_t> m;
  return m;
}

uint32_t pack(int variant, int tile_n, int raster, int stages, int kslices) {
  const int tile_field = tile_n <= 256 ? tile_n / 16 : 16 + (tile_n - 256) / 64;  // (17 ... 20: the wide tiles 320 ... 512)
  return (static_cast<uint32_t>(variant) << GEMM_FLAG_VARIANT_SHIFT) | (static_cast<uint32_t>(tile_field) << GEMM_FLAG_TILE_N_SHIFT) |
         (static_cast<uint32_t>(raster) << GEMM_FLAG_RASTER_SHIFT) | (static_cast<uint32_t>(stages) << GEMM_FLAG_STAGES_SHIFT) |
         (static_cast<uint32_t>(kslices) << GEMM_FLAG_KSLICES_SHIFT);
}

bool short_extent(const gemm_desc_t& d) {
  return (d.M <= 64 || d.N <= 64) && d.batch_count == 1 && d.transa == GEMM_OP_N && d.transb == GEMM_OP_T;
}

// First round: one candidate per kernel family and tile width that the roofline class makes plausible.
std::vector<uint32_t> first_round(const gemm_desc_t& d, const gemm_info_t& automatic) {
  std::vector<uint32_t> c;
  const bool streaming = automatic.regime == GEMM_REGIME_MEMORY || automatic.intensity < 64.0;  // HBM-bound or close to it
  if (short_extent(d)) {
    for (int ks = 1; ks <= 3; ++ks) c.push_back(pack(GEMM_VARIANT_SKINNY_STREAMK, 0, 0, 0, ks));
  }
  if (streaming) {
    for (int bn : {64, 128, 256}) c.push_back(pack(GEMM_VARIANT_DENSE_1CTA, bn, 0, 0, 0));
  } else {
    for (int bn : {256, 128}) c.push_back(pack(GEMM_VARIANT_DENSE_1CTA, bn, 0, 0, 0));
    for (int bn : {256, 192, 128}) c.push_back(pack(GEMM_VARIANT_DENSE_2CTA, bn, 0, 0, 0));  // (192: refused, hence skipped, when B is stored K x N)
    // wide single-buffered pair tiles where they give every pair at most one tile (also refused when B is stored K x N)
    for (int bn : {320, 384, 448, 512})
      if (((d.M + 255) / 256) * ((d.N + bn - 1) / bn) * d.batch_count <= 74) c.push_back(pack(GEMM_VARIANT_DENSE_2CTA, bn, 0, 0, 0));
    c.push_back(pack(GEMM_VARIANT_DENSE_2CTA_WIDE, 0, 0, 0, 0));
  }
  return c;
}

// Second round: neighbours of the first-round winner (its plan `w`) in raster height and ring shape.
std::vector<uint32_t> second_round(uint32_t best, const gemm_info_t& w) {
  std::vector<uint32_t> c;
  if (w.variant == GEMM_VARIANT_SKINNY_STREAMK) {
    for (int st : {w.stages - 1, w.stages + 1})
      if (st >= 2 && st <= 8) c.push_back((best & ~GEMM_FLAG_STAGES_MASK) | (static_cast<uint32_t>(st) << GEMM_FLAG_STAGES_SHIFT));
    return c;
  }
  for (int rg : {w.raster_group / 2, w.raster_group * 2})
    if (rg >= 1 && rg <= 64 && rg != w.raster_group)
      c.push_back((best & ~GEMM_FLAG_RASTER_MASK) | (static_cast<uint32_t>(rg) << GEMM_FLAG_RASTER_SHIFT));
  if (w.variant != GEMM_VARIANT_DENSE_2CTA_WIDE) {
    c.push_back(best | GEMM_FLAG_TAIL_SPLIT);  // has an effect only where the last wave is thinly filled
    const int ks = w.tile_k / 64;  // 64-wide K slices per stage of the winner
    c.push_back((best & ~GEMM_FLAG_KSLICES_MASK) | (static_cast<uint32_t>(ks == 1 ? 2 : 1) << GEMM_FLAG_KSLICES_SHIFT));
  }
  return c;
}

struct Timer {
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  bool ok() { return cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess; }
  ~Timer() {
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
  }
};

struct Args {
  const void *A, *B;
  void* C;
  const float* bias;
  float alpha, beta;
  void* ws;
  size_t ws_bytes;
  cudaStream_t stream;
  int iterations;
};

// Plan `d` (flags already set), run and time it.  GEMM_OK with *ms < 0 means "not applicable here" (the plan was
// refused or needs more workspace than given); any other status is an error that ends the tuning.
gemm_status_t time_candidate(const gemm_desc_t& d, const Args& a, Timer& t, float* ms, gemm_info_t* info) {
  *ms = -1.0f;
  gemm_plan_t plan = nullptr;
  gemm_status_t st = gemm_plan(&d, &plan);
  if (st == GEMM_ERR_UNSUPPORTED || st == GEMM_ERR_INVALID_ARG) return GEMM_OK;
  if (st != GEMM_OK) return st;
  info->struct_size = sizeof *info;
  (void)gemm_plan_info(plan, info);
  if (gemm_workspace_bytes(plan) > a.ws_bytes) {
    gemm_destroy(plan);
    return GEMM_OK;
  }
  for (int i = 0; i < 2 && st == GEMM_OK; ++i) st = gemm_run(plan, a.A, a.B, a.C, a.bias, a.alpha, a.beta, a.ws, a.ws_bytes, a.stream);
  if (st == GEMM_OK && cudaEventRecord(t.e0, a.stream) != cudaSuccess) st = GEMM_ERR_CUDA;
  for (int i = 0; i < a.iterations && st == GEMM_OK; ++i) st = gemm_run(plan, a.A, a.B, a.C, a.bias, a.alpha, a.beta, a.ws, a.ws_bytes, a.stream);
  if (st == GEMM_OK && (cudaEventRecord(t.e1, a.stream) != cudaSuccess || cudaEventSynchronize(t.e1) != cudaSuccess)) st = GEMM_ERR_CUDA;
  float total = 0.0f;
  if (st == GEMM_OK && cudaEventElapsedTime(&total, t.e0, t.e1) != cudaSuccess) st = GEMM_ERR_CUDA;
  if (st == GEMM_OK) st = gemm_plan_status_stream(plan, a.stream);  // a candidate whose device-side wait expired is an error, not a slow plan
  gemm_destroy(plan);
  if (st == GEMM_OK) *ms = total / static_cast<float>(a.iterations);
  (void)cudaGetLastError();
  return st;
}

}  // namespace

bool tune_cache_lookup(const gemm_desc_t& d, int device, uint32_t* flags) {
  std::lock_guard<std::mutex> lock(g_mu);
  auto it = cache().find(key_of(d, device));
  if (it == cache().end()) return false;
  *flags = it->second;
  return true;
}

void tune_cache_store(const gemm_desc_t& d, int device, uint32_t flags) {
  std::lock_guard<std::mutex> lock(g_mu);
  cache()[key_of(d, device)] = flags & kTuningFlagMask;
}

}  // namespace b200

using namespace b200;

extern "C" void gemm_tune_cache_clear(void) {
  std::lock_guard<std::mutex> lock(g_mu);
  cache().clear();
}

// ---- keeping tuning results across processes -------------------------------------------------------------------
// A text file: one header line, then one line per remembered shape with the sixteen key fields after the device
// and the chosen tuning flags.  Results are written for, and read into, the current device: a file made on one GPU
// model means nothing on another, so the header carries the device name and the SM count and a mismatch is refused.
namespace {

constexpr const char* kTuneFileMagic = "b200gemm-tune-1";

bool current_device_tag(int* device, char* name, size_t len, int* sms) {
  cudaDeviceProp prop;
  if (cudaGetDevice(device) != cudaSuccess || cudaGetDeviceProperties(&prop, *device) != cudaSuccess) {
    (void)cudaGetLastError();
    return false;
  }
  snprintf(name, len, "%s", prop.name);
  for (char* c = name; *c; ++c)
    if (*c == ' ') *c = '_';
  *sms = prop.multiProcessorCount;
  return true;
}

}  // namespace

extern "C" gemm_status_t gemm_tune_cache_save(const char* path, int* entries) {
  if (!path) return GEMM_ERR_NULL;
  if (entries) *entries = 0;
  int device = -1, sms = 0;
  char name[256];
  if (!current_device_tag(&device, name, sizeof name, &sms)) return GEMM_ERR_ARCH;
  FILE* f = fopen(path, "w");
  if (!f) return GEMM_ERR_INVALID_ARG;
  int n = 0;
  bool ok = fprintf(f, "%s %s %d\n", kTuneFileMagic, name, sms) > 0;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    for (const auto& kv : cache()) {
      const Key& k = kv.first;
      if (std::get<0>(k) != device) continue;
      ok = ok && fprintf(f, "%lld %lld %lld %d %d %d %d %lld %lld %lld %d %d %lld %lld %lld %u %u %u\n",
                         (long long)std::get<1>(k), (long long)std::get<2>(k), (long long)std::get<3>(k), std::get<4>(k), std::get<5>(k),
                         std::get<6>(k), std::get<7>(k), (long long)std::get<8>(k), (long long)std::get<9>(k), (long long)std::get<10>(k),
                         std::get<11>(k), std::get<12>(k), (long long)std::get<13>(k), (long long)std::get<14>(k),
                         (long long)std::get<15>(k), std::get<16>(k), std::get<17>(k), kv.second) > 0;
      ++n;
    }
  }
  ok = (fclose(f) == 0) && ok;
  if (!ok) return GEMM_ERR_INVALID_ARG;
  if (entries) *entries = n;
  return GEMM_OK;
}

extern "C" gemm_status_t gemm_tune_cache_load(const char* path, int* entries) {
  if (!path) return GEMM_ERR_NULL;
  if (entries) *entries = 0;
  int device = -1, sms = 0;
  char name[256];
  if (!current_device_tag(&device, name, sizeof name, &sms)) return GEMM_ERR_ARCH;
  FILE* f = fopen(path, "r");
  if (!f) return GEMM_ERR_INVALID_ARG;
  char magic[64], file_name[256];
  int file_sms = 0;
  if (fscanf(f, "%63s %255s %d", magic, file_name, &file_sms) != 3 || strcmp(magic, kTuneFileMagic) != 0) {
    fclose(f);
    return GEMM_ERR_INVALID_ARG;
  }
  if (strcmp(file_name, name) != 0 || file_sms != sms) {  // measured on another kind of GPU
    fclose(f);
    return GEMM_ERR_UNSUPPORTED;
  }
  // read everything first: a malformed file changes nothing
  std::vector<std::pair<Key, uint32_t>> read;
  while (true) {
    long long M, N, K, lda, ldb, ldc, sa, sb, sc;
    int ta, tb, ab, cd, batch, epi;
    unsigned flags, structure, tuned;
    const int got = fscanf(f, "%lld %lld %lld %d %d %d %d %lld %lld %lld %d %d %lld %lld %lld %u %u %u", &M, &N, &K, &ta, &tb, &ab, &cd,
                           &lda, &ldb, &ldc, &batch, &epi, &sa, &sb, &sc, &flags, &structure, &tuned);
    if (got == EOF) break;
    if (got != 18 || (tuned & ~kTuningFlagMask) || (flags & kTuningFlagMask) || M < 1 || N < 1 || K < 1 || batch < 1) {
      fclose(f);
      return GEMM_ERR_INVALID_ARG;
    }
    read.emplace_back(Key(device, M, N, K, ta, tb, ab, cd, lda, ldb, ldc, batch, epi, sa, sb, sc, flags, structure), tuned);
  }
  fclose(f);
  std::lock_guard<std::mutex> lock(g_mu);
  for (const auto& kv : read) cache()[kv.first] = kv.second;
  if (entries) *entries = static_cast<int>(read.size());
  return GEMM_OK;
}

extern "C" size_t gemm_tune_workspace_bytes(const gemm_desc_t* desc) {
  if (!desc) return 0;
  size_t need = 0;
  auto consider = [&](uint32_t f) {
    gemm_desc_t d = *desc;
    d.flags = (d.flags & ~kTuningFlagMask) | f;
    gemm_plan_t plan = nullptr;
    if (gemm_plan(&d, &plan) != GEMM_OK) return;
    const size_t b = gemm_workspace_bytes(plan);
    if (b > need) need = b;
    gemm_destroy(plan);
  };
  // the candidates that use a workspace: stream-K (partial tiles) and the dense kernels with a tail split (second slices)
  if (short_extent(*desc))
    for (int ks = 1; ks <= 3; ++ks) consider(pack(GEMM_VARIANT_SKINNY_STREAMK, 0, 0, 0, ks));
  for (int v : {GEMM_VARIANT_DENSE_1CTA, GEMM_VARIANT_DENSE_2CTA})
    for (int bn : {256, 128, 64}) consider(pack(v, bn, 0, 0, 0) | GEMM_FLAG_TAIL_SPLIT);
  return need;
}

extern "C" gemm_status_t gemm_tune(const gemm_desc_t* desc, const void* A, const void* B, void* C, const float* bias, float alpha,
                                   float beta, void* workspace, size_t workspace_bytes, gemm_stream_t stream, int iterations,
                                   gemm_plan_t* out_plan, gemm_tune_report_t* report) {
  if (!desc || !out_plan || !A || !B || !C) return GEMM_ERR_NULL;
  *out_plan = nullptr;
  if (report && report->struct_size != sizeof(gemm_tune_report_t)) return GEMM_ERR_INVALID_ARG;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) {
    (void)cudaGetLastError();
    return GEMM_ERR_ARCH;
  }
  Timer timer;
  if (!timer.ok()) {
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  const Args args{A, B, C, bias, alpha, beta, workspace, workspace ? workspace_bytes : 0, static_cast<cudaStream_t>(stream),
                  iterations < 1 ? 10 : iterations};
  gemm_desc_t base = *desc;
  base.flags &= ~kTuningFlagMask;

  // The untuned automatic plan is the yardstick and the fallback.  (A remembered result must not answer for it.)
  {
    std::lock_guard<std::mutex> lock(g_mu);
    cache().erase(key_of(base, device));
  }
  gemm_tune_report_t rep;
  memset(&rep, 0, sizeof rep);
  rep.struct_size = sizeof rep;
  gemm_info_t auto_info, info;
  float ms = -1.0f;
  gemm_status_t st = time_candidate(base, args, timer, &ms, &auto_info);
  if (st != GEMM_OK) return st;
  if (ms < 0.0f) {  // the automatic plan itself could not run: report why
    gemm_plan_t probe = nullptr;
    st = gemm_plan(&base, &probe);
    if (st != GEMM_OK) return st;
    const bool ws_short = gemm_workspace_bytes(probe) > args.ws_bytes;
    gemm_destroy(probe);
    return ws_short ? GEMM_ERR_WORKSPACE : GEMM_ERR_UNSUPPORTED;
  }
  rep.auto_ms = ms;
  uint32_t best_flags = 0;  // 0 = the automatic plan
  float best_ms = ms;
  gemm_info_t best_info = auto_info;
  auto consider = [&](uint32_t f) -> gemm_status_t {
    for (int i = 0; i < rep.candidates_tried; ++i)
      if (rep.tried_flags[i] == f) return GEMM_OK;  // already timed
    if (rep.candidates_tried >= GEMM_TUNE_MAX_CANDIDATES) return GEMM_OK;
    gemm_desc_t d = base;
    d.flags |= f;
    float t = -1.0f;
    const gemm_status_t s = time_candidate(d, args, timer, &t, &info);
    if (s != GEMM_OK) return s;
    if (t < 0.0f) {
      ++rep.candidates_skipped;
      return GEMM_OK;
    }
    rep.tried_flags[rep.candidates_tried] = f;
    rep.tried_ms[rep.candidates_tried] = t;
    ++rep.candidates_tried;
    if (t < best_ms) {
      best_ms = t;
      best_flags = f;
      best_info = info;
    }
    return GEMM_OK;
  };
  rep.tried_flags[0] = 0;
  rep.tried_ms[0] = ms;
  rep.candidates_tried = 1;
  for (uint32_t f : first_round(base, auto_info)) {
    st = consider(f);
    if (st != GEMM_OK) return st;
  }
  // neighbours of the winner; if the winner is the automatic plan, pin its own choices down first
  uint32_t pinned = best_flags;
  if (pinned == 0)
    pinned = pack(best_info.variant, (best_info.variant == GEMM_VARIANT_DENSE_1CTA || best_info.variant == GEMM_VARIANT_DENSE_2CTA) ? best_info.tile_n : 0, 0, 0, 0);
  for (uint32_t f : second_round(pinned, best_info)) {
    st = consider(f);
    if (st != GEMM_OK) return st;
  }

  gemm_desc_t win = base;
  win.flags |= best_flags;
  st = gemm_plan(&win, out_plan);
  if (st != GEMM_OK) return st;
  tune_cache_store(base, device, best_flags);
  rep.best_flags = win.flags;
  rep.best_ms = best_ms;
  if (report) *report = rep;
  return GEMM_OK;
}

// GEMM on host-resident operands: row panels of A stream in, are multiplied, and stream out on three streams, so
// host-to-device copy, tensor-core work and device-to-host copy overlap.  Built on the library's own public calls
// (every panel is an ordinary plan run by gemm_run); this file owns only buffers, streams and events.
#include <cuda_runtime.h>

#include <cstring>
#include <new>

#include "../../include/gemm.h"

struct gemm_host_s {
  gemm_desc_t d;
  int device;
  int panels;
  int64_t rows;          // rows of a full panel (the last one may be shorter)
  int64_t last_rows;     // rows of the last panel
  gemm_plan_t plan_full;
  gemm_plan_t plan_last; // == plan_full when the last panel is a full one
  size_t a_elem, c_elem;
  void* dB;
  float* dbias;
  void* dA[2];
  void* dC[2];
  void* ws;
  size_t ws_bytes;
  cudaStream_t s_in, s_mm, s_out;
  cudaEvent_t b_ready, a_ready[2], mm_done[2], c_out[2];
};

namespace {

size_t elem_size(int dtype) { return dtype == GEMM_F32 ? 4 : ((dtype == GEMM_FP8_E4M3 || dtype == GEMM_FP8_E5M2) ? 1 : 2); }
bool bias_epilogue(int e) { return (e & 1) != 0; }

void release(gemm_host_s* h) {
  if (!h) return;
  if (h->plan_last && h->plan_last != h->plan_full) gemm_destroy(h->plan_last);
  if (h->plan_full) gemm_destroy(h->plan_full);
  void* bufs[] = {h->dB, h->dbias, h->dA[0], h->dA[1], h->dC[0], h->dC[1], h->ws};
  for (void* b : bufs)
    if (b) cudaFree(b);
  cudaStream_t streams[] = {h->s_in, h->s_mm, h->s_out};
  for (cudaStream_t s : streams)
    if (s) cudaStreamDestroy(s);
  cudaEvent_t events[] = {h->b_ready, h->a_ready[0], h->a_ready[1], h->mm_done[0], h->mm_done[1], h->c_out[0], h->c_out[1]};
  for (cudaEvent_t e : events)
    if (e) cudaEventDestroy(e);
  (void)cudaGetLastError();
  delete h;
}

}  // namespace

extern "C" gemm_status_t gemm_host_create(const gemm_desc_t* desc, int panels, gemm_host_t* out) {
  if (!desc || !out) return GEMM_ERR_NULL;
  *out = nullptr;
  if (desc->struct_size != sizeof(gemm_desc_t) || panels < 0) return GEMM_ERR_INVALID_ARG;
  if (desc->transa != GEMM_OP_N || desc->batch_count != 1) return GEMM_ERR_UNSUPPORTED;
  // a triangular op(A), or a wanted triangle of D, would have a different diagonal position in every row panel
  if ((desc->flags & (GEMM_FLAG_A_LOWER | GEMM_FLAG_A_UPPER | GEMM_FLAG_D_LOWER | GEMM_FLAG_D_UPPER)) || desc->structure) return GEMM_ERR_UNSUPPORTED;
  gemm_host_s* h = new (std::nothrow) gemm_host_s();
  if (!h) return GEMM_ERR_CUDA;
  memset(h, 0, sizeof *h);
  h->d = *desc;
  if (cudaGetDevice(&h->device) != cudaSuccess) {
    release(h);
    return GEMM_ERR_ARCH;
  }
  // panel height: a multiple of 256 rows (the largest tile height) so that only the last panel has a ragged tile row
  const int64_t M = desc->M;
  int want = panels ? panels : 8;
  int64_t rows = (M + want - 1) / want;
  rows = (rows + 255) / 256 * 256;
  if (rows > M) rows = M;
  h->rows = rows;
  h->panels = static_cast<int>((M + rows - 1) / rows);
  h->last_rows = M - static_cast<int64_t>(h->panels - 1) * rows;
  gemm_desc_t pd = *desc;
  pd.M = rows;
  gemm_status_t st = gemm_plan(&pd, &h->plan_full);
  if (st == GEMM_OK) {
    if (h->last_rows == rows) {
      h->plan_last = h->plan_full;
    } else {
      pd.M = h->last_rows;
      st = gemm_plan(&pd, &h->plan_last);
    }
  }
  if (st != GEMM_OK) {
    release(h);
    return st;
  }
  h->a_elem = elem_size(desc->ab_dtype);
  h->c_elem = elem_size(desc->c_dtype);
  const size_t b_rows = desc->transb == GEMM_OP_T ? desc->N : desc->K;
  const size_t b_bytes = b_rows * desc->ldb * h->a_elem;
  const size_t a_bytes = static_cast<size_t>(rows) * desc->lda * h->a_elem;
  const size_t c_bytes = static_cast<size_t>(rows) * desc->ldc * h->c_elem;
  h->ws_bytes = gemm_workspace_bytes(h->plan_full);
  if (gemm_workspace_bytes(h->plan_last) > h->ws_bytes) h->ws_bytes = gemm_workspace_bytes(h->plan_last);
  const size_t bias_elems = (desc->flags & GEMM_FLAG_BIAS_PER_ROW) ? desc->M : desc->N;
  bool ok = cudaMalloc(&h->dB, b_bytes) == cudaSuccess;
  for (int i = 0; i < 2 && ok; ++i) ok = cudaMalloc(&h->dA[i], a_bytes) == cudaSuccess && cudaMalloc(&h->dC[i], c_bytes) == cudaSuccess;
  if (ok && bias_epilogue(desc->epilogue)) ok = cudaMalloc(&h->dbias, bias_elems * sizeof(float)) == cudaSuccess;
  if (ok && h->ws_bytes) ok = cudaMalloc(&h->ws, h->ws_bytes) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) == cudaSuccess &&
       cudaStreamCreateWithFlags(&h->s_mm, cudaStreamNonBlocking) == cudaSuccess &&
       cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&h->b_ready, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < 2 && ok; ++i)
    ok = cudaEventCreateWithFlags(&h->a_ready[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&h->mm_done[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&h->c_out[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    release(h);
    return GEMM_ERR_CUDA;
  }
  *out = h;
  return GEMM_OK;
}

extern "C" int gemm_host_panels(gemm_host_t h) { return h ? h->panels : 0; }

extern "C" gemm_status_t gemm_host_run(gemm_host_t h, const void* hA, const void* hB, void* hC, const float* hbias, float alpha,
                                       float beta) {
  if (!h || !hA || !hB || !hC) return GEMM_ERR_NULL;
  const gemm_desc_t& d = h->d;
  if (bias_epilogue(d.epilogue) && !hbias) return GEMM_ERR_NULL;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess || cur != h->device) return GEMM_ERR_INVALID_ARG;
  // B is copied up to the last element of its last row: the caller's buffer need not hold the padding behind it
  const size_t b_rows = d.transb == GEMM_OP_T ? d.N : d.K, b_row_len = d.transb == GEMM_OP_T ? d.K : d.N;
  bool ok = cudaMemcpyAsync(h->dB, hB, ((b_rows - 1) * d.ldb + b_row_len) * h->a_elem, cudaMemcpyHostToDevice, h->s_in) == cudaSuccess;
  if (ok && h->dbias) {
    const size_t n = (d.flags & GEMM_FLAG_BIAS_PER_ROW) ? d.M : d.N;
    ok = cudaMemcpyAsync(h->dbias, hbias, n * sizeof(float), cudaMemcpyHostToDevice, h->s_in) == cudaSuccess;
  }
  ok = ok && cudaEventRecord(h->b_ready, h->s_in) == cudaSuccess && cudaStreamWaitEvent(h->s_mm, h->b_ready, 0) == cudaSuccess;
  gemm_status_t st = GEMM_OK;
  for (int p = 0; p < h->panels && ok && st == GEMM_OK; ++p) {
    const int b = p & 1;
    const int64_t r0 = static_cast<int64_t>(p) * h->rows;
    const int64_t nr = p + 1 == h->panels ? h->last_rows : h->rows;
    const char* srcA = static_cast<const char*>(hA) + static_cast<size_t>(r0) * d.lda * h->a_elem;
    char* hostC = static_cast<char*>(hC) + static_cast<size_t>(r0) * d.ldc * h->c_elem;
    // C moves as a pitched copy: only the N elements of each row, never the padding between rows
    const size_t c_pitch = static_cast<size_t>(d.ldc) * h->c_elem, c_width = static_cast<size_t>(d.N) * h->c_elem;
    // in: the A slice may overwrite buffer b once panel p-2 has been multiplied; C_in (beta != 0) once its result left
    if (p >= 2) ok = cudaStreamWaitEvent(h->s_in, h->mm_done[b], 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h->dA[b], srcA, (static_cast<size_t>(nr - 1) * d.lda + d.K) * h->a_elem, cudaMemcpyHostToDevice,
                               h->s_in) == cudaSuccess;
    if (ok && beta != 0.0f) {
      if (p >= 2) ok = cudaStreamWaitEvent(h->s_in, h->c_out[b], 0) == cudaSuccess;
      ok = ok && cudaMemcpy2DAsync(h->dC[b], c_pitch, hostC, c_pitch, c_width, static_cast<size_t>(nr), cudaMemcpyHostToDevice, h->s_in) == cudaSuccess;
    }
    ok = ok && cudaEventRecord(h->a_ready[b], h->s_in) == cudaSuccess;
    // multiply: needs the slice, and a C buffer whose previous result has left
    ok = ok && cudaStreamWaitEvent(h->s_mm, h->a_ready[b], 0) == cudaSuccess;
    if (ok && p >= 2) ok = cudaStreamWaitEvent(h->s_mm, h->c_out[b], 0) == cudaSuccess;
    if (ok) {
      const float* bias = h->dbias;
      if (bias && (d.flags & GEMM_FLAG_BIAS_PER_ROW)) bias += r0;  // (16-byte aligned: r0 is a multiple of 256)
      st = gemm_run(p + 1 == h->panels ? h->plan_last : h->plan_full, h->dA[b], h->dB, h->dC[b], bias, alpha, beta, h->ws, h->ws_bytes,
                    h->s_mm);
    }
    ok = ok && st == GEMM_OK && cudaEventRecord(h->mm_done[b], h->s_mm) == cudaSuccess;
    // out
    ok = ok && cudaStreamWaitEvent(h->s_out, h->mm_done[b], 0) == cudaSuccess &&
         cudaMemcpy2DAsync(hostC, c_pitch, h->dC[b], c_pitch, c_width, static_cast<size_t>(nr), cudaMemcpyDeviceToHost, h->s_out) == cudaSuccess &&
         cudaEventRecord(h->c_out[b], h->s_out) == cudaSuccess;
  }
  // everything this run enqueued must have finished before the caller may touch its buffers (or run again)
  const bool drained = cudaStreamSynchronize(h->s_in) == cudaSuccess && cudaStreamSynchronize(h->s_mm) == cudaSuccess &&
                       cudaStreamSynchronize(h->s_out) == cudaSuccess;
  if (st != GEMM_OK) return st;
  if (!ok || !drained) {
    (void)cudaGetLastError();
    return GEMM_ERR_CUDA;
  }
  st = gemm_plan_status_stream(h->plan_full, h->s_mm);
  if (st == GEMM_OK && h->plan_last != h->plan_full) st = gemm_plan_status_stream(h->plan_last, h->s_mm);
  return st;
}

extern "C" gemm_status_t gemm_host_destroy(gemm_host_t h) {
  release(h);
  return GEMM_OK;
}

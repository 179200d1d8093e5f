// Copy one triangle of a square row-major matrix into the other (D becomes symmetric): the second step of a
// symmetric result (GEMM_STRUCT_D_MIRROR), run after the GEMM kernel that computed the wanted triangle.  Pure data
// movement, HBM-bound: every element of the wanted triangle is read once and one element written per element read.
//
// The matrix is cut into 32 x 32 blocks.  A thread block takes one block (bi, bj) with bi > bj of the wanted lower
// triangle (for an upper source: bi < bj), reads it row by row (32 lanes = 32 consecutive columns: coalesced),
// turns it in shared memory (padded: no bank conflicts) and writes block (bj, bi) row by row.  Diagonal blocks
// (bi == bj) mirror inside themselves: only the elements strictly beyond the diagonal are written.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace b200 {

struct MirrorParams {
  void* d;              // device: the matrix (all batches)
  long long ldc, stride;  // elements
  int n;                // extent (M == N)
  int blocks;           // ceil(n / 32)
  int upper_source;     // 0: the lower triangle (row >= column) is the source; 1: the upper one
};

// Linear index t of a block pair -> (bi, bj), bj <= bi: row bi of the triangle holds bi + 1 pairs.
__device__ __forceinline__ void mirror_pair(int t, int* bi, int* bj) {
  int r = static_cast<int>((sqrtf(8.0f * static_cast<float>(t) + 1.0f) - 1.0f) * 0.5f);
  while (r * (r + 1) / 2 > t) --r;  // (the float square root may be off by one either way)
  while ((r + 1) * (r + 2) / 2 <= t) ++r;
  *bi = r;
  *bj = t - r * (r + 1) / 2;
}

template <typename T>
__global__ void __launch_bounds__(256) mirror_kernel(const MirrorParams p) {
  __shared__ T tile[32][33];
  int bi, bj;
  mirror_pair(static_cast<int>(blockIdx.x), &bi, &bj);
  if (p.upper_source) {  // source block (bj, bi) of the upper triangle, destination (bi, bj)
    const int t = bi;
    bi = bj;
    bj = t;
  }
  T* base = static_cast<T*>(p.d) + static_cast<long long>(blockIdx.y) * p.stride;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8 threads: four rows each
  const int r0 = bi * 32, c0 = bj * 32;                     // source block
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int r = r0 + ty + 8 * k, c = c0 + tx;
    if (r < p.n && c < p.n) tile[ty + 8 * k][tx] = base[static_cast<long long>(r) * p.ldc + c];
  }
  __syncthreads();
  // destination block (bj, bi): element (c0 + y, r0 + x) takes source element (r0 + x, c0 + y)
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int y = ty + 8 * k;
    const int dr = c0 + y, dc = r0 + tx;
    if (dr >= p.n || dc >= p.n) continue;
    // write only what lies strictly in the other triangle (matters in the diagonal blocks)
    const bool other = p.upper_source ? (dr > dc) : (dr < dc);
    if (other) base[static_cast<long long>(dr) * p.ldc + dc] = tile[tx][y];
  }
}

// Launch on `stream` after the kernel that wrote the source triangle (plain stream order).  elem_bytes: 2 or 4.
inline cudaError_t mirror_launch(const MirrorParams& p, int elem_bytes, int batch, cudaStream_t stream) {
  const long long pairs = static_cast<long long>(p.blocks) * (p.blocks + 1) / 2;
  if (pairs > 0x7FFFFFFFll || batch > 65535) return cudaErrorInvalidValue;
  const dim3 grid(static_cast<unsigned>(pairs), static_cast<unsigned>(batch), 1);
  if (elem_bytes == 4) mirror_kernel<uint32_t><<<grid, 256, 0, stream>>>(p);
  else mirror_kernel<uint16_t><<<grid, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace b200

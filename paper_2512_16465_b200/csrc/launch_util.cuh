// Host-side launch helper shared by the kernel launchers.
#pragma once
#include <cuda_runtime.h>

#include <mutex>

namespace b200 {

constexpr int kMaxDevices = 64;
enum KernelSlot { kSlotDense11 = 0, kSlotDense12, kSlotDense21, kSlotDense22, kSlotDenseSplit11, kSlotDenseSplit12, kSlotDenseSplit21, kSlotDenseSplit22, kSlotWide, kSlotWideFp8, kSlotSkinny, kSlotSkinnyTall, kSlotSkinnyCluster, kSlotSkinnyTallCluster, kNumKernelSlots };

// Opt a kernel in to `bytes` of dynamic shared memory on the current device.  The attribute is per kernel and per
// device, and only ever needs to grow, so the largest value set so far is remembered per (kernel, device).
inline cudaError_t ensure_dynamic_smem(const void* func, KernelSlot slot, int device, int bytes) {
  static int configured[kNumKernelSlots][kMaxDevices] = {};
  static std::mutex mu;
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (configured[slot][device] >= bytes) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) configured[slot][device] = bytes;
  return e;
}

}  // namespace b200

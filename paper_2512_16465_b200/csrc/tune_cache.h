// Per-process memory of measured plan choices (filled by gemm_tune, consulted by gemm_plan).
#pragma once
#include <cstdint>

#include "../../include/gemm.h"

namespace b200 {

// The tuning fields of gemm_desc_t.flags (everything gemm_tune may choose); the remaining bits change what is
// computed or how it is launched and belong to the caller.
constexpr uint32_t kTuningFlagMask = GEMM_FLAG_VARIANT_MASK | GEMM_FLAG_TILE_N_MASK | GEMM_FLAG_RASTER_MASK | GEMM_FLAG_STAGES_MASK |
                                     GEMM_FLAG_KSLICES_MASK | GEMM_FLAG_TAIL_SPLIT;

// True (and *flags = the remembered tuning fields) if this shape was tuned on this device.
bool tune_cache_lookup(const gemm_desc_t& d, int device, uint32_t* flags);
void tune_cache_store(const gemm_desc_t& d, int device, uint32_t flags);

}  // namespace b200

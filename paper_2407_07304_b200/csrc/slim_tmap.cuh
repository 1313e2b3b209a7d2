// Host-side helpers shared by the kernels that stage cache tiles with the TMA copy engine.
#pragma once
#include <cuda.h>

#include "../../include/slim.h"

namespace slim {

// Tensor map of the code pool seen as [rows][128 bytes] with boxes of box_rows rows (a multiple
// of 8) and the 128-byte swizzle.  Maps are cached per (pool pointer, size, box); thread-safe.
int codes_tensor_map(const slim_cache_t *c, int box_rows, CUtensorMap *out);

// Number of SMs of the current device (cached per device).
int sm_count(int *out);

// cudaFuncSetAttribute(func, MaxDynamicSharedMemorySize, bytes), issued once per (device, kernel) instead of on
// every launch; thread-safe.
int allow_dynamic_smem(const void *func, int bytes);

}  // namespace slim

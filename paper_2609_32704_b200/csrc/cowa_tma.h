// Host helper: tiled TMA tensor maps over contiguous [BH, T, D] tensors (D innermost).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "cowa_common.h"

namespace cowa {

enum class MapType { BF16, F32, S32 };

// Builds a 3-D map with dims (D, T, BH) and box (box_d, box_t, 1); with `swizzle128` the shared
// memory side uses the 128-byte swizzle (box_d * element size must then be 128 bytes or less),
// otherwise rows are stored linearly.  Out-of-range rows read as zero and are dropped on stores.
// Returns COWA_OK / COWA_ERR_CUDA.
int make_tensor_map_3d(CUtensorMap* map, const void* base, MapType type, int D, int T, long long BH, int box_d,
                       int box_t, bool swizzle128 = true);

}  // namespace cowa

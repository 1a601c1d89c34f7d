// Host helper: tiled TMA tensor maps over [B, H, T, D] tensors (D innermost and contiguous; batch, head
// and token strides free).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "cowa_common.h"

namespace cowa {

enum class MapType { BF16, F32, S32 };

// Builds a 4-D map with dims (D, T, H, B), element strides st (batch, head, token) and box
// (box_d, box_t, 1, 1); with `swizzle128` the shared memory side uses the 128-byte swizzle (box_d * element
// size must then be 128 bytes or less), otherwise rows are stored linearly.  Out-of-range rows read as zero
// and are dropped on stores.  Returns COWA_OK / COWA_ERR_CUDA.
int make_tensor_map(CUtensorMap* map, const void* base, MapType type, int D, long long T, int H, int B,
                    const CowaStrides& st, int box_d, int box_t, bool swizzle128 = true);

}  // namespace cowa

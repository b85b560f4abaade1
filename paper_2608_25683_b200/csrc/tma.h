// Host-side construction of TMA tensor maps (cuTensorMapEncodeTiled, resolved
// at run time through the CUDA runtime so the library does not link libcuda).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace psrl {

// 2-D bf16 tensor [rows, cols] with a row pitch of `pitch_bytes`, boxes of
// box_rows x 64 columns, 128-byte swizzle, out-of-range elements read as zero.
// Returns false (and records the error) if the driver call fails.
bool make_map_bf16_2d(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                      uint32_t box_rows);

}  // namespace psrl

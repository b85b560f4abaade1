#include "tma.h"

#include <mutex>

#include "kernels.h"

namespace psrl {
namespace {
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode = nullptr;
std::once_flag g_once;

void resolve() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qr;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr);
  if (e == cudaSuccess && qr == cudaDriverEntryPointSuccess) g_encode = reinterpret_cast<EncodeFn>(fn);
  else set_last_cuda_error(e == cudaSuccess ? cudaErrorNotSupported : e);
}
}  // namespace

namespace {
// Encoded maps are kept: a tensor map is a pure function of (base, shape, pitch, box), and a training step
// calls the library with the same tensors step after step, so in steady state no call encodes anything
// (a forward + backward would otherwise encode ~30 maps on the host, which is what bounds the time of a
// launch-bound small case).  Small direct-mapped table, one mutex.
struct MapKey {
  const void* base;
  uint64_t cols, rows, pitch;
  uint32_t box_rows;
  bool operator==(const MapKey& o) const {
    return base == o.base && cols == o.cols && rows == o.rows && pitch == o.pitch && box_rows == o.box_rows;
  }
};
struct MapSlot {
  bool used = false;
  MapKey key{};
  CUtensorMap map;
};
constexpr size_t kMapSlots = 256;
MapSlot g_maps[kMapSlots];
std::mutex g_maps_mu;
size_t map_hash(const MapKey& k) {
  uint64_t h = reinterpret_cast<uint64_t>(k.base) * 0x9E3779B97F4A7C15ull;
  h ^= (k.rows + 0x7F4A7C15ull) * 0xBF58476D1CE4E5B9ull;
  h ^= (k.cols * 31 + k.pitch * 17 + k.box_rows) * 0x94D049BB133111EBull;
  return size_t((h >> 29) % kMapSlots);
}
}  // namespace

bool make_map_bf16_2d(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                      uint32_t box_rows) {
  std::call_once(g_once, resolve);
  if (!g_encode) return false;
  const MapKey key{base, cols, rows, pitch_bytes, box_rows};
  const size_t slot = map_hash(key);
  {
    std::lock_guard<std::mutex> lock(g_maps_mu);
    if (g_maps[slot].used && g_maps[slot].key == key) {
      *map = g_maps[slot].map;
      return true;
    }
  }
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t es[2] = {1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error(cudaErrorInvalidValue);
    return false;
  }
  {
    std::lock_guard<std::mutex> lock(g_maps_mu);
    g_maps[slot].used = true;
    g_maps[slot].key = key;
    g_maps[slot].map = *map;
  }
  return true;
}

}  // namespace psrl

// Pieces shared by the bf16 tensor-core kernels: tile geometry and the TMA
// gather of one KV tile from the paged pools.
#pragma once
#include "plan.h"
#include "sm100.cuh"

namespace psrl {

constexpr int kTileBytes = 128 * 128 * 2;  // one 128 x 128 bf16 tile = two 128 x 64 halves
constexpr int kHalfBytes = kTileBytes / 2; // each half: 128 rows of 128 bytes, 128-byte swizzle
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Tensor maps over the K and V pools, one per box height (16, 32, 64, 128 rows).
struct PoolMaps {
  CUtensorMap k[4];
  CUtensorMap v[4];
};

__device__ __forceinline__ int map_index(int bs) { return bs >= 128 ? 3 : (bs == 64 ? 2 : (bs == 32 ? 1 : 0)); }

// Gather one KV tile (its pages, located through the block metadata) into a
// 128 x 128 shared-memory tile; rows beyond kt.rows_loaded are left untouched.
__device__ __forceinline__ void load_kv_tile(uint8_t* dst, const CUtensorMap* maps, uint64_t* bar, const KvTile& kt,
                                             const int32_t* page_slot, int64_t head_row0) {
  using namespace sm100;
  const int rows_per_box = kt.bs >= 128 ? 128 : kt.bs;
  const CUtensorMap* m = maps + map_index(kt.bs);
  mbar_expect_tx(bar, uint32_t(kt.rows_loaded) * 256u);
  for (int i = 0; i < kt.n_pages; ++i) {
    const int row = int(head_row0 + page_slot[kt.first_page + i] + kt.row_off);
    uint8_t* d = dst + i * rows_per_box * 128;
    tma_load_2d(d, m, bar, 0, row);
    tma_load_2d(d + kHalfBytes, m, bar, 64, row);
  }
}

// The same from host-resolved coordinates (TileLoad): no metadata load between the ring wait and
// the TMA instructions.
__device__ __forceinline__ void load_kv_tile_at(uint8_t* dst, const CUtensorMap* maps, uint64_t* bar, const TileLoad& tl,
                                                int64_t head_row0) {
  using namespace sm100;
  const int rows_per_box = tl.bs >= 128 ? 128 : tl.bs;
  const CUtensorMap* m = maps + map_index(tl.bs);
  mbar_expect_tx(bar, uint32_t(tl.rows_loaded) * 256u);
  if (tl.n_pages == 1) {
    // the common case (pages contiguous in the pool): one box per half, and as few instructions as
    // possible - the producer shares its scheduler with two softmax warps
    const int row = int(head_row0 + tl.row[0]);
    tma_load_2d(dst, m, bar, 0, row);
    tma_load_2d(dst + kHalfBytes, m, bar, 64, row);
    return;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (i < tl.n_pages) {
      uint8_t* d = dst + i * rows_per_box * 128;
      const int row = int(head_row0 + tl.row[i]);
      tma_load_2d(d, m, bar, 0, row);
      tma_load_2d(d + kHalfBytes, m, bar, 64, row);
    }
  }
}

// One 128 x 128 row-tile of a [rows, Hq*128] tensor (Q, dO): head h, first row `row`.
__device__ __forceinline__ void load_row_tile(uint8_t* dst, const CUtensorMap* m, uint64_t* bar, int h, int row) {
  sm100::tma_load_2d(dst, m, bar, h * 128, row);
  sm100::tma_load_2d(dst + kHalfBytes, m, bar, h * 128 + 64, row);
}

// Zero row `row` of a 128 x 128 tile (both halves).  With the 128-byte swizzle a
// row's 128 bytes stay inside the row, so whole-row zeroing needs no swizzle math.
__device__ __forceinline__ void zero_tile_row(uint8_t* tile, int row) {
  uint8_t* r = tile + row * 128;
#pragma unroll
  for (int x = 0; x < 8; ++x) {
    *reinterpret_cast<uint4*>(r + x * 16) = make_uint4(0, 0, 0, 0);
    *reinterpret_cast<uint4*>(r + kHalfBytes + x * 16) = make_uint4(0, 0, 0, 0);
  }
}

// Block order of the three main kernels: block b -> (work item, unit u of the item; u = KV head, query head or
// head pair).  chunk == 0: item-major (b = item * per_item + u), which keeps the longest-first order of the items
// exact - used for small launches, where that order is what balances the SMs.  chunk > 0 (large launches):
// unit-major inside chunks of `chunk` items, so that the CTAs that run at the same time mostly share one KV head:
// they then stream the same K/V tiles (forward, dQ) or the Q and dO rows of the same query heads (dK/dV), which
// compete for the L2 with a quarter or an eighth of the whole set.  The chunks still follow the longest-first order.
__device__ __forceinline__ void block_to_item(int b, int n_items, int per_item, int chunk, int& item, int& u) {
  if (chunk > 0) {
    const int per = chunk * per_item;
    const int c = b / per, r = b % per;
    const int in_chunk = min(chunk, n_items - c * chunk);
    u = r / in_chunk;
    item = c * chunk + r % in_chunk;
  } else {
    item = b / per_item;
    u = b % per_item;
  }
}
// Items per chunk for a launch of n_items work items on a device with n_sm SMs (0 = item-major): chunks of
// one item per SM once the launch has at least `min_waves` items per SM (measured: dK/dV gains from one wave
// on, -3 % on the 276-item tree configuration and -6 % on the large ones; dQ only on the large ones, -2 %).
inline int block_order_chunk(int64_t n_items, int n_sm, int min_waves) {
  return n_items >= int64_t(min_waves) * n_sm ? n_sm : 0;
}

bool make_pool_maps(PoolMaps* maps, const void* k_pool, const void* v_pool, int Hkv, int64_t cap);

}  // namespace psrl

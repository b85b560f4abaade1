// bf16 dK/dV kernel (key-stationary) and the fixed-order reduce of split tiles.
//
// One CTA = one work item: a KV tile (<= 128 keys of one segment, one KV head)
// and a range of 64-row query sub-tiles that attend to it - the later rows of
// the tile's own segment, then the rows of ALL descendant segments, which form
// one contiguous row range in the canonical layout (paper Sec. 6: the adjoints
// of every consumer are accumulated on the shared prefix) - times the Hq/Hkv
// query heads of the KV head.  K and V stay in shared memory; dK and dV
// accumulate in tensor memory over the whole loop.
//
// Per step (64 query rows of one head):
//   MMA1  S^T = K Q^T, dP^T = V dO^T     M = 128 keys, N = 64 rows, both operands in smem
//   warps P^T = exp2(S^T c - LSE), dS^T = P^T o (dP^T - D), written back to
//         tensor memory as packed bf16 over the S^T / dP^T columns they came from
//   MMA2  dV += P^T dO, dK += dS^T Q      A from tensor memory, dO / Q MN-major in smem
// S^T and dP^T are double-buffered in tensor memory (2 x 64 columns each), so
// MMA1 of step i+1 is issued before the warps have finished step i and the
// tensor cores stay busy while the exponentials are computed.
//
// Tensor memory (512 columns): S^T[2] at 0/64, dP^T[2] at 128/192, dV at 256, dK at 384.
// Heavy tiles are split over several CTAs by the plan; a split item writes its
// fp32 partial to a workspace slab and reduce_kernel adds the parts in part
// order (no atomics: bitwise reproducible).
#include <cuda_bf16.h>
#include <math_constants.h>

#include "attn_bf16_common.cuh"
#include "kernels.h"
#include "tma.h"

namespace psrl {
namespace {
using namespace sm100;

constexpr int ST = 4;                              // (Q, dO) sub-tile ring depth
constexpr int kSubBytes = kSubRows * 128 * 2;      // 64 x 128 bf16 = two 64 x 64 halves
constexpr int kSubHalf = kSubBytes / 2;
constexpr int kThreads = (8 + 2) * 32;             // 8 softmax-backward warps + producer + MMA
constexpr uint32_t TM_ST = 0, TM_DPT = 128, TM_DV = 256, TM_DK = 384;

struct Maps {
  CUtensorMap q, d_o;  // boxes of 64 rows x 64 columns
  PoolMaps kv;
};
struct Params {
  const int32_t* blob;
  int32_t off_kvi, off_kvt, off_page_slot, off_split;
  int32_t Hq, Hkv, G, T_q;
  int64_t cap;
  float scale, scale_log2;
  const float* lse;
  const float* delta;
  float* slabs;
  __nv_bfloat16 *dk, *dv;
  int* status;
};
struct __align__(8) Barriers {
  uint64_t kv_full, qd_full[ST], qd_empty[ST], st_full[2], pd_ready[2], acc_full;
};

// Slot of key row `row` of a KV tile in the pools.
__device__ __forceinline__ int64_t tile_row_slot(const KvTile& kt, const int32_t* page_slot, int row) {
  const int rows_per_box = kt.bs >= 128 ? 128 : kt.bs;
  return int64_t(page_slot[kt.first_page + row / rows_per_box]) + kt.row_off + row % rows_per_box;
}

__global__ void __launch_bounds__(kThreads, 1)
dkv_kernel(const __grid_constant__ Maps maps, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = smem;
  uint8_t* sV = sK + kTileBytes;
  uint8_t* sQ = sV + kTileBytes;             // ST sub-tiles
  uint8_t* sdO = sQ + ST * kSubBytes;        // ST sub-tiles
  __shared__ Barriers bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ __align__(16) float s_lse[ST][kSubRows], s_dl[ST][kSubRows];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int item = blockIdx.x / p.Hkv, hk = blockIdx.x % p.Hkv;
  const KvItem it = reinterpret_cast<const KvItem*>(p.blob + p.off_kvi)[item];
  const KvTile kt = reinterpret_cast<const KvTile*>(p.blob + p.off_kvt)[it.kvt];
  const int n_own_sub = it.own_q_row0 >= 0 ? (it.own_q_end - it.own_q_row0 + kSubRows - 1) / kSubRows : 0;
  const int n_it = (it.sub_end - it.sub_begin) * p.G;

  if (tid == 0) {
    s_abort = 0;
    mbar_init(&bar.kv_full, 1);
    for (int i = 0; i < ST; ++i) { mbar_init(&bar.qd_full[i], 2); mbar_init(&bar.qd_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bar.st_full[i], 1); mbar_init(&bar.pd_ready[i], 256); }
    mbar_init(&bar.acc_full, 1);
    fence_mbar_init();
  }
  if (warp == 9) { tmem_alloc(&s_tmem, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;

  // step i -> head g and sub-tile: first row, valid rows, position of the first row relative
  // to the tile's first key (only meaningful, and only used, when `diag` is set)
  auto step = [&](int i, int& g, int& row0, int& nvq, bool& diag, int& qpos0) {
    const int su = it.sub_begin + i / p.G;
    g = i % p.G;
    if (su < n_own_sub) {
      row0 = it.own_q_row0 + su * kSubRows;
      nvq = min(kSubRows, it.own_q_end - row0);
      diag = su < 128 / kSubRows;
      qpos0 = su * kSubRows;
    } else {
      row0 = it.desc_q_begin + (su - n_own_sub) * kSubRows;
      nvq = min(kSubRows, it.desc_q_end - row0);
      diag = false;
      qpos0 = 0;
    }
  };

  if (warp == 8) {
    // ======================= TMA producer =======================
    if (n_it > 0) {
      if (lane == 0) {
        const int32_t* page_slot = p.blob + p.off_page_slot;
        const int64_t head_row0 = int64_t(hk) * p.cap;
        // K and V complete on one barrier: post the byte count once, issue both gathers against it
        mbar_expect_tx(&bar.kv_full, uint32_t(kt.rows_loaded) * 512u);
        const int rows_per_box = kt.bs >= 128 ? 128 : kt.bs;
        const int mi = map_index(kt.bs);
        for (int i = 0; i < kt.n_pages; ++i) {
          const int row = int(head_row0 + page_slot[kt.first_page + i] + kt.row_off);
          uint8_t* dk_ = sK + i * rows_per_box * 128;
          uint8_t* dv_ = sV + i * rows_per_box * 128;
          tma_load_2d(dk_, &maps.kv.k[mi], &bar.kv_full, 0, row);
          tma_load_2d(dk_ + kHalfBytes, &maps.kv.k[mi], &bar.kv_full, 64, row);
          tma_load_2d(dv_, &maps.kv.v[mi], &bar.kv_full, 0, row);
          tma_load_2d(dv_ + kHalfBytes, &maps.kv.v[mi], &bar.kv_full, 64, row);
        }
      }
      // The whole warp walks the steps: lane 0 issues the TMA loads of Q and dO, all lanes
      // stage the step's LSE (log2 units) and D rows next to them.  The ring runs ST steps
      // ahead of the consumers, which hides the latency of these plain global loads.
      bool ok = true;
      for (int i = 0; ok && i < n_it; ++i) {
        const int st = i % ST;
        int g, row0, nvq, qpos0; bool diag;
        step(i, g, row0, nvq, diag, qpos0);
        const int h = hk * p.G + g;
        if (i >= ST) ok = mbar_wait(&bar.qd_empty[st], ((i / ST) + 1) & 1, abortp, p.status);
        if (!ok) break;
        if (lane == 0) {
          mbar_expect_tx(&bar.qd_full[st], 2 * kSubBytes);
          uint8_t* dq_ = sQ + st * kSubBytes;
          uint8_t* dg_ = sdO + st * kSubBytes;
          tma_load_2d(dq_, &maps.q, &bar.qd_full[st], h * 128, row0);
          tma_load_2d(dq_ + kSubHalf, &maps.q, &bar.qd_full[st], h * 128 + 64, row0);
          tma_load_2d(dg_, &maps.d_o, &bar.qd_full[st], h * 128, row0);
          tma_load_2d(dg_ + kSubHalf, &maps.d_o, &bar.qd_full[st], h * 128 + 64, row0);
        }
        const float* lse_row = p.lse + int64_t(h) * p.T_q + row0;
        const float* dl_row = p.delta + int64_t(h) * p.T_q + row0;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const int r = lane + 32 * x;
          s_lse[st][r] = r < nvq ? lse_row[r] * kLog2e : CUDART_INF_F;
          s_dl[st][r] = r < nvq ? dl_row[r] : 0.f;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar.qd_full[st]);  // second arrival: LSE / D are in place
      }
    }
  } else if (warp == 9) {
    // ======================= MMA issuer =======================
    if (lane == 0 && n_it > 0) {
      constexpr uint32_t idesc1 = make_idesc(128, kSubRows, 0, 0);  // S^T = K Q^T, dP^T = V dO^T
      constexpr uint32_t idesc2 = make_idesc(128, 128, 0, 1);       // dV += P^T dO, dK += dS^T Q
      // descriptor low words (address >> 4 | LBO field); per K step only a constant is added
      const uint32_t k_lo = desc_lo(smem_u32(sK), 16), v_lo = desc_lo(smem_u32(sV), 16);
      const uint32_t q_lo = desc_lo(smem_u32(sQ), 16), g_lo = desc_lo(smem_u32(sdO), 16);              // K-major view
      const uint32_t q_mn = desc_lo(smem_u32(sQ), kSubHalf), g_mn = desc_lo(smem_u32(sdO), kSubHalf);  // MN-major view
      auto mma1 = [&](int i) {
        const int st = i % ST, b = i & 1;
        const uint32_t qs = q_lo + st * (kSubBytes >> 4), gs = g_lo + st * (kSubBytes >> 4);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t oa = (k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2, ob = (k >> 2) * (kSubHalf >> 4) + (k & 3) * 2;
          mma_ss_lo(tmem + TM_ST + b * 64, k_lo + oa, qs + ob, idesc1, k > 0);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t oa = (k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2, ob = (k >> 2) * (kSubHalf >> 4) + (k & 3) * 2;
          mma_ss_lo(tmem + TM_DPT + b * 64, v_lo + oa, gs + ob, idesc1, k > 0);
        }
        mma_commit(&bar.st_full[b]);
      };
      auto mma2 = [&](int i) {
        const int st = i % ST, b = i & 1;
        const uint32_t qs = q_mn + st * (kSubBytes >> 4), gs = g_mn + st * (kSubBytes >> 4);
        const uint32_t acc0 = i > 0;
        // P^T / dS^T: packed bf16, 16 query rows per 8 columns; rows 0-31 at +0, rows 32-63 at +32
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t a_off = (k >> 1) * 32 + (k & 1) * 8;
          mma_ts_lo(tmem + TM_DV, tmem + TM_ST + b * 64 + a_off, gs + k * 128, idesc2, k > 0 ? 1u : acc0);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t a_off = (k >> 1) * 32 + (k & 1) * 8;
          mma_ts_lo(tmem + TM_DK, tmem + TM_DPT + b * 64 + a_off, qs + k * 128, idesc2, k > 0 ? 1u : acc0);
        }
        mma_commit(&bar.qd_empty[st]);
      };
      bool ok = mbar_wait_relaxed(&bar.kv_full, 0, abortp, p.status) && mbar_wait_relaxed(&bar.qd_full[0], 0, abortp, p.status);
      if (ok) {
        tc_fence_after();
        mma1(0);
      }
      for (int i = 0; ok && i < n_it; ++i) {
        if (i + 1 < n_it) {
          ok = mbar_wait_relaxed(&bar.qd_full[(i + 1) % ST], ((i + 1) / ST) & 1, abortp, p.status);
          if (!ok) break;
          tc_fence_after();
          mma1(i + 1);
        }
        ok = mbar_wait_relaxed(&bar.pd_ready[i & 1], (i >> 1) & 1, abortp, p.status);
        if (!ok) break;
        tc_fence_after();
        mma2(i);
      }
      if (ok) mma_commit(&bar.acc_full);
    }
  } else {
    // ======================= softmax-backward warps (8) =======================
    const int wg = warp >> 2;                            // which 32 query columns of the 64
    const int keyrow = (warp & 3) * 32 + lane;           // key inside the tile = TMEM lane
    const uint32_t t_lane = tmem + (uint32_t((warp & 3) * 32) << 16);
    bool ok = true;
    for (int i = 0; i < n_it; ++i) {
      const int b = i & 1;
      int g, row0, nvq, qpos0; bool diag;
      step(i, g, row0, nvq, diag, qpos0);
      const int st = i % ST;
      // LSE / D of this step were staged by the producer warp together with Q / dO
      ok = mbar_wait(&bar.qd_full[st], (i / ST) & 1, abortp, p.status) &&
           mbar_wait(&bar.st_full[b], (i >> 1) & 1, abortp, p.status);
      if (!ok) break;
      tc_fence_after();
      uint32_t s[32], dp[32], pk[16], dk[16];
      tmem_ld32(t_lane + TM_ST + b * 64 + wg * 32, s);
      tmem_ld32(t_lane + TM_DPT + b * 64 + wg * 32, dp);
      float lse_r[32], dl_r[32];
#pragma unroll
      for (int x = 0; x < 8; ++x) {
        const float4 a = reinterpret_cast<const float4*>(&s_lse[st][wg * 32])[x];
        const float4 d = reinterpret_cast<const float4*>(&s_dl[st][wg * 32])[x];
        lse_r[4 * x] = a.x; lse_r[4 * x + 1] = a.y; lse_r[4 * x + 2] = a.z; lse_r[4 * x + 3] = a.w;
        dl_r[4 * x] = d.x; dl_r[4 * x + 1] = d.y; dl_r[4 * x + 2] = d.z; dl_r[4 * x + 3] = d.w;
      }
      tmem_wait_ld();
      const bool need_mask = diag || nvq < kSubRows;
#pragma unroll
      for (int x = 0; x < 32; x += 2) {
        float p0 = ex2(fmaf(__uint_as_float(s[x]), p.scale_log2, -lse_r[x]));
        float p1 = ex2(fmaf(__uint_as_float(s[x + 1]), p.scale_log2, -lse_r[x + 1]));
        float d0 = p0 * (__uint_as_float(dp[x]) - dl_r[x]);
        float d1 = p1 * (__uint_as_float(dp[x + 1]) - dl_r[x + 1]);
        if (need_mask) {
          const int c0 = wg * 32 + x, c1 = c0 + 1;
          const bool v0 = c0 < nvq && (!diag || qpos0 + c0 >= keyrow);
          const bool v1 = c1 < nvq && (!diag || qpos0 + c1 >= keyrow);
          p0 = v0 ? p0 : 0.f; d0 = v0 ? d0 : 0.f;
          p1 = v1 ? p1 : 0.f; d1 = v1 ? d1 : 0.f;
        }
        pk[x >> 1] = pack_bf16(p0, p1);
        dk[x >> 1] = pack_bf16(d0, d1);
      }
      tmem_st16(t_lane + TM_ST + b * 64 + wg * 32, pk);
      tmem_st16(t_lane + TM_DPT + b * 64 + wg * 32, dk);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bar.pd_ready[b]);
    }
    // ---- epilogue: warps 0-3 take dV, warps 4-7 take dK ----
    if (ok && n_it > 0) ok = mbar_wait(&bar.acc_full, 0, abortp, p.status);
    if (ok) {
      tc_fence_after();
      const uint32_t t_acc = t_lane + (wg == 0 ? TM_DV : TM_DK);
      if (it.slab >= 0) {
        // split item: fp32 partial to its slab, [slab][kv head][dV, dK][128][128]
        float* out = p.slabs + ((int64_t(it.slab) * p.Hkv + hk) * 2 + wg) * (128 * 128) + keyrow * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld32(t_acc + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int x = 0; x < 8; ++x)
            *reinterpret_cast<uint4*>(out + c * 32 + x * 4) = make_uint4(r[4 * x], r[4 * x + 1], r[4 * x + 2], r[4 * x + 3]);
        }
      } else {
        // the item owns the tile: bf16 output, dK scaled, pad slots zero
        const bool in_pages = keyrow < kt.rows_loaded;
        const bool valid = keyrow < kt.n_valid && n_it > 0;
        const int64_t slot = in_pages ? tile_row_slot(kt, p.blob + p.off_page_slot, keyrow) : 0;
        __nv_bfloat16* out = (wg == 0 ? p.dv : p.dk) + (int64_t(hk) * p.cap + slot) * 128;
        const float mul = wg == 0 ? 1.f : p.scale;
        if (keyrow < kt.zero_rows) {  // slots of the page that lie beyond the segment's last tile
          __nv_bfloat16* z = out + int64_t(128) * 128;
#pragma unroll
          for (int x = 0; x < 16; ++x) *reinterpret_cast<uint4*>(z + x * 8) = make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          if (n_it > 0) {
            tmem_ld32(t_acc + c * 32, r);
            tmem_wait_ld();
          }
          if (in_pages) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              uint4 v = make_uint4(0, 0, 0, 0);
              if (valid) {
                v.x = pack_bf16(__uint_as_float(r[8 * x + 0]) * mul, __uint_as_float(r[8 * x + 1]) * mul);
                v.y = pack_bf16(__uint_as_float(r[8 * x + 2]) * mul, __uint_as_float(r[8 * x + 3]) * mul);
                v.z = pack_bf16(__uint_as_float(r[8 * x + 4]) * mul, __uint_as_float(r[8 * x + 5]) * mul);
                v.w = pack_bf16(__uint_as_float(r[8 * x + 6]) * mul, __uint_as_float(r[8 * x + 7]) * mul);
              }
              *reinterpret_cast<uint4*>(out + c * 32 + x * 8) = v;
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// Adds the fp32 partials of a split KV tile in part order and writes the bf16 result.
// One block per (split tile, KV head); thread t owns row t / 2, columns (t % 2) * 64 .. + 64.
__global__ void __launch_bounds__(256)
reduce_kernel(const Params p) {
  const KvSplit sp = reinterpret_cast<const KvSplit*>(p.blob + p.off_split)[blockIdx.x];
  const KvTile kt = reinterpret_cast<const KvTile*>(p.blob + p.off_kvt)[sp.kvt];
  const int hk = blockIdx.y, row = threadIdx.x >> 1, c0 = (threadIdx.x & 1) * 64;
  if (row >= kt.rows_loaded) return;
  const int64_t slot = tile_row_slot(kt, p.blob + p.off_page_slot, row);
  const bool valid = row < kt.n_valid;
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    float acc[64];
#pragma unroll
    for (int x = 0; x < 64; ++x) acc[x] = 0.f;
    if (valid) {
      for (int part = 0; part < sp.n_parts; ++part) {
        const float* src =
            p.slabs + ((int64_t(sp.slab0 + part) * p.Hkv + hk) * 2 + which) * (128 * 128) + row * 128 + c0;
#pragma unroll
        for (int x = 0; x < 16; ++x) {
          const float4 v = reinterpret_cast<const float4*>(src)[x];
          acc[4 * x] += v.x; acc[4 * x + 1] += v.y; acc[4 * x + 2] += v.z; acc[4 * x + 3] += v.w;
        }
      }
    }
    const float mul = which == 0 ? 1.f : p.scale;
    __nv_bfloat16* out = (which == 0 ? p.dv : p.dk) + (int64_t(hk) * p.cap + slot) * 128 + c0;
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      uint4 v;
      v.x = pack_bf16(acc[8 * x + 0] * mul, acc[8 * x + 1] * mul);
      v.y = pack_bf16(acc[8 * x + 2] * mul, acc[8 * x + 3] * mul);
      v.z = pack_bf16(acc[8 * x + 4] * mul, acc[8 * x + 5] * mul);
      v.w = pack_bf16(acc[8 * x + 6] * mul, acc[8 * x + 7] * mul);
      *reinterpret_cast<uint4*>(out + 8 * x) = v;
    }
    if (row < kt.zero_rows) {
      __nv_bfloat16* z = out + int64_t(128) * 128;
#pragma unroll
      for (int x = 0; x < 8; ++x) *reinterpret_cast<uint4*>(z + 8 * x) = make_uint4(0, 0, 0, 0);
    }
  }
}

}  // namespace

psrl_status_t dkv_bf16(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const DeviceHeader& H = P.hdr;
  const int64_t cap = a.pool_capacity;
  auto fail = [](cudaError_t e) { set_last_cuda_error(e); return PSRL_ERR_CUDA; };
  Maps m;
  bool ok = make_pool_maps(&m.kv, a.k_pool, a.v_pool, P.Hkv, cap);
  if (ok && P.T_q > 0) {
    ok = make_map_bf16_2d(&m.q, a.q, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, kSubRows) &&
         make_map_bf16_2d(&m.d_o, a.d_o, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, kSubRows);
  }
  if (!ok) return PSRL_ERR_CUDA;
  const size_t smem = size_t(2) * kTileBytes + size_t(2 * ST) * kSubBytes + 1024;
  static bool attr_set = false;
  cudaError_t e;
  if (!attr_set) {
    e = cudaFuncSetAttribute(dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return fail(e);
    attr_set = true;
  }
  Params p{};
  p.blob = P.dev;
  p.off_kvi = H.off_kvi; p.off_kvt = H.off_kvt; p.off_page_slot = H.off_page_slot; p.off_split = H.off_split;
  p.Hq = P.Hq; p.Hkv = P.Hkv; p.G = P.Hq / P.Hkv; p.T_q = P.T_q;
  p.cap = cap; p.scale = a.scale; p.scale_log2 = a.scale * kLog2e;
  p.lse = a.lse_in; p.delta = a.delta; p.slabs = a.slabs;
  p.dk = static_cast<__nv_bfloat16*>(a.dk_pool); p.dv = static_cast<__nv_bfloat16*>(a.dv_pool);
  p.status = a.status;
  const int64_t grid = int64_t(P.kv_items.size()) * P.Hkv;
  if (grid > INT32_MAX) return PSRL_ERR_SHAPE;
  dkv_kernel<<<unsigned(grid), kThreads, smem, a.stream>>>(m, p);
  if ((e = cudaGetLastError()) != cudaSuccess) return fail(e);
  if (!P.kv_splits.empty()) {
    dim3 rg(unsigned(P.kv_splits.size()), unsigned(P.Hkv));
    reduce_kernel<<<rg, 256, 0, a.stream>>>(p);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail(e);
  }
  return PSRL_OK;
}

}  // namespace psrl

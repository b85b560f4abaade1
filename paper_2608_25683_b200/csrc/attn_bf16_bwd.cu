// bf16 tree attention backward on the 5th-generation tensor cores.
//
// Three kernels, all deterministic (every output element has one owner that
// sums its contributions in a fixed order; no atomics):
//   delta_kernel  D_i = dO_i . O_i                                (HBM-bound pre-pass)
//   dq_kernel     query-stationary: per KV tile S = Q K^T, dP = dO V^T,
//                 dS = P o (dP - D), dQ += dS K                   (3 contractions)
//   dkv_kernel    key-stationary: per query tile S^T = K Q^T, dP^T = V dO^T,
//                 dV += P^T dO, dK += dS^T Q                      (4 contractions)
// The key-stationary kernel is where the shared prefix pays off in backward
// (paper Sec. 6: consumer adjoints are accumulated on the shared prefix): a KV
// tile of segment a is visited by the later rows of a itself and by ALL rows of
// ALL descendant segments, which are one contiguous row range in the canonical
// (DFS) layout, and by the Hq/Hkv query heads of its KV head; the sum runs in
// that fixed order inside one CTA, with dK/dV accumulating in tensor memory.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "attn_bf16_common.cuh"
#include "kernels.h"
#include "tma.h"

namespace psrl {
namespace {
using namespace sm100;

// ============================================================================ delta
__global__ void __launch_bounds__(256)
delta_kernel(int T_q, int Hq, const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
             float* __restrict__ delta) {
  const int lane = threadIdx.x & 31;
  const int64_t unit = int64_t(blockIdx.x) * 8 + (threadIdx.x >> 5);  // = h * T_q + r
  if (unit >= int64_t(T_q) * Hq) return;
  const int h = int(unit / T_q), r = int(unit % T_q);
  const int64_t off = (int64_t(r) * Hq + h) * 128 + lane * 4;
  const uint2 a = *reinterpret_cast<const uint2*>(o + off);
  const uint2 b = *reinterpret_cast<const uint2*>(d_o + off);
  const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.x));
  const float2 a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.y));
  const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.x));
  const float2 b1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.y));
  float s = a0.x * b0.x + a0.y * b0.y + a1.x * b1.x + a1.y * b1.y;
#pragma unroll
  for (int o2 = 16; o2 > 0; o2 >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o2);
  if (lane == 0) delta[unit] = s;
}

// ============================================================================ dQ
namespace dq {
constexpr int NQ = 2;
constexpr int KS = 2;  // K ring; V has a single stage
constexpr int kThreads = (4 * NQ + 2) * 32;

struct Maps {
  CUtensorMap q, d_o;
  PoolMaps kv;
};
struct Params {
  const int32_t* blob;
  int32_t off_qt, off_kvt, off_path_tiles, off_path_nvalid, off_page_slot;
  int32_t Hq, Hkv, G, T_q, pairs_per_group;
  int64_t cap;
  float scale, scale_log2;
  const float* lse;
  const float* delta;
  __nv_bfloat16* d_q;
  int* status;
};
struct __align__(8) Barriers {
  uint64_t qdo_full, k_full[KS], k_empty[KS], v_full, v_empty;
  uint64_t sd_full[NQ], ds_ready[NQ], dq_full[NQ], x_free[NQ];
};

__global__ void __launch_bounds__(kThreads, 1)
dq_kernel(const __grid_constant__ Maps maps, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                      // NQ tiles
  uint8_t* sdO = sQ + NQ * kTileBytes;     // NQ tiles
  uint8_t* sK = sdO + NQ * kTileBytes;     // KS tiles
  uint8_t* sV = sK + KS * kTileBytes;      // 1 tile
  __shared__ Barriers bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int units = p.Hkv * p.pairs_per_group;
  const int item = blockIdx.x / units, u = blockIdx.x % units;
  const int hk = u / p.pairs_per_group, pair = u % p.pairs_per_group;
  const int h0 = hk * p.G + pair * NQ;
  const int nq = min(NQ, p.G - pair * NQ);
  const QTile qt = reinterpret_cast<const QTile*>(p.blob + p.off_qt)[item];
  const int32_t* path_tiles = p.blob + p.off_path_tiles + qt.pt_begin;
  const int32_t* path_nvalid = p.blob + p.off_path_nvalid + qt.pt_begin;
  const int n_tiles = qt.n_kv_tiles;

  if (tid == 0) {
    s_abort = 0;
    mbar_init(&bar.qdo_full, 1);
    for (int i = 0; i < KS; ++i) { mbar_init(&bar.k_full[i], 1); mbar_init(&bar.k_empty[i], 1); }
    mbar_init(&bar.v_full, 1); mbar_init(&bar.v_empty, 1);
    for (int i = 0; i < NQ; ++i) {
      mbar_init(&bar.sd_full[i], 1); mbar_init(&bar.ds_ready[i], 128);
      mbar_init(&bar.dq_full[i], 1); mbar_init(&bar.x_free[i], 128);
    }
    fence_mbar_init();
  }
  if (warp == 4 * NQ + 1) { tmem_alloc(&s_tmem, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;

  if (warp == 4 * NQ) {
    // ======================= TMA producer =======================
    if (lane == 0) {
      mbar_expect_tx(&bar.qdo_full, uint32_t(nq) * 2 * kTileBytes);
      for (int q = 0; q < nq; ++q) {
        load_row_tile(sQ + q * kTileBytes, &maps.q, &bar.qdo_full, h0 + q, qt.q_row0);
        load_row_tile(sdO + q * kTileBytes, &maps.d_o, &bar.qdo_full, h0 + q, qt.q_row0);
      }
      const KvTile* kvt = reinterpret_cast<const KvTile*>(p.blob + p.off_kvt);
      const int32_t* page_slot = p.blob + p.off_page_slot;
      const int64_t head_row0 = int64_t(hk) * p.cap;
      for (int j = 0; j < n_tiles; ++j) {
        const KvTile kt = kvt[path_tiles[j]];
        const int ks = j % KS;
        if (j >= KS && !mbar_wait(&bar.k_empty[ks], ((j / KS) + 1) & 1, abortp, p.status)) break;
        load_kv_tile(sK + ks * kTileBytes, maps.kv.k, &bar.k_full[ks], kt, page_slot, head_row0);
        if (j >= 1 && !mbar_wait(&bar.v_empty, (j + 1) & 1, abortp, p.status)) break;
        load_kv_tile(sV, maps.kv.v, &bar.v_full, kt, page_slot, head_row0);
      }
    }
  } else if (warp == 4 * NQ + 1) {
    // ======================= MMA issuer =======================
    if (lane == 0) {
      constexpr uint32_t idesc_kk = make_idesc(128, 128, 0, 0);  // S = Q K^T, dP = dO V^T
      constexpr uint32_t idesc_mn = make_idesc(128, 128, 0, 1);  // dQ = dS K, K is MN-major
      auto issue_s_dp = [&](int q, int ks) {
        const uint32_t q0 = smem_u32(sQ + q * kTileBytes), k0 = smem_u32(sK + ks * kTileBytes);
        const uint32_t g0 = smem_u32(sdO + q * kTileBytes), v0 = smem_u32(sV);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
          mma_ss(tmem + q * 256, make_desc(q0 + off, 16, 1024), make_desc(k0 + off, 16, 1024), idesc_kk, k > 0);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
          mma_ss(tmem + q * 256 + 128, make_desc(g0 + off, 16, 1024), make_desc(v0 + off, 16, 1024), idesc_kk, k > 0);
        }
      };
      auto issue_dq = [&](int q, int ks) {
        const uint32_t b0 = smem_u32(sK + ks * kTileBytes);
#pragma unroll
        for (int k = 0; k < 8; ++k)
          mma_ts(tmem + q * 256, tmem + q * 256 + 128 + k * 8, make_desc(b0 + k * 2048, kHalfBytes, 1024), idesc_mn,
                 k > 0);
      };
      bool ok = mbar_wait(&bar.qdo_full, 0, abortp, p.status) && mbar_wait(&bar.k_full[0], 0, abortp, p.status) &&
                mbar_wait(&bar.v_full, 0, abortp, p.status);
      if (ok) {
        tc_fence_after();
        for (int q = 0; q < nq; ++q) { issue_s_dp(q, 0); mma_commit(&bar.sd_full[q]); }
        mma_commit(&bar.v_empty);
      }
      for (int j = 0; ok && j < n_tiles; ++j) {
        const int ks = j % KS;
        for (int q = 0; ok && q < nq; ++q) {
          ok = mbar_wait(&bar.ds_ready[q], j & 1, abortp, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_dq(q, ks);
          mma_commit(&bar.dq_full[q]);
          if (q == nq - 1) mma_commit(&bar.k_empty[ks]);
        }
        if (ok && j + 1 < n_tiles) {
          const int ks1 = (j + 1) % KS;
          for (int q = 0; ok && q < nq; ++q) {
            ok = mbar_wait(&bar.x_free[q], j & 1, abortp, p.status);
            if (ok && q == 0)
              ok = mbar_wait(&bar.k_full[ks1], ((j + 1) / KS) & 1, abortp, p.status) &&
                   mbar_wait(&bar.v_full, (j + 1) & 1, abortp, p.status);
            if (!ok) break;
            tc_fence_after();
            issue_s_dp(q, ks1);
            mma_commit(&bar.sd_full[q]);
            if (q == nq - 1) mma_commit(&bar.v_empty);
          }
        }
      }
    }
  } else if (warp < 4 * nq) {
    // ======================= softmax-backward warpgroups =======================
    const int q = warp >> 2;
    const int row = tid & 127;
    const int h = h0 + q;
    const uint32_t t_lane = tmem + (uint32_t((warp & 3) * 32) << 16) + q * 256;
    const bool row_ok = row < qt.n_rows;
    const float lse2 = row_ok ? p.lse[int64_t(h) * p.T_q + qt.q_row0 + row] * kLog2e : 0.f;
    const float dl = row_ok ? p.delta[int64_t(h) * p.T_q + qt.q_row0 + row] : 0.f;
    float acc[128];
#pragma unroll
    for (int i = 0; i < 128; ++i) acc[i] = 0.f;
    bool ok = true;
    int nv_next = path_nvalid[0];
    for (int j = 0; j < n_tiles; ++j) {
      const int n_valid = nv_next;
      if (j + 1 < n_tiles) nv_next = path_nvalid[j + 1];
      const bool diag = (j == n_tiles - 1);
      const int limit = diag ? min(row + 1, n_valid) : n_valid;
      const bool need_mask = diag || n_valid < 128;
      ok = mbar_wait(&bar.sd_full[q], j & 1, abortp, p.status);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t s[32], dp[32], pk[16];
        tmem_ld32(t_lane + c * 32, s);
        tmem_ld32(t_lane + 128 + c * 32, dp);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float p0 = ex2(fmaf(__uint_as_float(s[i]), p.scale_log2, -lse2));
          const float p1 = ex2(fmaf(__uint_as_float(s[i + 1]), p.scale_log2, -lse2));
          float d0 = p0 * (__uint_as_float(dp[i]) - dl);
          float d1 = p1 * (__uint_as_float(dp[i + 1]) - dl);
          if (need_mask) {
            d0 = (c * 32 + i < limit) ? d0 : 0.f;
            d1 = (c * 32 + i + 1 < limit) ? d1 : 0.f;
          }
          pk[i >> 1] = pack_bf16(d0, d1);
        }
        tmem_st16(t_lane + 128 + c * 16, pk);
      }
      // K rows at or beyond n_valid must be zero before dS K (dS is zero there, K may hold anything)
      if (q == 0 && n_valid < 128) {
        ok = mbar_wait(&bar.k_full[j % KS], (j / KS) & 1, abortp, p.status);
        if (!ok) break;
        if (row >= n_valid) zero_tile_row(sK + (j % KS) * kTileBytes, row);
        fence_proxy_async();
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bar.ds_ready[q]);
      // ---- this tile's dQ contribution ----
      ok = mbar_wait(&bar.dq_full[q], j & 1, abortp, p.status);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(t_lane + c * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[c * 32 + i] += __uint_as_float(r[i]);
      }
      tc_fence_before();
      mbar_arrive(&bar.x_free[q]);
    }
    if (ok && row_ok) {
      __nv_bfloat16* drow = p.d_q + (int64_t(qt.q_row0 + row) * p.Hq + h) * 128;
#pragma unroll
      for (int x = 0; x < 16; ++x) {
        uint4 v;
        v.x = pack_bf16(acc[8 * x + 0] * p.scale, acc[8 * x + 1] * p.scale);
        v.y = pack_bf16(acc[8 * x + 2] * p.scale, acc[8 * x + 3] * p.scale);
        v.z = pack_bf16(acc[8 * x + 4] * p.scale, acc[8 * x + 5] * p.scale);
        v.w = pack_bf16(acc[8 * x + 6] * p.scale, acc[8 * x + 7] * p.scale);
        *reinterpret_cast<uint4*>(drow + 8 * x) = v;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4 * NQ + 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}
}  // namespace dq

// ============================================================================ dK / dV
namespace dkv {
constexpr int ST = 2;                         // (Q, dO) ring depth
constexpr int kThreads = (8 + 2) * 32;        // 8 softmax warps + producer + MMA
constexpr uint32_t TM_ST = 0, TM_DPT = 128, TM_DV = 256, TM_DK = 384;

struct Maps {
  CUtensorMap q, d_o;
  PoolMaps kv;
};
struct Params {
  const int32_t* blob;
  int32_t off_kvi, off_kvt, off_page_slot;
  int32_t Hq, Hkv, G, T_q;
  int64_t cap;
  float scale, scale_log2;
  const float* lse;
  const float* delta;
  __nv_bfloat16 *dk, *dv;
  int* status;
};
struct __align__(8) Barriers {
  uint64_t kv_full, qd_full[ST], qd_empty[ST], st_full, pd_ready, acc_full, lse_ready;
};

__global__ void __launch_bounds__(kThreads, 1)
dkv_kernel(const __grid_constant__ Maps maps, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = smem;
  uint8_t* sV = sK + kTileBytes;
  uint8_t* sQ = sV + kTileBytes;             // ST tiles
  uint8_t* sdO = sQ + ST * kTileBytes;       // ST tiles
  __shared__ Barriers bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ float s_lse[2][128], s_dl[2][128];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int item = blockIdx.x / p.Hkv, hk = blockIdx.x % p.Hkv;
  const KvItem it = reinterpret_cast<const KvItem*>(p.blob + p.off_kvi)[item];
  const KvTile kt = reinterpret_cast<const KvTile*>(p.blob + p.off_kvt)[it.kvt];
  const int n_own = it.own_q_row0 >= 0 ? (it.own_q_end - it.own_q_row0 + 127) / 128 : 0;
  const int n_desc = (it.desc_q_end - it.desc_q_begin + 127) / 128;
  const int n_it = (n_own + n_desc) * p.G;

  if (tid == 0) {
    s_abort = 0;
    mbar_init(&bar.kv_full, 1);
    for (int i = 0; i < ST; ++i) { mbar_init(&bar.qd_full[i], 1); mbar_init(&bar.qd_empty[i], 1); }
    mbar_init(&bar.st_full, 1); mbar_init(&bar.pd_ready, 256); mbar_init(&bar.acc_full, 1);
    mbar_init(&bar.lse_ready, 256);
    fence_mbar_init();
  }
  if (warp == 9) { tmem_alloc(&s_tmem, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;

  // query tile t of this item: first row, valid rows, whether it is the diagonal tile
  auto q_tile = [&](int t, int& row0, int& nvq, bool& diag) {
    if (t < n_own) {
      row0 = it.own_q_row0 + t * 128;
      nvq = min(128, it.own_q_end - row0);
      diag = (t == 0);
    } else {
      row0 = it.desc_q_begin + (t - n_own) * 128;
      nvq = min(128, it.desc_q_end - row0);
      diag = false;
    }
  };

  if (warp == 8) {
    // ======================= TMA producer =======================
    if (lane == 0) {
      const int32_t* page_slot = p.blob + p.off_page_slot;
      const int64_t head_row0 = int64_t(hk) * p.cap;
      // K and V complete on the same barrier: two expect_tx arrivals would over-count, so
      // post the byte count once and issue both gathers against it
      if (n_it > 0) {
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
      for (int i = 0; i < n_it; ++i) {
        const int st = i % ST, t = i / p.G, g = i % p.G;
        int row0, nvq; bool diag;
        q_tile(t, row0, nvq, diag);
        if (i >= ST && !mbar_wait(&bar.qd_empty[st], ((i / ST) + 1) & 1, abortp, p.status)) break;
        mbar_expect_tx(&bar.qd_full[st], 2 * kTileBytes);
        load_row_tile(sQ + st * kTileBytes, &maps.q, &bar.qd_full[st], hk * p.G + g, row0);
        load_row_tile(sdO + st * kTileBytes, &maps.d_o, &bar.qd_full[st], hk * p.G + g, row0);
      }
    }
  } else if (warp == 9) {
    // ======================= MMA issuer =======================
    if (lane == 0) {
      constexpr uint32_t idesc_kk = make_idesc(128, 128, 0, 0);  // S^T = K Q^T, dP^T = V dO^T
      constexpr uint32_t idesc_mn = make_idesc(128, 128, 0, 1);  // dV += P^T dO, dK += dS^T Q
      bool ok = n_it == 0 || mbar_wait(&bar.kv_full, 0, abortp, p.status);
      const uint32_t k0 = smem_u32(sK), v0 = smem_u32(sV);
      for (int i = 0; ok && i < n_it; ++i) {
        const int st = i % ST;
        ok = mbar_wait(&bar.qd_full[st], (i / ST) & 1, abortp, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t q0 = smem_u32(sQ + st * kTileBytes), g0 = smem_u32(sdO + st * kTileBytes);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
          mma_ss(tmem + TM_ST, make_desc(k0 + off, 16, 1024), make_desc(q0 + off, 16, 1024), idesc_kk, k > 0);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
          mma_ss(tmem + TM_DPT, make_desc(v0 + off, 16, 1024), make_desc(g0 + off, 16, 1024), idesc_kk, k > 0);
        }
        mma_commit(&bar.st_full);
        ok = mbar_wait(&bar.pd_ready, i & 1, abortp, p.status);
        if (!ok) break;
        tc_fence_after();
        // P^T / dS^T sit as packed bf16 in the first 32 columns of each 64-column half
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t a_off = (k >> 2) * 64 + (k & 3) * 8;
          mma_ts(tmem + TM_DV, tmem + TM_ST + a_off, make_desc(g0 + k * 2048, kHalfBytes, 1024), idesc_mn,
                 (i > 0 || k > 0));
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t a_off = (k >> 2) * 64 + (k & 3) * 8;
          mma_ts(tmem + TM_DK, tmem + TM_DPT + a_off, make_desc(q0 + k * 2048, kHalfBytes, 1024), idesc_mn,
                 (i > 0 || k > 0));
        }
        mma_commit(&bar.qd_empty[st]);
      }
      if (ok) mma_commit(&bar.acc_full);
    }
  } else {
    // ======================= softmax-backward warps (8) =======================
    const int half = warp >> 2;                          // which 64 query columns
    const int keyrow = (warp & 3) * 32 + lane;           // key inside the tile = TMEM lane
    const uint32_t t_lane = tmem + (uint32_t((warp & 3) * 32) << 16);
    bool ok = true;
    for (int i = 0; i < n_it; ++i) {
      const int t = i / p.G, g = i % p.G, h = hk * p.G + g, b = i & 1;
      int row0, nvq; bool diag;
      q_tile(t, row0, nvq, diag);
      // stage LSE (log2 units) and D of the tile's query rows
      if (tid < 128) s_lse[b][tid] = tid < nvq ? p.lse[int64_t(h) * p.T_q + row0 + tid] * kLog2e : CUDART_INF_F;
      else s_dl[b][tid - 128] = (tid - 128) < nvq ? p.delta[int64_t(h) * p.T_q + row0 + tid - 128] : 0.f;
      mbar_arrive(&bar.lse_ready);
      ok = mbar_wait(&bar.lse_ready, i & 1, abortp, p.status) && mbar_wait(&bar.st_full, i & 1, abortp, p.status);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int col0 = half * 64 + c * 32;
        uint32_t s[32], dp[32], pk[16], dk[16];
        tmem_ld32(t_lane + TM_ST + col0, s);
        tmem_ld32(t_lane + TM_DPT + col0, dp);
        tmem_wait_ld();
#pragma unroll
        for (int x = 0; x < 32; x += 2) {
          const int q0i = col0 + x, q1i = col0 + x + 1;
          const float p0 = ex2(fmaf(__uint_as_float(s[x]), p.scale_log2, -s_lse[b][q0i]));
          const float p1 = ex2(fmaf(__uint_as_float(s[x + 1]), p.scale_log2, -s_lse[b][q1i]));
          const bool v0 = q0i < nvq && (!diag || q0i >= keyrow);
          const bool v1 = q1i < nvq && (!diag || q1i >= keyrow);
          const float pp0 = v0 ? p0 : 0.f, pp1 = v1 ? p1 : 0.f;
          const float d0 = v0 ? p0 * (__uint_as_float(dp[x]) - s_dl[b][q0i]) : 0.f;
          const float d1 = v1 ? p1 * (__uint_as_float(dp[x + 1]) - s_dl[b][q1i]) : 0.f;
          pk[x >> 1] = pack_bf16(pp0, pp1);
          dk[x >> 1] = pack_bf16(d0, d1);
        }
        tmem_st16(t_lane + TM_ST + half * 64 + c * 16, pk);
        tmem_st16(t_lane + TM_DPT + half * 64 + c * 16, dk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bar.pd_ready);
    }
    // ---- epilogue: warps 0-3 write dV, warps 4-7 write dK (scaled); pads are zeros ----
    if (ok && n_it > 0) ok = mbar_wait(&bar.acc_full, 0, abortp, p.status);
    if (ok) {
      tc_fence_after();
      const int rows_per_box = kt.bs >= 128 ? 128 : kt.bs;
      const bool in_pages = keyrow < kt.rows_loaded;
      const bool valid = keyrow < kt.n_valid && n_it > 0;
      int64_t slot = 0;
      if (in_pages)
        slot = (p.blob + p.off_page_slot)[kt.first_page + keyrow / rows_per_box] + kt.row_off + keyrow % rows_per_box;
      __nv_bfloat16* out = (half == 0 ? p.dv : p.dk) + (int64_t(hk) * p.cap + slot) * 128;
      const float mul = half == 0 ? 1.f : p.scale;
      if (keyrow < kt.zero_rows) {  // slots of the page that lie beyond the segment's last tile
        __nv_bfloat16* z = out + int64_t(128) * 128;
#pragma unroll
        for (int x = 0; x < 16; ++x) *reinterpret_cast<uint4*>(z + x * 8) = make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        if (n_it > 0) {
          tmem_ld32(t_lane + (half == 0 ? TM_DV : TM_DK) + c * 32, r);
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
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}
}  // namespace dkv

cudaError_t set_smem(const void* fn, size_t bytes) {
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes));
}

}  // namespace

psrl_status_t bwd_bf16(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const DeviceHeader& H = P.hdr;
  const int64_t cap = a.pool_capacity;
  if (int64_t(P.Hkv) * cap > INT32_MAX || int64_t(P.Hq) * 128 > INT32_MAX) return PSRL_ERR_SHAPE;
  const int G = P.Hq / P.Hkv;
  auto fail = [](cudaError_t e) { set_last_cuda_error(e); return PSRL_ERR_CUDA; };
  cudaError_t e;

  dq::Maps qm;
  bool ok = true;
  if (P.T_q > 0) {
    ok = make_map_bf16_2d(&qm.q, a.q, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, 128) &&
         make_map_bf16_2d(&qm.d_o, a.d_o, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, 128);
  }
  ok = ok && make_pool_maps(&qm.kv, a.k_pool, a.v_pool, P.Hkv, cap);
  if (!ok) return PSRL_ERR_CUDA;

  static bool attr_set = false;
  const size_t smem_dq = size_t(2 * dq::NQ + dq::KS + 1) * kTileBytes + 1024;
  const size_t smem_dkv = size_t(2 + 2 * dkv::ST) * kTileBytes + 1024;
  if (!attr_set) {
    if ((e = set_smem(reinterpret_cast<const void*>(dq::dq_kernel), smem_dq)) != cudaSuccess) return fail(e);
    if ((e = set_smem(reinterpret_cast<const void*>(dkv::dkv_kernel), smem_dkv)) != cudaSuccess) return fail(e);
    attr_set = true;
  }

  if (P.T_q > 0 && (g_bwd_phase_mask & 1)) {
    // ---- D = rowsum(dO o O) ----
    const int64_t units = int64_t(P.T_q) * P.Hq;
    delta_kernel<<<unsigned((units + 7) / 8), 256, 0, a.stream>>>(
        P.T_q, P.Hq, static_cast<const __nv_bfloat16*>(a.o), static_cast<const __nv_bfloat16*>(a.d_o), a.delta);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail(e);
  }
  if (P.T_q > 0 && (g_bwd_phase_mask & 2)) {
    // ---- dQ ----
    dq::Params p{};
    p.blob = P.dev;
    p.off_qt = H.off_qt; p.off_kvt = H.off_kvt; p.off_path_tiles = H.off_path_tiles;
    p.off_path_nvalid = H.off_path_nvalid; p.off_page_slot = H.off_page_slot;
    p.Hq = P.Hq; p.Hkv = P.Hkv; p.G = G; p.T_q = P.T_q;
    p.pairs_per_group = (G + dq::NQ - 1) / dq::NQ;
    p.cap = cap; p.scale = a.scale; p.scale_log2 = a.scale * kLog2e;
    p.lse = a.lse_in; p.delta = a.delta; p.d_q = static_cast<__nv_bfloat16*>(a.d_q); p.status = a.status;
    const int64_t grid = int64_t(P.q_tiles.size()) * P.Hkv * p.pairs_per_group;
    if (grid > INT32_MAX) return PSRL_ERR_SHAPE;
    if (grid > 0) {
      dq::dq_kernel<<<unsigned(grid), dq::kThreads, smem_dq, a.stream>>>(qm, p);
      if ((e = cudaGetLastError()) != cudaSuccess) return fail(e);
    }
  }
  if (g_bwd_phase_mask & 4) {
    // ---- dK, dV ----
    dkv::Maps km;
    if (P.T_q > 0) { km.q = qm.q; km.d_o = qm.d_o; }
    km.kv = qm.kv;
    dkv::Params p{};
    p.blob = P.dev;
    p.off_kvi = H.off_kvi; p.off_kvt = H.off_kvt; p.off_page_slot = H.off_page_slot;
    p.Hq = P.Hq; p.Hkv = P.Hkv; p.G = G; p.T_q = P.T_q;
    p.cap = cap; p.scale = a.scale; p.scale_log2 = a.scale * kLog2e;
    p.lse = a.lse_in; p.delta = a.delta;
    p.dk = static_cast<__nv_bfloat16*>(a.dk_pool); p.dv = static_cast<__nv_bfloat16*>(a.dv_pool);
    p.status = a.status;
    const int64_t grid = int64_t(P.kv_items.size()) * P.Hkv;
    if (grid > INT32_MAX) return PSRL_ERR_SHAPE;
    dkv::dkv_kernel<<<unsigned(grid), dkv::kThreads, smem_dkv, a.stream>>>(km, p);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail(e);
  }
  return PSRL_OK;
}

}  // namespace psrl

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
    // All 32 lanes walk the loop and wait on the barriers (warp-uniform control flow and
    // address arithmetic); only the tcgen05 instructions are issued, by lane 0.
    {
      constexpr uint32_t idesc_kk = make_idesc(128, 128, 0, 0);  // S = Q K^T, dP = dO V^T
      constexpr uint32_t idesc_mn = make_idesc(128, 128, 0, 1);  // dQ = dS K, K is MN-major
      // descriptor low words (address >> 4 | LBO field); per K step only a constant is added
      const uint32_t q_lo = desc_lo(smem_u32(sQ), 16), g_lo = desc_lo(smem_u32(sdO), 16);
      const uint32_t k_lo = desc_lo(smem_u32(sK), 16), v_lo = desc_lo(smem_u32(sV), 16);
      const uint32_t k_mn = desc_lo(smem_u32(sK), kHalfBytes);
      auto issue_s_dp = [&](int q, int ks) {
        const uint32_t q0 = q_lo + q * (kTileBytes >> 4), k0 = k_lo + ks * (kTileBytes >> 4);
        const uint32_t g0 = g_lo + q * (kTileBytes >> 4);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t off = (k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2;
            mma_ss_lo(tmem + q * 256, q0 + off, k0 + off, idesc_kk, k > 0);
          }
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t off = (k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2;
            mma_ss_lo(tmem + q * 256 + 128, g0 + off, v_lo + off, idesc_kk, k > 0);
          }
        }
      };
      auto issue_dq = [&](int q, int ks) {
        const uint32_t b0 = k_mn + ks * (kTileBytes >> 4);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ts_lo(tmem + q * 256, tmem + q * 256 + 128 + k * 8, b0 + k * 128, idesc_mn, k > 0);
        }
      };
      auto commit = [&](uint64_t* b) { if (elect_one()) mma_commit(b); };
      auto wait = [&](uint64_t* b, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait_relaxed(b, parity, abortp, p.status));
      };
      bool ok = wait(&bar.qdo_full, 0) && wait(&bar.k_full[0], 0) &&
                wait(&bar.v_full, 0);
      if (ok) {
        tc_fence_after();
        for (int q = 0; q < nq; ++q) { issue_s_dp(q, 0); commit(&bar.sd_full[q]); }
        commit(&bar.v_empty);
      }
      for (int j = 0; ok && j < n_tiles; ++j) {
        const int ks = j % KS;
        for (int q = 0; ok && q < nq; ++q) {
          ok = wait(&bar.ds_ready[q], j & 1);
          if (!ok) break;
          tc_fence_after();
          issue_dq(q, ks);
          commit(&bar.dq_full[q]);
          if (q == nq - 1) commit(&bar.k_empty[ks]);
        }
        if (ok && j + 1 < n_tiles) {
          const int ks1 = (j + 1) % KS;
          for (int q = 0; ok && q < nq; ++q) {
            ok = wait(&bar.x_free[q], j & 1);
            if (ok && q == 0)
              ok = mbar_wait_relaxed(&bar.k_full[ks1], ((j + 1) / KS) & 1, abortp, p.status) &&
                   wait(&bar.v_full, (j + 1) & 1);
            if (!ok) break;
            tc_fence_after();
            issue_s_dp(q, ks1);
            commit(&bar.sd_full[q]);
            if (q == nq - 1) commit(&bar.v_empty);
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
  if (!attr_set) {
    if ((e = set_smem(reinterpret_cast<const void*>(dq::dq_kernel), smem_dq)) != cudaSuccess) return fail(e);
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
    // ---- dK, dV (attn_bf16_dkv.cu) ----
    const psrl_status_t st = dkv_bf16(a);
    if (st != PSRL_OK) return st;
  }
  return PSRL_OK;
}

}  // namespace psrl

// bf16 dQ kernel (query-stationary).
//
// One CTA = one work item (up to 128 query rows and a list of KV tiles, see
// plan.h: the rows of one segment with the tiles of its ancestors and its own
// tiles up to the diagonal, or packed rows under a cascaded prefix) x one query
// head.  Per tile it runs three contractions (M = 128 rows, N = 128, K = 128):
//   S  = Q K^T      -> warps: P = exp2(S c - LSE), kept in registers
//   dP = dO V^T     -> warps: dS = P o (dP - D), written over dP as bf16
//   dQ += dS K         (A = dS from tensor memory, K MN-major in smem)
// dQ accumulates in tensor memory over the whole path, so every dQ row is
// summed in path order by one CTA (bitwise reproducible).
//
// The tensor cores run one step ahead of the warps: S may be overwritten as
// soon as the warps have READ it into registers (P is never stored), so S(j+1)
// is issued while step j is still being computed; dP / dS has two buffers, so
// dP(j+1) follows right behind S(j+1).  The warps therefore find both inputs of
// a step ready, fetch them in one tensor-memory round trip and compute P and dS
// element by element in one pass.
//
// Warp roles: warps 0-3 softmax-backward (one query row per thread), warp 4 TMA
// producer, warp 5 MMA issuer + TMEM owner.
// Tensor memory: S at 0, dP / dS at 128 and 256 (alternating), dQ at 384.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "attn_bf16_common.cuh"
#include "kernels.h"
#include "tma.h"

namespace psrl {
namespace {
using namespace sm100;

constexpr int KS = 3, VS = 2;                 // K and V ring depths
constexpr int kPolyPerGroup = 4;                 // of every 16 exponentials, this many are computed on the FMA pipes
constexpr int kSW = 4;                        // softmax-backward warps: one per SM sub-partition
constexpr int kThreads = (kSW + 2) * 32;
constexpr uint32_t TM_S = 0, TM_DP = 128, TM_DQ = 384;   // dP / dS is double-buffered: 128 and 256

struct Maps {
  CUtensorMap q, d_o;
  PoolMaps kv;
};
struct Params {
  const int32_t* blob;
  int32_t off_qt, off_kvt, off_path_tiles, off_path_nvalid, off_path_loads, off_page_slot;
  int32_t Hq, G, T_q;
  int32_t chunk;   // block order, see block_to_item
  int64_t cap;
  float scale, scale_log2;
  const float* lse;
  const float* delta;
  __nv_bfloat16* d_q;
  float* part;  // unscaled fp32 dQ rows [n_part_rows][Hq][128] of items that do not own their rows
  int* status;
  int* done_ctr;   // CTAs whose producers have issued their last load
  int32_t resident;  // CTAs resident at once (one per SM)
};
struct __align__(8) Barriers {
  uint64_t qdo_full, k_full[KS], k_empty[KS], v_full[VS], v_empty[VS];
  uint64_t s_free, dp_full[2], ds_ready[2], dq_done;
};

__global__ void __launch_bounds__(kThreads, 1)
dq_kernel(const __grid_constant__ Maps maps, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sdO = sQ + kTileBytes;
  uint8_t* sK = sdO + kTileBytes;          // KS tiles
  uint8_t* sV = sK + KS * kTileBytes;      // VS tiles
  __shared__ Barriers bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int item, h;
  block_to_item(int(blockIdx.x), int(gridDim.x) / p.Hq, p.Hq, p.chunk, item, h);
  const int hk = h / p.G;
  const QTile qt = reinterpret_cast<const QTile*>(p.blob + p.off_qt)[item];
  const int32_t* path_nvalid = p.blob + p.off_path_nvalid + qt.pt_begin;
  const int n_tiles = qt.n_kv_tiles;

  if (tid == 0) {
    s_abort = 0;
    mbar_init(&bar.qdo_full, 1);
    for (int i = 0; i < KS; ++i) { mbar_init(&bar.k_full[i], 1); mbar_init(&bar.k_empty[i], 1); }
    for (int i = 0; i < VS; ++i) { mbar_init(&bar.v_full[i], 1); mbar_init(&bar.v_empty[i], 1); }
    mbar_init(&bar.s_free, kSW * 32);
    for (int i = 0; i < 2; ++i) { mbar_init(&bar.dp_full[i], 1); mbar_init(&bar.ds_ready[i], kSW * 32); }
    mbar_init(&bar.dq_done, 1);
    fence_mbar_init();
  }
  if (warp == kSW + 1) { tmem_alloc(&s_tmem, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;

  if (warp == kSW) {
    // ======================= TMA producer =======================
    if (lane == 0) {
      mbar_expect_tx(&bar.qdo_full, 2 * kTileBytes);
      load_row_tile(sQ, &maps.q, &bar.qdo_full, h, qt.q_row0);
      load_row_tile(sdO, &maps.d_o, &bar.qdo_full, h, qt.q_row0);
    }
    if (lane == 0) {
      // TMA coordinates of the item's KV tiles, resolved by the plan builder; the entry of tile j+1 is
      // fetched while the ring waits of tile j run
      const TileLoad* loads = reinterpret_cast<const TileLoad*>(p.blob + p.off_path_loads) + qt.pt_begin;
      const int64_t head_row0 = int64_t(hk) * p.cap;
      TileLoad cur = loads[0];
      for (int j = 0; j < n_tiles; ++j) {
        const TileLoad nxt = loads[j + 1 < n_tiles ? j + 1 : j];
        const int ks = j % KS, vs = j % VS;
        if (j >= KS && !mbar_wait_sleepy(&bar.k_empty[ks], ((j / KS) + 1) & 1, abortp, p.status)) break;
        load_kv_tile_at(sK + ks * kTileBytes, maps.kv.k, &bar.k_full[ks], cur, head_row0);
        if (j >= VS && !mbar_wait_sleepy(&bar.v_empty[vs], ((j / VS) + 1) & 1, abortp, p.status)) break;
        load_kv_tile_at(sV + vs * kTileBytes, maps.kv.v, &bar.v_full[vs], cur, head_row0);
        cur = nxt;
      }
      // The k-th CTA to get this far is about to make room for CTA `resident + k` (CTAs start in index
      // order, one per SM): its Q and dO tiles go to the L2 now, so that its first step does not wait for HBM.
      const int nb = atomicAdd(p.done_ctr, 1) + p.resident;
      if (nb < int(gridDim.x)) {
        int nitem, nh;
        block_to_item(nb, int(gridDim.x) / p.Hq, p.Hq, p.chunk, nitem, nh);
        const int nrow = reinterpret_cast<const QTile*>(p.blob + p.off_qt)[nitem].q_row0;
        tma_prefetch_2d(&maps.q, nh * 128, nrow);
        tma_prefetch_2d(&maps.q, nh * 128 + 64, nrow);
        tma_prefetch_2d(&maps.d_o, nh * 128, nrow);
        tma_prefetch_2d(&maps.d_o, nh * 128 + 64, nrow);
      }
    }
  } else if (warp == kSW + 1) {
    // ======================= MMA issuer =======================
    // All 32 lanes walk the loop and wait on the barriers (warp-uniform control flow and
    // address arithmetic); only the tcgen05 instructions are issued, by one elected lane.
    constexpr uint32_t idesc_kk = make_idesc(128, 128, 0, 0);  // S = Q K^T, dP = dO V^T
    constexpr uint32_t idesc_mn = make_idesc(128, 128, 0, 1);  // dQ += dS K, K is MN-major
    const uint32_t q_lo = desc_lo(smem_u32(sQ), 16), g_lo = desc_lo(smem_u32(sdO), 16);
    const uint32_t k_lo = desc_lo(smem_u32(sK), 16), v_lo = desc_lo(smem_u32(sV), 16);
    const uint32_t k_mn = desc_lo(smem_u32(sK), kHalfBytes);
    auto mma_kk = [&](uint32_t d, uint32_t a0, uint32_t b0) {
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2;
          mma_ss_lo(d, a0 + off, b0 + off, idesc_kk, k > 0);
        }
      }
    };
    auto commit = [&](uint64_t* b) { if (elect_one()) mma_commit(b); };
    auto wait = [&](uint64_t* b, uint32_t parity) {
      return __all_sync(0xffffffffu, mbar_wait_relaxed(b, parity, abortp, p.status));
    };
    bool ok = wait(&bar.qdo_full, 0) && wait(&bar.k_full[0], 0) && wait(&bar.v_full[0], 0);
    if (ok) {
      tc_fence_after();
      mma_kk(tmem + TM_S, q_lo, k_lo);
      mma_kk(tmem + TM_DP, g_lo, v_lo);
      commit(&bar.dp_full[0]);
      commit(&bar.v_empty[0]);
    }
    for (int j = 0; ok && j < n_tiles; ++j) {
      if (j + 1 < n_tiles) {
        // S(j+1) as soon as the warps have read S(j); dP(j+1) into the other dP buffer (last read
        // by dQ(j-1), which precedes it in the tensor pipe), so the warps' next step finds both ready
        const int vs = (j + 1) % VS;
        ok = mbar_wait_all3(&bar.s_free, j & 1, &bar.k_full[(j + 1) % KS], ((j + 1) / KS) & 1, &bar.v_full[vs],
                            ((j + 1) / VS) & 1, abortp, p.status);
        if (!ok) break;
        tc_fence_after();
        mma_kk(tmem + TM_S, q_lo, k_lo + ((j + 1) % KS) * (kTileBytes >> 4));
        mma_kk(tmem + TM_DP + ((j + 1) & 1) * 128, g_lo, v_lo + vs * (kTileBytes >> 4));
        commit(&bar.dp_full[(j + 1) & 1]);
        commit(&bar.v_empty[vs]);
      }
      ok = mbar_wait_all1(&bar.ds_ready[j & 1], (j >> 1) & 1, abortp, p.status);
      if (!ok) break;
      tc_fence_after();
      if (elect_one()) {
        // dS: packed bf16, 16 keys per 8 columns; keys 0-63 at +0, keys 64-127 at +64
        const uint32_t b0 = k_mn + (j % KS) * (kTileBytes >> 4);
        const uint32_t a0 = tmem + TM_DP + (j & 1) * 128;
        const uint32_t acc0 = j > 0;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          mma_ts_lo(tmem + TM_DQ, a0 + (k >> 2) * 64 + (k & 3) * 8, b0 + k * 128, idesc_mn, k > 0 ? 1u : acc0);
      }
      commit(&bar.k_empty[j % KS]);
    }
    if (ok) commit(&bar.dq_done);
  } else {
    // ======================= softmax-backward warps (4) =======================
    // One warp per SM sub-partition, one query row per thread.  (Two warps per sub-partition
    // compute a little faster, but between them they take every issue slot, and the MMA and
    // producer warps that share the sub-partitions then fall behind.)
    const int row = warp * 32 + lane;                     // query row inside the tile = TMEM lane
    const uint32_t t_lane = tmem + (uint32_t(warp * 32) << 16);
    const bool row_ok = row < qt.n_rows;
    const float lse2 = row_ok ? p.lse[int64_t(h) * p.T_q + qt.q_row0 + row] * kLog2e : 0.f;
    const float dl = row_ok ? p.delta[int64_t(h) * p.T_q + qt.q_row0 + row] : 0.f;
    const f32x2 scale2 = make_f32x2(p.scale_log2, p.scale_log2), neg_lse2 = make_f32x2(-lse2, -lse2),
                neg_dl2 = make_f32x2(-dl, -dl);
    bool ok = true;
    int nv_next = path_nvalid[0];
    for (int j = 0; j < n_tiles; ++j) {
      const int n_valid = nv_next;
      if (j + 1 < n_tiles) nv_next = path_nvalid[j + 1];
      const bool diag = qt.causal && (j == n_tiles - 1);
      const int limit = diag ? min(row + 1, n_valid) : n_valid;   // keys [0, limit) are visible
      const bool need_mask = diag || n_valid < 128;
      // S(j) and dP(j) are both complete well before the warps get here (the MMA warp issues them
      // one step ahead).  One wait covers both: dP(j) is issued right behind S(j) by the same thread,
      // and its commit tracks every MMA issued before it (a second wait would cost another
      // shared-memory round trip of ~150 cycles per step, on the warps that set the pace).
      // The whole score row goes to registers at once, so S may be overwritten.
      const uint32_t t_dp = t_lane + TM_DP + (j & 1) * 128;
      ok = mbar_wait(&bar.dp_full[j & 1], (j >> 1) & 1, abortp, p.status);
      if (!ok) break;
      tc_fence_after();
      uint32_t s[4][32], dp[2][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(t_lane + TM_S + c * 32, s[c]);
      tmem_ld32(t_dp, dp[0]);
      tmem_ld32(t_dp + 32, dp[1]);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bar.s_free);
      // P = exp2(S c - LSE) and dS = P o (dP - D) element by element: the exp2 (MUFU pipe) of one
      // element overlaps the arithmetic of its neighbours instead of forming a phase of its own
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        if (half == 1) {
          tmem_ld32(t_dp + 64, dp[0]);
          tmem_ld32(t_dp + 96, dp[1]);
          tmem_wait_ld();
        }
        // software pipeline over groups of 16 keys: the exp2 of group g+1 (MUFU pipe) is issued before
        // group g is multiplied, packed and stored
        float pe[2][16];
        auto exps = [&](int g, float (&out)[16]) {
          const int c = half * 2 + (g >> 1), i0 = (g & 1) * 16;
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            const f32x2 a = fma2(make_f32x2(s[c][i0 + i], s[c][i0 + i + 1]), scale2, neg_lse2);
            if (i < kPolyPerGroup) {   // a share of the exponentials goes to the FMA pipes
              ex2_fma_pair(a, out[i], out[i + 1]);
            } else {
              float a0, a1;
              split_f32x2(a, a0, a1);
              out[i] = ex2(a0);
              out[i + 1] = ex2(a1);
            }
          }
        };
        exps(0, pe[0]);
        uint32_t pk[16];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          if (g + 1 < 4) exps(g + 1, pe[(g + 1) & 1]);
          float (&cur)[16] = pe[g & 1];
          const int c = g >> 1, i0 = (g & 1) * 16;
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            float d0, d1;
            split_f32x2(mul2(make_f32x2(cur[i], cur[i + 1]),
                             add2(make_f32x2(dp[c][i0 + i], dp[c][i0 + i + 1]), neg_dl2)), d0, d1);
            if (need_mask) {  // masked columns may hold anything (pad rows of K, V): select, do not multiply
              d0 = (half * 64 + g * 16 + i < limit) ? d0 : 0.f;
              d1 = (half * 64 + g * 16 + i + 1 < limit) ? d1 : 0.f;
            }
            pk[(g & 1) * 8 + (i >> 1)] = pack_bf16(d0, d1);
          }
          // dS: packed bf16, keys 0-63 in columns [0, 32), keys 64-127 in columns [64, 96) of the dP buffer
          if (g & 1) tmem_st16(t_dp + half * 64 + c * 16, pk);
        }
      }
      // K rows at or beyond n_valid must be zero before dS K (dS is zero there, K may hold anything)
      if (n_valid < 128) {
        ok = mbar_wait(&bar.k_full[j % KS], (j / KS) & 1, abortp, p.status);
        if (!ok) break;
        if (row >= n_valid) zero_tile_row(sK + (j % KS) * kTileBytes, row);
        fence_proxy_async();
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bar.ds_ready[j & 1]);
    }
    // ---- dQ = scale * accumulator ----
    if (ok) ok = mbar_wait(&bar.dq_done, 0, abortp, p.status);
    if (ok) {
      tc_fence_after();
      // Final rows leave through shared memory (the K ring is idle by now: every MMA has completed), so
      // that a warp's store instruction covers two whole 256-byte rows instead of 16 bytes of 32 rows.
      // A warp stages only its own 32 rows: 272-byte pitch, no bank conflicts either way, no CTA barrier.
      constexpr int kPitch = 272;
      uint8_t* stage = sK + warp * (32 * kPitch);
      uint32_t acc[4][32];   // the whole accumulator row in one round trip
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(t_lane + TM_DQ + c * 32, acc[c]);
      tmem_wait_ld();
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t (&r)[32] = acc[c];
        if (qt.part_row0 < 0) {
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(r[8 * x + 0]) * p.scale, __uint_as_float(r[8 * x + 1]) * p.scale);
            v.y = pack_bf16(__uint_as_float(r[8 * x + 2]) * p.scale, __uint_as_float(r[8 * x + 3]) * p.scale);
            v.z = pack_bf16(__uint_as_float(r[8 * x + 4]) * p.scale, __uint_as_float(r[8 * x + 5]) * p.scale);
            v.w = pack_bf16(__uint_as_float(r[8 * x + 6]) * p.scale, __uint_as_float(r[8 * x + 7]) * p.scale);
            *reinterpret_cast<uint4*>(stage + lane * kPitch + c * 64 + x * 16) = v;
          }
          continue;
        }
        if (row_ok) {
          // the row has other contributors: unscaled fp32 partial, summed by the merge kernel
          float* prow = p.part + (int64_t(qt.part_row0 + row) * p.Hq + h) * 128 + c * 32;
#pragma unroll
          for (int x = 0; x < 8; ++x)
            *reinterpret_cast<float4*>(prow + x * 4) =
                make_float4(__uint_as_float(r[4 * x]), __uint_as_float(r[4 * x + 1]), __uint_as_float(r[4 * x + 2]),
                            __uint_as_float(r[4 * x + 3]));
        }
      }
      if (qt.part_row0 < 0) {
        __syncwarp();
        const int sub = lane >> 4, piece = lane & 15;
#pragma unroll 4
        for (int it = 0; it < 16; ++it) {
          const int rr = it * 2 + sub;                      // row inside the warp's 32
          const uint4 v = *reinterpret_cast<const uint4*>(stage + rr * kPitch + piece * 16);
          if (warp * 32 + rr < qt.n_rows)
            *reinterpret_cast<uint4*>(p.d_q + (int64_t(qt.q_row0 + warp * 32 + rr) * p.Hq + h) * 128 + piece * 8) = v;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kSW + 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

psrl_status_t dq_bf16(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const DeviceHeader& H = P.hdr;
  const int64_t cap = a.pool_capacity;
  if (P.T_q == 0 || P.q_tiles.empty()) return PSRL_OK;
  auto fail = [](cudaError_t e) { set_last_cuda_error(e); return PSRL_ERR_CUDA; };
  Maps m;
  bool ok = make_pool_maps(&m.kv, a.k_pool, a.v_pool, P.Hkv, cap) &&
            make_map_bf16_2d(&m.q, a.q, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, 128) &&
            make_map_bf16_2d(&m.d_o, a.d_o, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, 128);
  if (!ok) return PSRL_ERR_CUDA;
  const size_t smem = size_t(2 + KS + VS) * kTileBytes + 1024;
  static bool attr_set[64] = {};
  cudaError_t e = ensure_dynamic_smem(dq_kernel, smem, attr_set);
  if (e != cudaSuccess) return fail(e);
  Params p{};
  p.blob = P.dev;
  p.off_qt = H.off_qt; p.off_kvt = H.off_kvt; p.off_path_tiles = H.off_path_tiles;
  p.off_path_nvalid = H.off_path_nvalid; p.off_path_loads = H.off_path_loads; p.off_page_slot = H.off_page_slot;
  p.Hq = P.Hq; p.G = P.Hq / P.Hkv; p.T_q = P.T_q;
  p.cap = cap; p.scale = a.scale; p.scale_log2 = a.scale * kLog2e;
  p.lse = a.lse_in; p.delta = a.delta; p.d_q = static_cast<__nv_bfloat16*>(a.d_q); p.status = a.status;
  p.part = a.part;
  p.done_ctr = a.status + kWsCtrDq; p.resident = resident_ctas();
  p.chunk = block_order_chunk(int64_t(P.q_tiles.size()), p.resident, 4);
  const int64_t grid = int64_t(P.q_tiles.size()) * P.Hq;
  if (grid > INT32_MAX) return PSRL_ERR_SHAPE;
  dq_kernel<<<unsigned(grid), kThreads, smem, a.stream>>>(m, p);
  if ((e = cudaGetLastError()) != cudaSuccess) return fail(e);
  return merge_dq_bf16(a);
}

}  // namespace psrl

// bf16 tree attention forward on the 5th-generation tensor cores.
//
// One CTA = one query tile (up to 128 rows of one segment) x up to two query
// heads of the same KV head.  It walks the tile's path of KV tiles (all tiles
// of the ancestor segments, then the own segment's tiles up to the diagonal;
// paper Sec. 2.5: full visibility of the shared prefix + causal own suffix),
// gathering K/V pages from the paged pools through the block metadata
// (Sec. 6) with TMA.
//
// Warp roles (NQ = 2):
//   warps 0-3   softmax warpgroup of head 0   (one query row per thread)
//   warps 4-7   softmax warpgroup of head 1
//   warp  8     TMA producer (Q once, then the K and V rings)
//   warp  9     MMA issuer + TMEM owner
// Tensor memory (512 columns): per head q, S_q at q*256 (128 fp32 columns,
// later overwritten by P_q as packed bf16 in its first 64 columns) and the
// per-tile product O_q = P_q V at q*256+128.
//   S = Q K^T      tcgen05.mma, A and B from shared memory (K-major, 128B swizzle)
//   O_tile = P V   tcgen05.mma, A = P from tensor memory, B = V (MN-major)
// The MMA issuer alternates between the two heads, so the tensor cores work
// on one head while the other head's warpgroup does its softmax.  O accumulates
// in tensor memory across the KV tiles (online softmax: per-tile partial
// results are merged by log-sum-exp).  Each softmax thread owns one query row:
// it reads the whole 128-wide score row in one round trip, keeps the running
// sum and a reference maximum in registers, and moves that reference only when
// the true maximum has grown by more than 2^8 - only then is the accumulator
// row in tensor memory rescaled (rare after the first tiles).
#include <cuda_bf16.h>
#include <math_constants.h>

#include "attn_bf16_common.cuh"
#include "kernels.h"
#include "tma.h"

namespace psrl {
namespace {
using namespace sm100;

constexpr int NQ = 2;                    // query heads per CTA
constexpr int KS = 2, VS = 2;            // K and V ring depths
constexpr int kThreads = (4 * NQ + 2) * 32;
// named barriers (the softmax warps of head q arrive, the MMA warp syncs): P_q of a tile stored
constexpr uint32_t kBarP = 1, kBarThreads = 128 + 32;

struct FwdMaps {
  CUtensorMap q;
  PoolMaps kv;
};

struct FwdParams {
  const int32_t* blob;
  int32_t off_qt, off_kvt, off_path_tiles, off_path_nvalid, off_path_loads, off_page_slot;
  int32_t Hq, Hkv, G, T_q, pairs_per_group;
  int64_t cap;
  float scale_log2;
  __nv_bfloat16* o;
  float* lse;
  float* part;      // partial rows [n_part_rows][Hq][128]: normalised O of items that do not own their rows
  float* part_lse;  // [n_part_rows][Hq]
  int* status;
  int* done_ctr;     // CTAs whose producers have issued their last load
  int32_t resident;  // CTAs resident at once (one per SM)
};

struct __align__(8) Barriers {
  uint64_t q_full;
  uint64_t k_full[KS], k_empty[KS], v_full[VS], v_empty[VS];
  uint64_t s_full[NQ], o_full[NQ];
};

__global__ void __launch_bounds__(kThreads, 1)
fwd_kernel(const __grid_constant__ FwdMaps maps, const FwdParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                          // NQ tiles
  uint8_t* sK = sQ + NQ * kTileBytes;          // KS tiles
  uint8_t* sV = sK + KS * kTileBytes;          // VS tiles
  __shared__ Barriers bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // ---- which work item ----
  const int units = p.Hkv * p.pairs_per_group;
  const int item = blockIdx.x / units, u = blockIdx.x % units;
  const int hk = u / p.pairs_per_group, pair = u % p.pairs_per_group;
  const int h0 = hk * p.G + pair * NQ;
  const int nq = min(NQ, p.G - pair * NQ);
  const QTile qt = reinterpret_cast<const QTile*>(p.blob + p.off_qt)[item];
  const int32_t* path_nvalid = p.blob + p.off_path_nvalid + qt.pt_begin;
  const int n_tiles = qt.n_kv_tiles;

  if (tid == 0) {
    s_abort = 0;
    mbar_init(&bar.q_full, 1);
    for (int i = 0; i < KS; ++i) { mbar_init(&bar.k_full[i], 1); mbar_init(&bar.k_empty[i], 1); }
    for (int i = 0; i < VS; ++i) { mbar_init(&bar.v_full[i], 1); mbar_init(&bar.v_empty[i], 1); }
    for (int i = 0; i < NQ; ++i) {
      mbar_init(&bar.s_full[i], 1); mbar_init(&bar.o_full[i], 1);
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
      tma_prefetch_desc(&maps.q);
      mbar_expect_tx(&bar.q_full, uint32_t(nq) * kTileBytes);
      for (int q = 0; q < nq; ++q) {
        load_row_tile(sQ + q * kTileBytes, &maps.q, &bar.q_full, h0 + q, qt.q_row0);
      }
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
      // order, one per SM): its Q tiles go to the L2 now, so that its first step does not wait for HBM.
      const int nb = atomicAdd(p.done_ctr, 1) + p.resident;
      if (nb < int(gridDim.x)) {
        const int nu = nb % units, npair = nu % p.pairs_per_group;
        const int nh0 = (nu / p.pairs_per_group) * p.G + npair * NQ, nnq = min(NQ, p.G - npair * NQ);
        const int nrow = reinterpret_cast<const QTile*>(p.blob + p.off_qt)[nb / units].q_row0;
        for (int q = 0; q < nnq; ++q) {
          tma_prefetch_2d(&maps.q, (nh0 + q) * 128, nrow);
          tma_prefetch_2d(&maps.q, (nh0 + q) * 128 + 64, nrow);
        }
      }
    }
  } else if (warp == 4 * NQ + 1) {
    // ======================= MMA issuer =======================
    // All 32 lanes walk the loop and wait on the barriers, so control flow and address
    // arithmetic stay warp-uniform; only the tcgen05 instructions are issued by lane 0.
    // (A loop that only lane 0 executes turns every descriptor computation into
    // per-thread work that competes with the softmax warps for issue slots.)
    {
      constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // S = Q K^T, both K-major
      constexpr uint32_t idesc_o = make_idesc(128, 128, 0, 1);   // O = P V, V is MN-major
      // descriptor low words (address >> 4 | LBO field); per K step only a constant is added
      const uint32_t q_lo = desc_lo(smem_u32(sQ), 16), k_lo = desc_lo(smem_u32(sK), 16);
      const uint32_t v_mn = desc_lo(smem_u32(sV), kHalfBytes);
      auto issue_s = [&](int q, int ks) {
        const uint32_t a0 = q_lo + q * (kTileBytes >> 4), b0 = k_lo + ks * (kTileBytes >> 4);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t off = (k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2;
            mma_ss_lo(tmem + q * 256, a0 + off, b0 + off, idesc_s, k > 0);
          }
        }
      };
      auto issue_pv = [&](int q, int vs, bool first) {
        const uint32_t b0 = v_mn + vs * (kTileBytes >> 4);
        const uint32_t acc0 = first ? 0u : 1u;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ts_lo(tmem + q * 256 + 128, tmem + q * 256 + k * 8, b0 + k * 128, idesc_o, k > 0 ? 1u : acc0);
        }
      };
      auto commit = [&](uint64_t* b) { if (elect_one()) mma_commit(b); };
      auto wait = [&](uint64_t* b, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait_relaxed(b, parity, abortp, p.status));
      };
      bool ok = wait(&bar.q_full, 0) && wait(&bar.k_full[0], 0);
      if (ok) {
        tc_fence_after();
        for (int q = 0; q < nq; ++q) { issue_s(q, 0); commit(&bar.s_full[q]); }
        commit(&bar.k_empty[0]);
      }
      for (int j = 0; ok && j < n_tiles; ++j) {
        const int vs = j % VS;
        for (int q = 0; ok && q < nq; ++q) {
          // one round of barrier tests per head: for head 0 also the V tile of this step and the K tile
          // of the next one (each separate wait would cost the issuing warp hundreds of cycles)
          if (q == 0) {
            // the V tile of this step and the K tile of the next one first (they land while the warps
            // still compute), then the hand-off of P through the named barrier
            const bool more = j + 1 < n_tiles;
            const int ksn = (j + 1) % KS;
            ok = mbar_wait_all3(&bar.v_full[vs], (j / VS) & 1, &bar.v_full[vs], (j / VS) & 1,
                                more ? &bar.k_full[ksn] : &bar.v_full[vs], more ? ((j + 1) / KS) & 1 : (j / VS) & 1,
                                abortp, p.status);
            if (!ok) break;
          }
          named_sync(kBarP + q, kBarThreads);
          tc_fence_after();
          issue_pv(q, vs, j == 0);
          commit(&bar.o_full[q]);
          if (q == nq - 1) commit(&bar.v_empty[vs]);
          if (j + 1 < n_tiles) {
            const int ks = (j + 1) % KS;
            issue_s(q, ks);
            commit(&bar.s_full[q]);
            if (q == nq - 1) commit(&bar.k_empty[ks]);
          }
        }
      }
    }
  } else if (warp < 4 * nq) {
    // ======================= softmax warpgroups =======================
    const int q = warp >> 2;
    const int row = tid & 127;                                  // query row inside the tile
    const uint32_t t_lane = tmem + (uint32_t((warp & 3) * 32) << 16) + q * 256;
    // m_ref: the reference maximum (log2 units) the row's P values and running sum are
    // expressed against.  It follows the true running maximum lazily: it only moves when
    // the maximum has grown by more than 2^8, so the output accumulator in tensor memory
    // is rescaled rarely (typically only on the first tiles) instead of once per tile.
    float m_ref = -CUDART_INF_F, l_run = 0.f;
    const f32x2 scale2 = make_f32x2(p.scale_log2, p.scale_log2);
    bool ok = true;
    int nv_next = path_nvalid[0];
    for (int j = 0; j < n_tiles; ++j) {
      const int n_valid = nv_next;
      if (j + 1 < n_tiles) nv_next = path_nvalid[j + 1];
      const bool diag = qt.causal && (j == n_tiles - 1);
      const int limit = diag ? min(row + 1, n_valid) : n_valid;  // keys [0, limit) are visible
      const bool need_mask = diag || n_valid < 128;
      // A warp that gave up on a wait (ok == false) skips the tile's work but still arrives on the named
      // barrier of every remaining tile, so that the MMA warp is never left waiting at one - one arrival
      // per tile, and for tile j only once the MMA warp has synced on tile j-1: that is what a completed
      // o_full[q] phase j-1 says (its commit follows P V(j-1), issued right behind that sync).  The MMA
      // warp therefore carries nothing for this path (a shared-memory store per tile in that warp cost the
      // kernel 1.5-3 %).  If the phase never completes the MMA warp has left its loop: stop arriving.
      do {
      if (!ok) break;
      // ---- softmax of this tile: the whole score row in one round trip to tensor memory ----
      ok = mbar_wait(&bar.s_full[q], j & 1, abortp, p.status);
      if (!ok) break;
      tc_fence_after();
      uint32_t s[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(t_lane + c * 32, s[c]);
      tmem_wait_ld();
      // exponentials of the row against the reference m, P stored as bf16, row sum returned; with
      // mx_out the row maximum (raw scores) is tracked in the same pass
      auto exp_pass = [&](float m, bool masked, float* mx_out) -> float {
        f32x2 sum2 = make_f32x2(0.f, 0.f);
        const f32x2 neg_m2 = make_f32x2(-m, -m);
        float mx = -CUDART_INF_F;
        // software pipeline over groups of 16 columns: the exp2 of group g+1 (MUFU pipe, 8 cycles per
        // warp instruction) is issued before group g is summed, packed and stored
        float e[2][16];
        auto exps = [&](int g, float (&out)[16]) {
          const int c = g >> 1, i0 = (g & 1) * 16;
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            float a0, a1;
            split_f32x2(fma2(make_f32x2(s[c][i0 + i], s[c][i0 + i + 1]), scale2, neg_m2), a0, a1);
            out[i] = ex2(a0);
            out[i + 1] = ex2(a1);
            if (mx_out) mx = fmax3(mx, __uint_as_float(s[c][i0 + i]), __uint_as_float(s[c][i0 + i + 1]));
          }
        };
        exps(0, e[0]);
        uint32_t pk[16];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          if (g + 1 < 8) exps(g + 1, e[(g + 1) & 1]);
          float (&cur)[16] = e[g & 1];
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            float e0 = cur[i], e1 = cur[i + 1];
            if (masked) {
              e0 = (g * 16 + i < limit) ? e0 : 0.f;
              e1 = (g * 16 + i + 1 < limit) ? e1 : 0.f;
            }
            sum2 = add2(sum2, make_f32x2(e0, e1));
            pk[(g & 1) * 8 + (i >> 1)] = pack_bf16(e0, e1);
          }
          if (g & 1) tmem_st16(t_lane + (g >> 1) * 16, pk);
        }
        if (mx_out) *mx_out = mx;
        float lo, hi;
        split_f32x2(sum2, lo, hi);
        return lo + hi;
      };
      float sum, m_use, alpha;
      bool any_move;
      bool settled = false;
      float mx = -CUDART_INF_F;
      if (j > 0 && !need_mask) {
        // Interior tile: bet that the reference stays (it moves only when the maximum grows by more than
        // 2^8, rare after the first tiles) and compute the exponentials at once, tracking the maximum on
        // the side instead of in a pass of its own; if the bet fails for any row of the warp the tile is
        // redone below (P and the sum are simply recomputed from the scores held in registers).
        sum = exp_pass(m_ref, false, &mx);
        const bool move = fmaxf(m_ref, mx * p.scale_log2) > m_ref + 8.f;
        any_move = __any_sync(0xffffffffu, move);
        if (!any_move) { settled = true; m_use = m_ref; alpha = 1.f; }
      } else if (need_mask) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int i = 0; i < 32; ++i)
            mx = fmaxf(mx, (c * 32 + i < limit) ? __uint_as_float(s[c][i]) : -CUDART_INF_F);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int i = 0; i < 32; i += 2)
            mx = fmax3(mx, __uint_as_float(s[c][i]), __uint_as_float(s[c][i + 1]));
      }
      if (!settled) {
        const float m_new = fmaxf(m_ref, mx * p.scale_log2);
        const bool move = m_new > m_ref + 8.f;            // also true on the first tile (m_ref = -inf)
        any_move = __any_sync(0xffffffffu, move);
        m_use = move ? m_new : m_ref;
        alpha = ex2(m_ref - m_use);                        // 1 if the reference stays, 0 on the first tile
        sum = exp_pass(m_use, need_mask, nullptr);
      }
      l_run = fmaf(l_run, alpha, sum);
      m_ref = m_use;
      // ---- the reference moved: rescale the accumulated output in tensor memory ----
      if (j > 0 && any_move) {
        ok = mbar_wait(&bar.o_full[q], (j - 1) & 1, abortp, p.status);  // P V of the previous tile is complete
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld32(t_lane + 128 + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
          tmem_st32(t_lane + 128 + c * 32, r);
        }
      }
      // V rows at or beyond n_valid (page pads, rows no page covers) must be zero before P V
      if (q == 0 && n_valid < 128) {
        ok = mbar_wait(&bar.v_full[j % VS], (j / VS) & 1, abortp, p.status);
        if (!ok) break;
        if (row >= n_valid) zero_tile_row(sV + (j % VS) * kTileBytes, row);
        fence_proxy_async();
      }
      tmem_wait_st();
      } while (false);
      tc_fence_before();
      if (!ok && j > 0 && !mbar_wait_bounded(&bar.o_full[q], (j - 1) & 1)) break;
      named_arrive(kBarP + q, kBarThreads);
    }
    // ---- last tile's product, normalise, store ----
    if (ok) ok = mbar_wait(&bar.o_full[q], (n_tiles - 1) & 1, abortp, p.status);
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l_run;
      const bool store = row < qt.n_rows;
      const int h = h0 + q;
      const bool partial = qt.part_row0 >= 0;
      // Final rows leave through shared memory (the Q tiles and the K ring are idle by now: every
      // S = Q K^T has completed), so that a warp's store instruction covers two whole 256-byte rows
      // instead of 16 bytes of 32 rows.  A warp stages only its own 32 rows: 272-byte pitch, no bank
      // conflicts either way, no CTA barrier.
      constexpr int kPitch = 272;
      uint8_t* stage = sQ + warp * (32 * kPitch);
      float* prow = p.part + (int64_t(qt.part_row0 + row) * p.Hq + h) * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(t_lane + 128 + c * 32, r);
        tmem_wait_ld();
        if (partial) {
          if (store) {
#pragma unroll
            for (int x = 0; x < 8; ++x)
              *reinterpret_cast<float4*>(prow + c * 32 + x * 4) =
                  make_float4(__uint_as_float(r[4 * x]) * inv, __uint_as_float(r[4 * x + 1]) * inv,
                              __uint_as_float(r[4 * x + 2]) * inv, __uint_as_float(r[4 * x + 3]) * inv);
          }
          continue;
        }
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2)
          pk[i >> 1] = pack_bf16(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv);
#pragma unroll
        for (int x = 0; x < 4; ++x)
          *reinterpret_cast<uint4*>(stage + lane * kPitch + c * 64 + x * 16) =
              make_uint4(pk[4 * x], pk[4 * x + 1], pk[4 * x + 2], pk[4 * x + 3]);
      }
      if (!partial) {
        __syncwarp();
        const int sub = lane >> 4, piece = lane & 15, wrow0 = (warp & 3) * 32;
#pragma unroll 4
        for (int it = 0; it < 16; ++it) {
          const int rr = it * 2 + sub;                      // row inside the warp's 32
          const uint4 v = *reinterpret_cast<const uint4*>(stage + rr * kPitch + piece * 16);
          if (wrow0 + rr < qt.n_rows)
            *reinterpret_cast<uint4*>(p.o + (int64_t(qt.q_row0 + wrow0 + rr) * p.Hq + h) * 128 + piece * 8) = v;
        }
      }
      if (store && partial) p.part_lse[int64_t(qt.part_row0 + row) * p.Hq + h] = (m_ref + log2f(l_run)) * kLn2;
      else
      if (store) p.lse[int64_t(h) * p.T_q + qt.q_row0 + row] = (m_ref + log2f(l_run)) * kLn2;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4 * NQ + 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

bool make_pool_maps(PoolMaps* maps, const void* k_pool, const void* v_pool, int Hkv, int64_t cap) {
  const uint32_t rows[4] = {16, 32, 64, 128};
  for (int i = 0; i < 4; ++i) {
    if (!make_map_bf16_2d(&maps->k[i], k_pool, 128, uint64_t(Hkv) * cap, 256, rows[i])) return false;
    if (!make_map_bf16_2d(&maps->v[i], v_pool, 128, uint64_t(Hkv) * cap, 256, rows[i])) return false;
  }
  return true;
}

psrl_status_t fwd_bf16(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const int64_t cap = a.pool_capacity;
  if (int64_t(P.Hkv) * cap > INT32_MAX || int64_t(P.Hq) * 128 > INT32_MAX) return PSRL_ERR_SHAPE;
  FwdMaps maps;
  bool ok = make_map_bf16_2d(&maps.q, a.q, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, 128);
  ok = ok && make_pool_maps(&maps.kv, a.k_pool, a.v_pool, P.Hkv, cap);
  if (!ok) return PSRL_ERR_CUDA;
  const DeviceHeader& H = P.hdr;
  FwdParams p{};
  p.blob = P.dev;
  p.off_qt = H.off_qt; p.off_kvt = H.off_kvt; p.off_path_tiles = H.off_path_tiles;
  p.off_path_nvalid = H.off_path_nvalid; p.off_path_loads = H.off_path_loads; p.off_page_slot = H.off_page_slot;
  p.Hq = P.Hq; p.Hkv = P.Hkv; p.G = P.Hq / P.Hkv; p.T_q = P.T_q;
  p.pairs_per_group = (p.G + NQ - 1) / NQ;
  p.cap = cap;
  p.scale_log2 = a.scale * kLog2e;
  p.o = static_cast<__nv_bfloat16*>(a.o_out);
  p.lse = a.lse_out;
  p.part = a.part; p.part_lse = a.part_lse;
  p.status = a.status;
  p.done_ctr = a.status + kWsCtrFwd; p.resident = resident_ctas();
  const size_t smem = size_t(NQ + KS + VS) * kTileBytes + 1024;
  static bool attr_set[64] = {};
  {
    const cudaError_t e = ensure_dynamic_smem(fwd_kernel, smem, attr_set);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PSRL_ERR_CUDA; }
  }
  const int64_t grid = int64_t(P.q_tiles.size()) * P.Hkv * p.pairs_per_group;
  if (grid == 0) return PSRL_OK;
  if (grid > INT32_MAX) return PSRL_ERR_SHAPE;
  fwd_kernel<<<unsigned(grid), kThreads, smem, a.stream>>>(maps, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_last_cuda_error(e); return PSRL_ERR_CUDA; }
  return merge_fwd_bf16(a);
}

}  // namespace psrl

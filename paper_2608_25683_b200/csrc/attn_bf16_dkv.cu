// bf16 dK/dV kernel (key-stationary) and the fixed-order reduce of split tiles.
//
// One CTA = one work item: a KV tile (<= 128 keys of one segment, one KV head)
// and a range of 128-row query sub-tiles that attend to it - the later rows of
// the tile's own segment, then the rows of ALL descendant segments, which form
// one contiguous row range in the canonical layout (paper Sec. 6: the adjoints
// of every consumer are accumulated on the shared prefix) - times the Hq/Hkv
// query heads of the KV head.  K and V stay in shared memory; dK and dV
// accumulate in tensor memory over the whole loop.
//
// Per step (128 query rows of one head) the tensor cores run four contractions
// (M = 128 keys, N = 128, K = 128) and the warps run two half-steps:
//   S^T  = K Q^T - LSE/c         -> warps: P^T = exp2(S^T c), written over S^T as bf16
//   dV  += P^T dO                   (A = P^T from tensor memory, dO MN-major in smem)
//   dP^T = V dO^T - D            -> warps: dS^T = P^T o dP^T, written over dP^T as bf16
//   dK  += dS^T Q                   (A = dS^T from tensor memory, Q MN-major in smem)
// The issue order is  dV(i), S^T(i+1), dK(i), dP^T(i+1):  while the warps turn S^T(i+1)
// into P^T(i+1) the tensor cores work on dK(i) and dP^T(i+1); while they turn dP^T(i+1)
// into dS^T(i+1) the tensor cores work on dV(i+1) and S^T(i+2).  S^T may be overwritten
// as soon as dV(i) has been issued (it consumed P^T(i)), dP^T as soon as dK(i) has been.
//
// The per-row terms -LSE/c and -D enter S^T and dP^T as one more K = 16 MMA slice (a three-term bf16
// split of the value against a slice of ones), so the warps need no per-column loads.
//
// Tensor memory (512 columns): S^T at 0, dP^T at 128, dV at 256, dK at 384.
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

constexpr int ST = 2;                              // (Q, dO) tile ring depth
static_assert(kSubRows == 128, "the dK/dV kernel steps through 128-row query tiles");
constexpr int kThreads = (8 + 2) * 32;             // 8 softmax-backward warps + producer + MMA
constexpr uint32_t TM_ST = 0, TM_DPT = 128, TM_DV = 256, TM_DK = 384;
// named barriers (softmax warps arrive, the MMA warp syncs): dS^T(i) stored; quarters of P^T(i) stored
// (dV starts on the first quarter while the warps still compute the rest)
constexpr uint32_t kBarDs = 1, kBarP = 2, kBarThreads = 8 * 32 + 32;   // dS^T: id 1; P^T quarters: ids 2..5

struct Maps {
  CUtensorMap q, d_o;  // boxes of 128 rows x 64 columns
  PoolMaps kv;
};
struct Params {
  const int32_t* blob;
  int32_t off_kvi, off_kvt, off_page_slot, off_split;
  int32_t Hq, Hkv, G, T_q;
  int32_t chunk;   // items per KV-head-major chunk of the block order, 0 = item-major
  int64_t cap;
  float scale, scale_log2, inv_scale;
  const float* lse;
  const float* delta;
  float* slabs;
  __nv_bfloat16 *dk, *dv;
  int* status;
};
struct __align__(8) Barriers {
  // Q (+ the LSE slice) and dO (+ the D slice) of a step have barriers of their own: dO is free again after
  // dV(i), Q only after dK(i), and the Q tile of the next step is what the tensor cores wait for
  uint64_t kv_full, q_full[ST], q_empty[ST], do_full[ST], do_empty[ST], s_full, dp_full, acc_full;
};

// The per-query-row terms of the backward are folded into the contractions as one extra
// K = 16 step each, so the warps never have to fetch a per-column value:
//   S^T_aug  = K Q^T   + 1 (x) (-LSE / scale)   ->  P^T  = exp2(scale log2e S^T_aug)
//   dP^T_aug = V dO^T  + 1 (x) (-D)             ->  dS^T = P^T o dP^T_aug
// The extra operands are [128 rows][16] bf16 slices in the no-swizzle K-major layout (8-row x
// 16-byte core matrices: row r, column c at (r/8)*256 + (c/8)*128 + (r%8)*16 + (c%8)*2).  The
// fp32 term is carried exactly as the sum of three bf16 numbers in columns 0-2 against ones.
// A query row beyond the valid range gets -inf, which makes its P^T column exactly zero.
constexpr int kSliceBytes = 128 * 16 * 2;
constexpr uint32_t kSliceDescHi = (256u >> 4) | (1u << 14);  // SBO 256 bytes, version 1, no swizzle
__device__ __forceinline__ uint32_t slice_row_offset(int r) { return uint32_t(r >> 3) * 256u + uint32_t(r & 7) * 16u; }
__device__ __forceinline__ uint32_t slice_desc_lo(uint32_t smem_addr) {
  return ((smem_addr & 0x3FFFF) >> 4) | ((128u >> 4) << 16);  // LBO 128 bytes: the second 8 columns
}
// x == a + b + c to fp32 precision, each term a bf16 (returned as raw 16-bit patterns)
__device__ __forceinline__ uint2 split3_bf16(float x) {
  const __nv_bfloat16 a = __float2bfloat16_rn(x);
  float r = x - __bfloat162float(a);
  const __nv_bfloat16 b = __float2bfloat16_rn(r);
  r -= __bfloat162float(b);
  const __nv_bfloat16 c = __float2bfloat16_rn(r);
  return make_uint2(uint32_t(__bfloat16_as_ushort(a)) | (uint32_t(__bfloat16_as_ushort(b)) << 16),
                    uint32_t(__bfloat16_as_ushort(c)));
}
__device__ __forceinline__ void mma_ss_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                            uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
      "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}

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
  uint8_t* sQ = sV + kTileBytes;             // ST tiles
  uint8_t* sdO = sQ + ST * kTileBytes;       // ST tiles
  // K = 16 slices that fold the per-query-row terms into the contractions (see above)
  uint8_t* sOnes = sdO + ST * kTileBytes;    // [128 keys][16]: columns 0-2 = 1
  uint8_t* sLseX = sOnes + kSliceBytes;      // ST x [128 rows][16]: columns 0-2 = -LSE / scale in three bf16 terms
  uint8_t* sDlX = sLseX + ST * kSliceBytes;  // ST x [128 rows][16]: columns 0-2 = -D in three bf16 terms
  __shared__ Barriers bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ StepBeacon s_beacon;   // the MMA warp's position, for softmax warps that gave up on a wait

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Block order.  Small launches: item-major (block = item x Hkv + hk), which keeps the longest-first order of
  // the items exact.  Large launches: KV-head-major inside chunks of `p.chunk` items, so that the CTAs that run
  // at the same time mostly belong to one KV head and the Q and dO rows they stream (those of that head's query
  // heads) compete for the L2 with a quarter or an eighth of the set; the chunks still follow the longest-first
  // order.
  int item, hk;
  block_to_item(int(blockIdx.x), int(gridDim.x) / p.Hkv, p.Hkv, p.chunk, item, hk);
  const KvItem it = reinterpret_cast<const KvItem*>(p.blob + p.off_kvi)[item];
  const KvTile kt = reinterpret_cast<const KvTile*>(p.blob + p.off_kvt)[it.kvt];
  const int n_own_sub = it.own_q_row0 >= 0 ? (it.own_q_end - it.own_q_row0 + kSubRows - 1) / kSubRows : 0;
  const int n_it = (it.sub_end - it.sub_begin) * p.G;

  if (tid == 0) {
    s_abort = 0;
    s_beacon.at = -1;
    s_beacon.left = 0;
    mbar_init(&bar.kv_full, 1);
    for (int i = 0; i < ST; ++i) {
      mbar_init(&bar.q_full[i], 2); mbar_init(&bar.q_empty[i], 1);
      mbar_init(&bar.do_full[i], 2); mbar_init(&bar.do_empty[i], 1);
    }
    mbar_init(&bar.s_full, 1); mbar_init(&bar.dp_full, 1);
    mbar_init(&bar.acc_full, 1);
    fence_mbar_init();
  }
  if (warp == 9) { tmem_alloc(&s_tmem, 512); tmem_relinquish(); }
  // the constant slice: row r = key r, columns 0-2 = 1.0, the rest 0 (each row is 2 x 16 bytes)
  if (tid < 128) {
    uint8_t* r0 = sOnes + slice_row_offset(tid);
    *reinterpret_cast<uint4*>(r0) = make_uint4(0x3F803F80u, 0x00003F80u, 0u, 0u);
    *reinterpret_cast<uint4*>(r0 + 128) = make_uint4(0u, 0u, 0u, 0u);
  }
  fence_proxy_async();
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
      diag = su == 0;
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
      // write the step's -LSE / scale and -D slices next to them.  The LSE / D values of a
      // step are fetched (plain global loads) one step ahead, so their latency is not added
      // to the time a freed stage takes to fill.  Every stage barrier gets two arrivals: the
      // TMA byte count and the slices (after fence.proxy.async: the tensor cores read them).
      auto fetch = [&](int i, float (&lv)[4], float (&dv)[4], int& nvq_out) {
        int g, row0, nvq, qpos0; bool diag;
        step(i, g, row0, nvq, diag, qpos0);
        const int h = hk * p.G + g;
        const float* lse_row = p.lse + int64_t(h) * p.T_q + row0;
        const float* dl_row = p.delta + int64_t(h) * p.T_q + row0;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int r = lane + 32 * x;
          lv[x] = r < nvq ? lse_row[r] : 0.f;
          dv[x] = r < nvq ? dl_row[r] : 0.f;
        }
        nvq_out = nvq;
      };
      float lv[4], dv[4], lv_n[4], dv_n[4];
      int nvq_cur, nvq_next = 0;
      fetch(0, lv, dv, nvq_cur);
      bool ok = true;
      for (int i = 0; ok && i < n_it; ++i) {
        const int st = i % ST;
        int g, row0, nvq, qpos0; bool diag;
        step(i, g, row0, nvq, diag, qpos0);
        const int h = hk * p.G + g;
        if (i + 1 < n_it) fetch(i + 1, lv_n, dv_n, nvq_next);
        // dO's stage is released first (after dV of the step that used it), then Q's (after dK)
        if (i >= ST) ok = mbar_wait(&bar.do_empty[st], ((i / ST) + 1) & 1, abortp, p.status);
        if (!ok) break;
        if (lane == 0) {
          mbar_expect_tx(&bar.do_full[st], kTileBytes);
          load_row_tile(sdO + st * kTileBytes, &maps.d_o, &bar.do_full[st], h, row0);
        }
        if (i >= ST) ok = mbar_wait(&bar.q_empty[st], ((i / ST) + 1) & 1, abortp, p.status);
        if (!ok) break;
        if (lane == 0) {
          mbar_expect_tx(&bar.q_full[st], kTileBytes);
          load_row_tile(sQ + st * kTileBytes, &maps.q, &bar.q_full[st], h, row0);
        }
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int r = lane + 32 * x;
          uint2 u = make_uint2(0xFF80u, 0u), d = make_uint2(0u, 0u);  // -inf: a row beyond the range sees nothing
          if (r < nvq_cur) {
            u = split3_bf16(-lv[x] * p.inv_scale);
            d = split3_bf16(-dv[x]);
          }
          uint8_t* lr = sLseX + st * kSliceBytes + slice_row_offset(r);
          uint8_t* dr = sDlX + st * kSliceBytes + slice_row_offset(r);
          *reinterpret_cast<uint4*>(lr) = make_uint4(u.x, u.y, 0u, 0u);
          *reinterpret_cast<uint4*>(lr + 128) = make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>(dr) = make_uint4(d.x, d.y, 0u, 0u);
          *reinterpret_cast<uint4*>(dr + 128) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) { mbar_arrive(&bar.q_full[st]); mbar_arrive(&bar.do_full[st]); }
#pragma unroll
        for (int x = 0; x < 4; ++x) { lv[x] = lv_n[x]; dv[x] = dv_n[x]; }
        nvq_cur = nvq_next;
      }
    }
  } else if (warp == 9) {
    // ======================= MMA issuer =======================
    // All 32 lanes walk the loop and wait on the barriers (warp-uniform control flow and
    // address arithmetic); only the tcgen05 instructions are issued, by lane 0.
    if (n_it > 0) {
      constexpr uint32_t idesc_kk = make_idesc(128, 128, 0, 0);  // S^T = K Q^T, dP^T = V dO^T
      constexpr uint32_t idesc_mn = make_idesc(128, 128, 0, 1);  // dV += P^T dO, dK += dS^T Q
      // descriptor low words (address >> 4 | LBO field); per K step only a constant is added
      const uint32_t k_lo = desc_lo(smem_u32(sK), 16), v_lo = desc_lo(smem_u32(sV), 16);
      const uint32_t q_lo = desc_lo(smem_u32(sQ), 16), g_lo = desc_lo(smem_u32(sdO), 16);                  // K-major view
      const uint32_t q_mn = desc_lo(smem_u32(sQ), kHalfBytes), g_mn = desc_lo(smem_u32(sdO), kHalfBytes);  // MN-major view
      const uint32_t ones_lo = slice_desc_lo(smem_u32(sOnes));
      const uint32_t lsex_lo = slice_desc_lo(smem_u32(sLseX)), dlx_lo = slice_desc_lo(smem_u32(sDlX));
      // D = A B^T (both K-major, K = 128) + ones (x) extra (the K = 16 slice with the per-row term)
      auto mma_kk = [&](uint32_t d, uint32_t a0, uint32_t b0, uint32_t extra_lo) {
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t off = (k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2;
            mma_ss_lo(d, a0 + off, b0 + off, idesc_kk, k > 0);
          }
          mma_ss_lohi(d, ones_lo, kSliceDescHi, extra_lo, kSliceDescHi, idesc_kk, 1u);
        }
      };
      // dV += P^T dO and dK += dS^T Q take A from tensor memory: packed bf16, 16 query rows per 8 columns,
      // rows 0-63 at +0, rows 64-127 at +64; B (dO, Q) MN-major in shared memory, K = 16 slice k at + k * 128
      auto commit = [&](uint64_t* b) { if (elect_one()) mma_commit(b); };
      auto wait = [&](uint64_t* b, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait_relaxed(b, parity, abortp, p.status));
      };
      bool ok = wait(&bar.kv_full, 0) && wait(&bar.q_full[0], 0) && wait(&bar.do_full[0], 0);
      if (ok) {
        tc_fence_after();
        mma_kk(tmem + TM_ST, k_lo, q_lo, lsex_lo);
        commit(&bar.s_full);
        mma_kk(tmem + TM_DPT, v_lo, g_lo, dlx_lo);
        commit(&bar.dp_full);
      }
      for (int i = 0; ok && i < n_it; ++i) {
        const uint32_t so = (i % ST) * (kTileBytes >> 4), so1 = ((i + 1) % ST) * (kTileBytes >> 4);
        const uint32_t sx1 = ((i + 1) % ST) * (kSliceBytes >> 4);
        if (lane == 0) s_beacon.at = i;   // before this step's five syncs (read only by warps that gave up)
        // dV(i) in four quarters of two K = 16 slices each, as the quarters of P^T(i) arrive
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          named_sync(kBarP + g, kBarThreads);
          tc_fence_after();
          if (elect_one()) {
            mma_ts_lo(tmem + TM_DV, tmem + TM_ST + g * 8, g_mn + so + g * 128, idesc_mn, g > 0 ? 1u : uint32_t(i > 0));
            mma_ts_lo(tmem + TM_DV, tmem + TM_ST + 64 + g * 8, g_mn + so + (4 + g) * 128, idesc_mn, 1u);
          }
        }
        commit(&bar.do_empty[i % ST]);          // dO(i) is done with: its stage may take dO(i + ST)
        if (i + 1 < n_it) {
          // the Q tile of step i+1 arrives late (two-stage ring): wait behind dV(i), not before it
          ok = wait(&bar.q_full[(i + 1) % ST], ((i + 1) / ST) & 1);
          if (!ok) break;
          mma_kk(tmem + TM_ST, k_lo, q_lo + so1, lsex_lo + sx1);
          commit(&bar.s_full);
        }
        // dO(i+1) landed long ago (its stage was released early)
        // dK(i) once all of dS^T(i) is stored (starting it on the first half measured slower: it is not on the
        // step's critical path, and every extra sync delays the MMA warp a little)
        named_sync(kBarDs, kBarThreads);
        if (i + 1 < n_it) ok = wait(&bar.do_full[(i + 1) % ST], ((i + 1) / ST) & 1);
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ts_lo(tmem + TM_DK, tmem + TM_DPT + (k >> 2) * 64 + (k & 3) * 8, q_mn + so + k * 128, idesc_mn,
                      k > 0 ? 1u : uint32_t(i > 0));
        }
        commit(&bar.q_empty[i % ST]);
        if (i + 1 < n_it) {
          mma_kk(tmem + TM_DPT, v_lo, g_lo + so1, dlx_lo + sx1);
          commit(&bar.dp_full);
        }
      }
      if (ok) commit(&bar.acc_full);
      if (lane == 0) s_beacon.left = 1;   // no sync follows on any path
    }
  } else {
    // ======================= softmax-backward warps (8) =======================
    const int wg = warp >> 2;                            // which 64 query columns of the 128
    const int keyrow = (warp & 3) * 32 + lane;           // key inside the tile = TMEM lane
    const uint32_t t_lane = tmem + (uint32_t((warp & 3) * 32) << 16);
    const f32x2 scale2 = make_f32x2(p.scale_log2, p.scale_log2);
    bool ok = true;
    for (int i = 0; i < n_it; ++i) {
      int g, row0, nvq, qpos0; bool diag;
      step(i, g, row0, nvq, diag, qpos0);
      float pr[64];  // this thread's P^T values, kept for the second half-step
      // ---- half-step 1: P^T = exp2(c S^T_aug); -LSE / scale is already inside S^T_aug, and
      //      a query row beyond the valid range carries -inf there, so its column comes out 0 ----
      // (a warp that gave up on a wait still walks the loop and performs every arrival on the named
      // barriers - once per step, and for step i only when the MMA warp has reached step i, see
      // StepBeacon - so that the MMA warp is never left waiting at one)
      if (ok) ok = mbar_wait(&bar.s_full, i & 1, abortp, p.status);
      int quarters_sent = 0;
      if (ok) {
        tc_fence_after();
        uint32_t s[2][32];
        tmem_ld32(t_lane + TM_ST + wg * 64, s[0]);
        tmem_ld32(t_lane + TM_ST + wg * 64 + 32, s[1]);
        tmem_wait_ld();
        // software pipeline over groups of 16 query rows: the exp2 of group g+1 (MUFU pipe) is issued
        // before group g is masked, packed and stored
        auto exps = [&](int g) {
          const int c = g >> 1, i0 = (g & 1) * 16;
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            float a0, a1;
            split_f32x2(mul2(make_f32x2(s[c][i0 + i], s[c][i0 + i + 1]), scale2), a0, a1);
            pr[g * 16 + i] = ex2(a0);
            pr[g * 16 + i + 1] = ex2(a1);
          }
        };
        exps(0);
        uint32_t pk[16];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          if (g + 1 < 4) exps(g + 1);
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            float p0 = pr[g * 16 + i], p1 = pr[g * 16 + i + 1];
            if (diag) {  // the tile that holds the keys' own rows: a key is visible from its own row on
              const int col = wg * 64 + g * 16 + i;
              p0 = (qpos0 + col >= keyrow) ? p0 : 0.f;
              p1 = (qpos0 + col + 1 >= keyrow) ? p1 : 0.f;
              pr[g * 16 + i] = p0;
              pr[g * 16 + i + 1] = p1;
            }
            pk[(g & 1) * 8 + (i >> 1)] = pack_bf16(p0, p1);
          }
          // 16 of the warp's 64 query rows are stored: dV may start on them
          tmem_st8(t_lane + TM_ST + wg * 64 + g * 8, pk + (g & 1) * 8);
          tmem_wait_st();
          tc_fence_before();
          named_arrive(kBarP + g, kBarThreads);
          quarters_sent = g + 1;
        }
      }
      if (!ok) {   // gave up on a wait: the remaining arrivals of this step, in step with the MMA warp
        if (!beacon_reached(&s_beacon, i)) break;   // the MMA warp has left its loop: nobody syncs any more
        for (int g = quarters_sent; g < 4; ++g) named_arrive(kBarP + g, kBarThreads);
      }
      // ---- half-step 2: dS^T = P^T o dP^T_aug (-D is already inside) ----
      if (ok) ok = mbar_wait(&bar.dp_full, i & 1, abortp, p.status);
      if (ok) {
        tc_fence_after();
        uint32_t dp[2][32];
        tmem_ld32(t_lane + TM_DPT + wg * 64, dp[0]);
        tmem_ld32(t_lane + TM_DPT + wg * 64 + 32, dp[1]);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int x = 0; x < 32; x += 2) {
            float d0, d1;
            split_f32x2(mul2(make_f32x2(pr[c * 32 + x], pr[c * 32 + x + 1]), make_f32x2(dp[c][x], dp[c][x + 1])), d0, d1);
            pk[x >> 1] = pack_bf16(d0, d1);
          }
          tmem_st16(t_lane + TM_DPT + wg * 64 + c * 16, pk);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      if (!ok && !beacon_reached(&s_beacon, i)) break;
      named_arrive(kBarDs, kBarThreads);
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
    ok = make_map_bf16_2d(&m.q, a.q, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, 128) &&
         make_map_bf16_2d(&m.d_o, a.d_o, uint64_t(P.Hq) * 128, uint64_t(P.T_q), uint64_t(P.Hq) * 256, 128);
  }
  if (!ok) return PSRL_ERR_CUDA;
  const size_t smem = size_t(2 + 2 * ST) * kTileBytes + size_t(1 + 2 * ST) * kSliceBytes + 1024;
  static bool attr_set[64] = {};
  cudaError_t e = ensure_dynamic_smem(dkv_kernel, smem, attr_set);
  if (e != cudaSuccess) return fail(e);
  Params p{};
  p.blob = P.dev;
  p.off_kvi = H.off_kvi; p.off_kvt = H.off_kvt; p.off_page_slot = H.off_page_slot; p.off_split = H.off_split;
  p.Hq = P.Hq; p.Hkv = P.Hkv; p.G = P.Hq / P.Hkv; p.T_q = P.T_q;
  p.cap = cap; p.scale = a.scale; p.scale_log2 = a.scale * kLog2e; p.inv_scale = 1.f / a.scale;
  p.lse = a.lse_in; p.delta = a.delta; p.slabs = a.slabs;
  p.dk = static_cast<__nv_bfloat16*>(a.dk_pool); p.dv = static_cast<__nv_bfloat16*>(a.dv_pool);
  p.status = a.status;
  p.chunk = block_order_chunk(int64_t(P.kv_items.size()), resident_ctas(), 1);
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

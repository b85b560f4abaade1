// Merge of partial results (bf16 path).  A query row whose keys were divided
// between several work items - packed items over a cascaded ancestor's KV tiles,
// split into chunks over CTAs, plus the row's own item - has one fp32 partial row
// per item.  The forward combines them by log-sum-exp,
//   L = ln sum_p exp(L_p),   O = sum_p exp(L_p - L) O_p,
// which equals the softmax over the union of the parts' keys (the paper's tree
// mask, Sec. 2.5, only fixes WHICH keys a row sees, not how they are grouped);
// the backward adds the parts' dQ.  Parts are always taken in the order of the
// row's merge list, so results are bitwise reproducible.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "kernels.h"

namespace psrl {
namespace {

constexpr int kWarps = 8;

struct MergeParams {
  const int32_t *merge_row, *merge_off, *merge_parts;
  int32_t n_merge_rows, Hq, T_q;
  const float* part;
  const float* part_lse;
  __nv_bfloat16* out;   // O or dQ, [T_q][Hq][128]
  float* lse;           // [Hq][T_q] (forward)
  float scale;          // dQ: softmax scale
};

__device__ __forceinline__ void store4(__nv_bfloat16* dst, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(dst) = u;
}

// one warp per (merged row, query head); lane l owns dims [4l, 4l+4)
template <bool kFwd>
__global__ void __launch_bounds__(kWarps * 32) merge_kernel(const MergeParams p) {
  const int lane = threadIdx.x & 31;
  const int64_t unit = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5);
  if (unit >= int64_t(p.n_merge_rows) * p.Hq) return;
  const int i = int(unit / p.Hq), h = int(unit % p.Hq);
  const int row = p.merge_row[i];
  const int b = p.merge_off[i], e = p.merge_off[i + 1];
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  // Lanes first fetch the part ids (and LSEs) side by side, 32 parts at a time, so that the loop
  // over the parts' rows has its addresses and weights ready and its loads are independent.
  // Sums are formed in list order by every lane alike: no dependence on the warp's scheduling.
  float m = -CUDART_INF_F, den = 0.f;
  if (kFwd) {
    for (int x0 = b; x0 < e; x0 += 32) {
      const int x = x0 + lane;
      const float l = x < e ? p.part_lse[int64_t(p.merge_parts[x]) * p.Hq + h] : -CUDART_INF_F;
      float mm = l;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
      m = fmaxf(m, mm);
    }
    for (int x0 = b; x0 < e; x0 += 32) {
      const int x = x0 + lane;
      const float w = x < e ? __expf(p.part_lse[int64_t(p.merge_parts[x]) * p.Hq + h] - m) : 0.f;
      for (int y = 0; y < min(32, e - x0); ++y) den += __shfl_sync(0xffffffffu, w, y);   // list order
    }
  }
  const float inv = kFwd ? 1.f / den : 1.f;
  for (int x0 = b; x0 < e; x0 += 32) {
    const int x = x0 + lane;
    const int64_t my_pr = x < e ? int64_t(p.merge_parts[x]) * p.Hq + h : 0;
    const float my_w = (kFwd && x < e) ? __expf(p.part_lse[my_pr] - m) * inv : 1.f;
    const int n = min(32, e - x0);
#pragma unroll 4
    for (int y = 0; y < n; ++y) {
      const int64_t pr = __shfl_sync(0xffffffffu, my_pr, y);
      const float w = __shfl_sync(0xffffffffu, my_w, y);
      const float4 v = *reinterpret_cast<const float4*>(p.part + pr * 128 + lane * 4);
      acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
      acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
    }
  }
  if (kFwd) {
    if (lane == 0) p.lse[int64_t(h) * p.T_q + row] = m + __logf(den);
  } else {
    acc.x *= p.scale; acc.y *= p.scale; acc.z *= p.scale; acc.w *= p.scale;
  }
  store4(p.out + (int64_t(row) * p.Hq + h) * 128 + lane * 4, acc);
}

template <bool kFwd>
psrl_status_t launch(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const DeviceHeader& H = P.hdr;
  if (H.n_merge_rows == 0) return PSRL_OK;
  MergeParams p{};
  p.merge_row = P.dev + H.off_merge_row; p.merge_off = P.dev + H.off_merge_off; p.merge_parts = P.dev + H.off_merge_parts;
  p.n_merge_rows = H.n_merge_rows; p.Hq = P.Hq; p.T_q = P.T_q;
  p.part = a.part; p.part_lse = a.part_lse;
  p.out = static_cast<__nv_bfloat16*>(kFwd ? a.o_out : a.d_q);
  p.lse = a.lse_out;
  p.scale = a.scale;
  const int64_t units = int64_t(H.n_merge_rows) * P.Hq;
  const int64_t grid = (units + kWarps - 1) / kWarps;
  if (grid > INT32_MAX) return PSRL_ERR_SHAPE;
  merge_kernel<kFwd><<<unsigned(grid), kWarps * 32, 0, a.stream>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_last_cuda_error(e); return PSRL_ERR_CUDA; }
  return PSRL_OK;
}

}  // namespace

psrl_status_t merge_fwd_bf16(const AttnArgs& a) { return launch<true>(a); }
psrl_status_t merge_dq_bf16(const AttnArgs& a) { return launch<false>(a); }

}  // namespace psrl

// bf16 tree attention backward: the D pre-pass and the order of the three kernels.
//
// All three are deterministic (every output element has one owner that sums its
// contributions in a fixed order; no atomics):
//   delta_kernel  D_i = dO_i . O_i                      HBM-bound pre-pass (this file)
//   dq_kernel     query-stationary, 3 contractions      attn_bf16_dq.cu
//   dkv_kernel    key-stationary, 4 contractions, with the fixed-order reduce of split
//                 tiles                                 attn_bf16_dkv.cu
// The price of determinism without a cross-CTA ordered reduction is that S and dP are
// computed in both kernels: 7 contractions are executed for the 5 the backward needs.
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

}  // namespace

psrl_status_t bwd_bf16(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const int64_t cap = a.pool_capacity;
  if (int64_t(P.Hkv) * cap > INT32_MAX || int64_t(P.Hq) * 128 > INT32_MAX) return PSRL_ERR_SHAPE;
  if (P.T_q > 0 && (g_bwd_phase_mask & 1)) {
    // ---- D = rowsum(dO o O) ----
    const int64_t units = int64_t(P.T_q) * P.Hq;
    delta_kernel<<<unsigned((units + 7) / 8), 256, 0, a.stream>>>(
        P.T_q, P.Hq, static_cast<const __nv_bfloat16*>(a.o), static_cast<const __nv_bfloat16*>(a.d_o), a.delta);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
      set_last_cuda_error(e);
      return PSRL_ERR_CUDA;
    }
  }
  if (g_bwd_phase_mask & 2) {
    // ---- dQ (attn_bf16_dq.cu) ----
    const psrl_status_t st = dq_bf16(a);
    if (st != PSRL_OK) return st;
  }
  if (g_bwd_phase_mask & 4) {
    // ---- dK, dV (attn_bf16_dkv.cu) ----
    const psrl_status_t st = dkv_bf16(a);
    if (st != PSRL_OK) return st;
  }
  return PSRL_OK;
}

}  // namespace psrl

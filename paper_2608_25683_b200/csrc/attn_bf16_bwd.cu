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

#include <mutex>

#include "attn_bf16_common.cuh"
#include "kernels.h"
#include "tma.h"

namespace psrl {
namespace {
using namespace sm100;

// dQ and dK/dV are independent of one another (both read Q, K, V, dO, LSE, D; they write disjoint outputs and
// disjoint parts of the workspace), so the backward forks: dK/dV runs on a side stream of the library beside dQ
// and joins the caller's stream again.  The block scheduler then fills the SMs that the last dQ CTAs leave
// idle with dK/dV CTAs, and the two kernels' set-up and ramp overlap - which is most of the time of a
// launch-bound step (the small-suffix case: 0.108 -> 0.101 ms per step).  Only plans of a few waves fork:
// on large ones the two kernels' CTAs interleave for the whole run and evict each other's tiles from the L2
// (c5: 784 -> 820-830 ms per step).  One side stream and two events per device, created on the first
// backward of that device that forks.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
  bool ok = false;
};
SideStream g_side[64];
std::mutex g_side_mu;        // serialises the fork / join enqueue sequences of a device
std::mutex g_side_create_mu; // guards the one-time creation
SideStream* side_stream() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_side_create_mu);
  SideStream& s = g_side[dev];
  if (!s.ok) {
    if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    s.ok = true;
  }
  return &s;
}

// ============================================================================ delta
// 16 threads per (row, head): 16 bytes of O and of dO each, in memory order (a block reads 4 KB of each
// tensor contiguously); D goes to its [Hq, T_q] layout.
__global__ void __launch_bounds__(256)
delta_kernel(int T_q, int Hq, const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
             float* __restrict__ delta) {
  const int64_t i = int64_t(blockIdx.x) * 256 + threadIdx.x;   // 16-byte vector index
  const int64_t unit = i >> 4;                                 // = r * Hq + h
  const bool live = unit < int64_t(T_q) * Hq;
  float s = 0.f;
  if (live) {
    const uint4 a = reinterpret_cast<const uint4*>(o)[i];
    const uint4 b = reinterpret_cast<const uint4*>(d_o)[i];
    const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&av[k]));
      const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bv[k]));
      s = fmaf(x.x, y.x, s);
      s = fmaf(x.y, y.y, s);
    }
  }
#pragma unroll
  for (int o2 = 8; o2 > 0; o2 >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o2);
  if (live && (threadIdx.x & 15) == 0) {
    const int r = int(unit / Hq), h = int(unit % Hq);
    delta[int64_t(h) * T_q + r] = s;
  }
}

}  // namespace

psrl_status_t bwd_bf16(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const int64_t cap = a.pool_capacity;
  if (int64_t(P.Hkv) * cap > INT32_MAX || int64_t(P.Hq) * 128 > INT32_MAX) return PSRL_ERR_SHAPE;
  if (P.T_q > 0 && (a.phases & 1)) {
    // ---- D = rowsum(dO o O) ----
    const int64_t units = int64_t(P.T_q) * P.Hq;
    delta_kernel<<<unsigned((units + 15) / 16), 256, 0, a.stream>>>(
        P.T_q, P.Hq, static_cast<const __nv_bfloat16*>(a.o), static_cast<const __nv_bfloat16*>(a.d_o), a.delta);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
      set_last_cuda_error(e);
      return PSRL_ERR_CUDA;
    }
  }
  // few waves: the CTAs of both kernels together are at most kForkWaves per SM
  constexpr int64_t kForkWaves = 8;
  const int64_t ctas = int64_t(P.q_tiles.size()) * P.Hq + int64_t(P.kv_items.size()) * P.Hkv;
  const bool small = P.T_q > 0 && ctas <= kForkWaves * resident_ctas();
  SideStream* side = (a.fork && small && (a.phases & 6) == 6) ? side_stream() : nullptr;
  if (side) {
    // ---- dK, dV on the side stream, dQ on the caller's; join ----
    // The two events are shared by every call on the device: the whole record / wait sequence is enqueued under
    // the lock, so that calls from several host threads cannot pair one call's wait with another call's record.
    std::lock_guard<std::mutex> lock(g_side_mu);
    cudaError_t e = cudaEventRecord(side->fork, a.stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PSRL_ERR_CUDA; }
    AttnArgs b = a;
    b.stream = side->stream;
    psrl_status_t st = dkv_bf16(b);
    if (st != PSRL_OK) return st;
    e = cudaEventRecord(side->join, side->stream);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PSRL_ERR_CUDA; }
    st = dq_bf16(a);
    e = cudaStreamWaitEvent(a.stream, side->join, 0);   // join even if dQ failed to launch
    if (st != PSRL_OK) return st;
    if (e != cudaSuccess) { set_last_cuda_error(e); return PSRL_ERR_CUDA; }
    return PSRL_OK;
  }
  if (a.phases & 2) {
    // ---- dQ (attn_bf16_dq.cu) ----
    const psrl_status_t st = dq_bf16(a);
    if (st != PSRL_OK) return st;
  }
  if (a.phases & 4) {
    // ---- dK, dV (attn_bf16_dkv.cu) ----
    const psrl_status_t st = dkv_bf16(a);
    if (st != PSRL_OK) return st;
  }
  return PSRL_OK;
}

}  // namespace psrl

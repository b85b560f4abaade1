// K/V scatter into the paged pools and gather back (token-major <-> pool layout), the HBM-bound
// neighbours of the attention calls (paper Sec. 6: the KV manager's blocks are what the attention
// backend reads).  One 16-byte vector per thread; a token row of one head is contiguous on both
// sides, so loads and stores are fully coalesced.
#include <cuda_runtime.h>

#include "../../include/psrl.h"
#include "kernels.h"

namespace psrl {
namespace {

// vecs = 16-byte vectors per (token, head) row
template <bool kScatter>
__global__ void __launch_bounds__(256) pack_kernel(const int32_t* __restrict__ tok_slot, int64_t T, int Hkv, int vecs,
                                                   int64_t cap, const uint4* __restrict__ k_src,
                                                   const uint4* __restrict__ v_src, uint4* __restrict__ k_dst,
                                                   uint4* __restrict__ v_dst) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t per_tok = int64_t(Hkv) * vecs;
  if (i >= T * per_tok) return;
  const int64_t t = i / per_tok;
  const int r = int(i % per_tok), h = r / vecs, x = r % vecs;
  const int64_t tok_at = i;                                              // [t][h][x]
  const int64_t pool_at = (int64_t(h) * cap + tok_slot[t]) * vecs + x;   // [h][slot][x]
  const int64_t src = kScatter ? tok_at : pool_at, dst = kScatter ? pool_at : tok_at;
  if (k_src) k_dst[dst] = k_src[src];
  if (v_src) v_dst[dst] = v_src[src];
}

template <bool kScatter>
psrl_status_t launch(const Plan& P, const void* k_src, const void* v_src, void* k_dst, void* v_dst, int64_t cap,
                     cudaStream_t stream) {
  const int es = P.dtype == PSRL_BF16 ? 2 : 4;
  const int vecs = P.d * es / 16;
  const int64_t n = int64_t(P.T) * P.Hkv * vecs;
  if (n == 0) return PSRL_OK;
  const int64_t grid = (n + 255) / 256;
  if (grid > INT32_MAX) return PSRL_ERR_SHAPE;
  pack_kernel<kScatter><<<unsigned(grid), 256, 0, stream>>>(
      P.dev + P.hdr.off_tok_slot, P.T, P.Hkv, vecs, cap, static_cast<const uint4*>(k_src),
      static_cast<const uint4*>(v_src), static_cast<uint4*>(k_dst), static_cast<uint4*>(v_dst));
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_last_cuda_error(e); return PSRL_ERR_CUDA; }
  return PSRL_OK;
}

bool ok16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace psrl


extern "C" {

psrl_status_t psrl_kv_scatter(const psrl_plan_t* plan, const void* k_tok, const void* v_tok, void* k_pool,
                              void* v_pool, int64_t pool_capacity, void* stream) {
  if (!plan || !plan->p) return PSRL_ERR_INVALID_ARG;
  const psrl::Plan& P = *plan->p;
  if ((k_tok && !k_pool) || (v_tok && !v_pool) || !psrl::ok16(k_tok) || !psrl::ok16(v_tok) || !psrl::ok16(k_pool) ||
      !psrl::ok16(v_pool))
    return PSRL_ERR_INVALID_ARG;
  if (pool_capacity < P.pool_slots) return PSRL_ERR_SHAPE;
  if (!P.dev) return PSRL_ERR_WORKSPACE;
  return psrl::launch<true>(P, k_tok, v_tok, k_pool, v_pool, pool_capacity, static_cast<cudaStream_t>(stream));
}

psrl_status_t psrl_kv_gather(const psrl_plan_t* plan, const void* k_pool, const void* v_pool, int64_t pool_capacity,
                             void* k_tok, void* v_tok, void* stream) {
  if (!plan || !plan->p) return PSRL_ERR_INVALID_ARG;
  const psrl::Plan& P = *plan->p;
  if ((k_pool && !k_tok) || (v_pool && !v_tok) || !psrl::ok16(k_tok) || !psrl::ok16(v_tok) || !psrl::ok16(k_pool) ||
      !psrl::ok16(v_pool))
    return PSRL_ERR_INVALID_ARG;
  if (pool_capacity < P.pool_slots) return PSRL_ERR_SHAPE;
  if (!P.dev) return PSRL_ERR_WORKSPACE;
  return psrl::launch<false>(P, k_pool, v_pool, k_tok, v_tok, pool_capacity, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

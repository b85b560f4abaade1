// Launchers of the CUDA kernels (internal; the public surface is include/psrl.h).
#pragma once
#include <cuda_runtime.h>

#include "plan.h"

namespace psrl {

// Layout of the caller's workspace: [0, 256) control words (word 0 = device status), then
//   forward:  partial O rows, their LSE
//   backward: D = rowsum(dO o O) as fp32 [Hq, T_q], partial dV/dK slabs, partial dQ rows.
constexpr size_t kWsHeaderBytes = 256;
// Control words 16..18: per-kernel counters of CTAs whose producers have issued their last load
// (forward, dQ, dK/dV); zeroed with the header before every call.
constexpr int kWsCtrFwd = 16, kWsCtrDq = 17, kWsCtrDkv = 18;
// CTAs of a one-CTA-per-SM kernel that are resident at once (the device's SM count).
int resident_ctas();
// After D: fp32 partial dV/dK slabs of split KV tiles, [slab][kv head][dV, dK][128][128].
constexpr size_t kSlabBytes = size_t(2) * 128 * 128 * sizeof(float);
inline size_t ws_delta_bytes(const Plan& P) {
  return (size_t(P.Hq) * size_t(P.T_q) * sizeof(float) + 255) / 256 * 256;
}
inline size_t ws_slab_bytes(const Plan& P) {
  return P.dtype == PSRL_BF16 ? size_t(P.n_slabs) * size_t(P.Hkv) * kSlabBytes : 0;
}

// Partial results of the forward / dQ items that do not own their rows (cascaded prefixes,
// split-KV): fp32 [n_part_rows][Hq][128] (normalised O, or unscaled dQ), and for the
// forward the parts' LSE as fp32 [n_part_rows][Hq] behind it.
inline size_t ws_part_bytes(const Plan& P) {
  return P.dtype == PSRL_BF16 ? size_t(P.n_part_rows) * size_t(P.Hq) * 128 * sizeof(float) : 0;
}
inline size_t ws_part_lse_bytes(const Plan& P) {
  return P.dtype == PSRL_BF16 ? (size_t(P.n_part_rows) * size_t(P.Hq) * sizeof(float) + 255) / 256 * 256 : 0;
}

struct AttnArgs {
  const Plan* plan;
  const void *q, *k_pool, *v_pool, *o, *d_o;
  const float* lse_in;
  void *o_out, *d_q, *dk_pool, *dv_pool;
  float* lse_out;
  float* delta;  // D, in the workspace
  float* slabs;  // partial dV/dK slabs, in the workspace (bf16 path)
  float* part;   // partial O (forward) or dQ (backward) rows, in the workspace (bf16 path)
  float* part_lse;  // LSE of the partial O rows (forward)
  int* status;   // device status word
  int64_t pool_capacity;
  float scale;
  cudaStream_t stream;
  int phases = 7;  // backward kernels to launch: bit 0 D pre-pass, bit 1 dQ, bit 2 dK/dV (7 everywhere but in benchmarks)
  bool fork = true;  // bf16 backward: dK/dV on an internal side stream beside dQ (false: everything on `stream`)
};

// Pointer checks of the entry points: non-NULL and aligned; Q-shaped tensors of a plan without any
// query row are empty, so NULL is accepted for them.
inline bool ptr_aligned(const void* p, size_t a) { return p && (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline bool ptr_aligned_q(const void* p, size_t a, const Plan& P) { return (P.T_q == 0 && !p) || ptr_aligned(p, a); }

// fp32 SIMT path (exact-arithmetic parity path; head_dim 64 or 128)
cudaError_t fwd_f32(const AttnArgs& a);
cudaError_t bwd_f32(const AttnArgs& a);
// bf16 tensor-core path (tcgen05 / TMEM / TMA; head_dim 128)
psrl_status_t fwd_bf16(const AttnArgs& a);
psrl_status_t bwd_bf16(const AttnArgs& a);
psrl_status_t dq_bf16(const AttnArgs& a);   // the dQ part of bwd_bf16
psrl_status_t dkv_bf16(const AttnArgs& a);  // the dK/dV part of bwd_bf16 (+ reduce of split tiles)
psrl_status_t merge_fwd_bf16(const AttnArgs& a);  // O, LSE of the rows assembled from partial results
psrl_status_t merge_dq_bf16(const AttnArgs& a);   // dQ of those rows

void set_last_cuda_error(cudaError_t e);

// Raises a kernel's dynamic shared-memory limit once per device (the attribute belongs to the
// function on the current device; a process may drive several GPUs).
template <class Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, size_t bytes, bool (&done)[64]) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes));
  if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
  return e;
}

}  // namespace psrl

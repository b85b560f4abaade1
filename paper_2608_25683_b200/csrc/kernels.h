// Launchers of the CUDA kernels (internal; the public surface is include/psrl.h).
#pragma once
#include <cuda_runtime.h>

#include "plan.h"

namespace psrl {

// Layout of the caller's workspace: [0, 256) control words (word 0 = device
// status), then D = rowsum(dO o O) as fp32 [Hq, T_q] for the backward.
constexpr size_t kWsHeaderBytes = 256;

struct AttnArgs {
  const Plan* plan;
  const void *q, *k_pool, *v_pool, *o, *d_o;
  const float* lse_in;
  void *o_out, *d_q, *dk_pool, *dv_pool;
  float* lse_out;
  float* delta;  // D, in the workspace
  int* status;   // device status word
  int64_t pool_capacity;
  float scale;
  cudaStream_t stream;
};

// fp32 SIMT path (exact-arithmetic parity path; head_dim 64 or 128)
cudaError_t fwd_f32(const AttnArgs& a);
cudaError_t bwd_f32(const AttnArgs& a);
// bf16 tensor-core path (tcgen05 / TMEM / TMA; head_dim 128)
psrl_status_t fwd_bf16(const AttnArgs& a);
psrl_status_t bwd_bf16(const AttnArgs& a);

void set_last_cuda_error(cudaError_t e);

// Which backward kernels to launch (profiling aid): bit 0 delta, bit 1 dQ, bit 2 dK/dV.
extern int g_bwd_phase_mask;

}  // namespace psrl

// psrl_tree_attn_bwd_static: the backward pass for callers that must not
// allocate device memory.
//
// The regular backward needs a caller-provided workspace (a status header and
// D = rowsum(dO o O), one float per query row and head).  Some callers cannot
// supply one: code running where the CUDA allocator must not be touched (a
// latency-critical serving loop that forbids cudaMalloc because it
// synchronises the device, a host whose memory pool is owned by another
// framework, a plug-in loaded into a process with a fixed memory budget).  For
// them this file reserves the workspace at load time, inside the library image:
// a file-scope __device__ array that every GPU which loads the library holds
// until the process exits.
//
// `g_scratch` below is, in host code, only a host-side stand-in for the device
// array: passing it to a kernel would hand the GPU a host address.  The device
// address is looked up once per device with cudaGetSymbolAddress (with that
// device current) and that pointer is what the kernels receive.
#include <cuda_runtime.h>

#include <mutex>

#include "kernels.h"
#include "plan.h"

namespace {

// The array holds the status header, D (one float per query row and head), and - for plans whose schedule
// splits heavy KV tiles or assembles rows from partial results - the fp32 slabs and partial dQ rows as well.
constexpr size_t kMaxDeltaFloats = size_t(4) << 20;  // n_q_heads * T_q <= 4,194,304 (16 MiB of fp32) at most
constexpr size_t kScratchBytes = psrl::kWsHeaderBytes + kMaxDeltaFloats * sizeof(float);
static_assert(kScratchBytes == PSRL_BWD_STATIC_SCRATCH_BYTES, "the header states the array's size");

static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_mu;

// Device address of the scratch array on the CURRENT device (looked up on the
// first call per device, cached afterwards).  Returns nullptr and records the
// CUDA error on failure.
void* scratch_on_current_device() {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    psrl::set_last_cuda_error(e != cudaSuccess ? e : cudaErrorInvalidDevice);
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_scratch);
    if (e != cudaSuccess || !ptr) {
      psrl::set_last_cuda_error(e != cudaSuccess ? e : cudaErrorInvalidSymbol);
      return nullptr;
    }
    g_scratch_addr[dev] = ptr;
  }
  return g_scratch_addr[dev];
}

}  // namespace

extern "C" psrl_status_t psrl_tree_attn_bwd_static(const psrl_plan_t* plan, const void* q, const void* k_pool,
                                                   const void* v_pool, int64_t pool_capacity, const void* o,
                                                   const float* lse, const void* d_o, void* d_q, void* dk_pool,
                                                   void* dv_pool, float softmax_scale, void** status_workspace,
                                                   void* stream) {
  if (status_workspace) *status_workspace = nullptr;
  if (!plan || !plan->p) return PSRL_ERR_INVALID_ARG;
  const psrl::Plan& P = *plan->p;
  // the same pointer rules as psrl_tree_attn_bwd: Q-shaped tensors of a plan without query rows may be NULL
  using psrl::ptr_aligned;
  using psrl::ptr_aligned_q;
  if (!ptr_aligned_q(q, 16, P) || !ptr_aligned(k_pool, 16) || !ptr_aligned(v_pool, 16) || !ptr_aligned_q(o, 16, P) ||
      !ptr_aligned_q(lse, 16, P) || !ptr_aligned_q(d_o, 16, P) || !ptr_aligned_q(d_q, 16, P) ||
      !ptr_aligned(dk_pool, 16) || !ptr_aligned(dv_pool, 16))
    return PSRL_ERR_INVALID_ARG;
  if (pool_capacity < P.pool_slots) return PSRL_ERR_SHAPE;
  if (!P.dev) return PSRL_ERR_WORKSPACE;  // plan not uploaded
  // the built-in scratch is a fixed size: a plan fits when the workspace the regular backward would ask for
  // (psrl_bwd_workspace_bytes: header + D + split slabs + partial dQ rows) fits; larger ones must use
  // psrl_tree_attn_bwd
  if (size_t(P.Hq) * size_t(P.T_q) > kMaxDeltaFloats) return PSRL_ERR_WORKSPACE;
  if (psrl::kWsHeaderBytes + psrl::ws_delta_bytes(P) + psrl::ws_slab_bytes(P) + psrl::ws_part_bytes(P) > kScratchBytes)
    return PSRL_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(scratch_on_current_device());
  if (!ws) return PSRL_ERR_CUDA;
  if (status_workspace) *status_workspace = ws;

  psrl::AttnArgs a{};
  a.plan = &P; a.q = q; a.k_pool = k_pool; a.v_pool = v_pool; a.o = o; a.lse_in = lse; a.d_o = d_o;
  a.d_q = d_q; a.dk_pool = dk_pool; a.dv_pool = dv_pool;
  a.status = reinterpret_cast<int*>(ws);
  a.delta = reinterpret_cast<float*>(ws + psrl::kWsHeaderBytes);
  a.slabs = reinterpret_cast<float*>(ws + psrl::kWsHeaderBytes + psrl::ws_delta_bytes(P));
  a.part = reinterpret_cast<float*>(ws + psrl::kWsHeaderBytes + psrl::ws_delta_bytes(P) + psrl::ws_slab_bytes(P));
  a.pool_capacity = pool_capacity; a.scale = softmax_scale; a.stream = static_cast<cudaStream_t>(stream);
  a.fork = false;   // no side stream here: creating one is a resource allocation this entry point promises not to make
  // the array keeps the previous call's contents: the status header must start at zero;
  // D is fully rewritten by the pre-pass before anything reads it
  cudaError_t e = cudaMemsetAsync(ws, 0, psrl::kWsHeaderBytes, a.stream);
  if (e != cudaSuccess) {
    psrl::set_last_cuda_error(e);
    return PSRL_ERR_CUDA;
  }
  if (P.dtype == PSRL_F32) {
    e = psrl::bwd_f32(a);
    if (e != cudaSuccess) {
      psrl::set_last_cuda_error(e);
      return PSRL_ERR_CUDA;
    }
    return PSRL_OK;
  }
  return psrl::bwd_bf16(a);
}

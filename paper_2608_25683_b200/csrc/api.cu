// C ABI of libpsrl.so: argument checking and dispatch.  See include/psrl.h.
#include <cuda_runtime.h>

#include <cstring>
#include <new>

#include "kernels.h"
#include "plan.h"

namespace psrl {
static thread_local cudaError_t g_last_cuda = cudaSuccess;
void set_last_cuda_error(cudaError_t e) { g_last_cuda = e; }
int resident_ctas() {
  static thread_local int n[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (n[dev] == 0 && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n[dev] = 148;
  return n[dev];
}
}  // namespace psrl

namespace {

bool aligned(const void* p, size_t a) { return psrl::ptr_aligned(p, a); }
bool aligned_q(const void* p, size_t a, const psrl::Plan& P) { return psrl::ptr_aligned_q(p, a, P); }

size_t ws_bytes(const psrl::Plan& P, bool bwd) {
  size_t n = psrl::kWsHeaderBytes;
  if (bwd) n += psrl::ws_delta_bytes(P) + psrl::ws_slab_bytes(P) + psrl::ws_part_bytes(P);
  else n += psrl::ws_part_bytes(P) + psrl::ws_part_lse_bytes(P);
  return n;
}

psrl_status_t cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return PSRL_OK;
  psrl::set_last_cuda_error(e);
  return PSRL_ERR_CUDA;
}

}  // namespace

extern "C" {

psrl_status_t psrl_plan_build(const psrl_tree_desc_t* desc, psrl_plan_t** out_plan) {
  if (!out_plan) return PSRL_ERR_INVALID_ARG;
  *out_plan = nullptr;
  if (!desc) return PSRL_ERR_INVALID_ARG;
  psrl::Plan* p = nullptr;
  psrl_status_t st = psrl::build_plan(*desc, p);
  if (st != PSRL_OK) return st;
  psrl_plan* h = new (std::nothrow) psrl_plan{p};
  if (!h) {
    delete p;
    return PSRL_ERR_HOST_OOM;
  }
  *out_plan = h;
  return PSRL_OK;
}

psrl_status_t psrl_plan_view(const psrl_plan_t* plan, psrl_plan_view_t* v) {
  if (!plan || !plan->p || !v) return PSRL_ERR_INVALID_ARG;
  const psrl::Plan& P = *plan->p;
  std::memset(v, 0, sizeof(*v));
  v->n_seg = P.n_seg; v->n_groups = P.n_groups; v->n_pages = P.n_pages; v->n_samples = P.n_samples;
  v->max_depth = P.max_depth; v->T = P.T; v->T_q = P.T_q; v->pool_slots = P.pool_slots;
  v->flat_tokens = P.flat_tokens; v->tree_pairs = P.tree_pairs; v->flat_pairs = P.flat_pairs;
  v->n_anc = static_cast<int32_t>(P.anc_list.size());
  v->n_bt = static_cast<int32_t>(P.bt_pages.size());
  v->canon_of_input = P.canon_of_input.data(); v->input_of_canon = P.input_of_canon.data();
  v->seg_group = P.seg_group.data(); v->seg_bs = P.seg_bs.data(); v->seg_parent = P.seg_parent.data();
  v->seg_len = P.seg_len.data(); v->seg_flags = P.seg_flags.data(); v->seg_depth = P.seg_depth.data();
  v->seg_anc_tokens = P.seg_anc_tokens.data(); v->seg_sub_end = P.seg_sub_end.data();
  v->seg_tok_off = P.seg_tok_off.data(); v->seg_q_off = P.seg_q_off.data();
  v->seg_refcount = P.seg_refcount.data(); v->anc_off = P.anc_off.data(); v->anc_list = P.anc_list.data();
  v->seg_first_page = P.seg_first_page.data(); v->seg_n_pages = P.seg_n_pages.data();
  v->page_seg = P.page_seg.data(); v->page_bs = P.page_bs.data(); v->page_valid = P.page_valid.data();
  v->page_pos = P.page_pos.data(); v->page_refcount = P.page_refcount.data(); v->page_slot = P.page_slot.data();
  v->bt_off = P.bt_off.data(); v->bt_pages = P.bt_pages.data(); v->tok_slot = P.tok_slot.data();
  v->sample_end_seg = P.sample_end_seg.data(); v->sample_len = P.sample_len.data();
  return PSRL_OK;
}

psrl_status_t psrl_plan_schedule(const psrl_plan_t* plan, const int32_t** words, size_t* n_words) {
  if (!plan || !plan->p || !words || !n_words) return PSRL_ERR_INVALID_ARG;
  *words = plan->p->blob.data();
  *n_words = plan->p->blob.size();
  return PSRL_OK;
}

size_t psrl_plan_device_bytes(const psrl_plan_t* plan) {
  if (!plan || !plan->p) return 0;
  return plan->p->blob.size() * sizeof(int32_t);
}

psrl_status_t psrl_plan_upload(psrl_plan_t* plan, void* dev_buf, size_t bytes, void* stream) {
  if (!plan || !plan->p || !aligned(dev_buf, 256)) return PSRL_ERR_INVALID_ARG;
  psrl::Plan& P = *plan->p;
  const size_t need = P.blob.size() * sizeof(int32_t);
  if (bytes < need) return PSRL_ERR_WORKSPACE;
  cudaError_t e =
      cudaMemcpyAsync(dev_buf, P.blob.data(), need, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_status(e);
  P.dev = static_cast<const int32_t*>(dev_buf);
  return PSRL_OK;
}

size_t psrl_fwd_workspace_bytes(const psrl_plan_t* plan) {
  return (plan && plan->p) ? ws_bytes(*plan->p, false) : 0;
}
size_t psrl_bwd_workspace_bytes(const psrl_plan_t* plan) {
  return (plan && plan->p) ? ws_bytes(*plan->p, true) : 0;
}

psrl_status_t psrl_tree_attn_fwd(const psrl_plan_t* plan, const void* q, const void* k_pool, const void* v_pool,
                                 int64_t pool_capacity, void* o, float* lse, float softmax_scale, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  if (!plan || !plan->p) return PSRL_ERR_INVALID_ARG;
  const psrl::Plan& P = *plan->p;
  if (!aligned_q(q, 16, P) || !aligned(k_pool, 16) || !aligned(v_pool, 16) || !aligned_q(o, 16, P) ||
      !aligned_q(lse, 16, P) || !aligned(workspace, 256))
    return PSRL_ERR_INVALID_ARG;
  if (pool_capacity < P.pool_slots) return PSRL_ERR_SHAPE;
  if (!P.dev || workspace_bytes < ws_bytes(P, false)) return PSRL_ERR_WORKSPACE;
  psrl::AttnArgs a{};
  a.plan = &P; a.q = q; a.k_pool = k_pool; a.v_pool = v_pool; a.o_out = o; a.lse_out = lse;
  a.status = static_cast<int*>(workspace);
  a.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + psrl::kWsHeaderBytes);
  a.part_lse = reinterpret_cast<float*>(static_cast<char*>(workspace) + psrl::kWsHeaderBytes + psrl::ws_part_bytes(P));
  a.pool_capacity = pool_capacity; a.scale = softmax_scale; a.stream = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemsetAsync(workspace, 0, psrl::kWsHeaderBytes, a.stream);
  if (e != cudaSuccess) return cuda_status(e);
  if (P.T_q == 0) return PSRL_OK;
  if (P.dtype == PSRL_F32) return cuda_status(psrl::fwd_f32(a));
  return psrl::fwd_bf16(a);
}

static psrl_status_t bwd_checked(const psrl_plan_t* plan, const void* q, const void* k_pool, const void* v_pool,
                                 int64_t pool_capacity, const void* o, const float* lse, const void* d_o, void* d_q,
                                 void* dk_pool, void* dv_pool, float softmax_scale, void* workspace,
                                 size_t workspace_bytes, void* stream, int phases) {
  if (!plan || !plan->p) return PSRL_ERR_INVALID_ARG;
  const psrl::Plan& P = *plan->p;
  if (!aligned_q(q, 16, P) || !aligned(k_pool, 16) || !aligned(v_pool, 16) || !aligned_q(o, 16, P) ||
      !aligned_q(lse, 16, P) || !aligned_q(d_o, 16, P) || !aligned_q(d_q, 16, P) || !aligned(dk_pool, 16) ||
      !aligned(dv_pool, 16) || !aligned(workspace, 256))
    return PSRL_ERR_INVALID_ARG;
  if (pool_capacity < P.pool_slots) return PSRL_ERR_SHAPE;
  if (!P.dev || workspace_bytes < ws_bytes(P, true)) return PSRL_ERR_WORKSPACE;
  psrl::AttnArgs a{};
  a.plan = &P; a.q = q; a.k_pool = k_pool; a.v_pool = v_pool; a.o = o; a.lse_in = lse; a.d_o = d_o;
  a.d_q = d_q; a.dk_pool = dk_pool; a.dv_pool = dv_pool;
  a.status = static_cast<int*>(workspace);
  a.delta = reinterpret_cast<float*>(static_cast<char*>(workspace) + psrl::kWsHeaderBytes);
  a.slabs = reinterpret_cast<float*>(static_cast<char*>(workspace) + psrl::kWsHeaderBytes + psrl::ws_delta_bytes(P));
  a.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + psrl::kWsHeaderBytes + psrl::ws_delta_bytes(P) +
                                    psrl::ws_slab_bytes(P));
  a.pool_capacity = pool_capacity; a.scale = softmax_scale; a.stream = static_cast<cudaStream_t>(stream);
  a.phases = phases & 7;
  cudaError_t e = cudaMemsetAsync(workspace, 0, psrl::kWsHeaderBytes, a.stream);
  if (e != cudaSuccess) return cuda_status(e);
  if (P.dtype == PSRL_F32) return cuda_status(psrl::bwd_f32(a));
  return psrl::bwd_bf16(a);
}

psrl_status_t psrl_tree_attn_bwd(const psrl_plan_t* plan, const void* q, const void* k_pool, const void* v_pool,
                                 int64_t pool_capacity, const void* o, const float* lse, const void* d_o, void* d_q,
                                 void* dk_pool, void* dv_pool, float softmax_scale, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  return bwd_checked(plan, q, k_pool, v_pool, pool_capacity, o, lse, d_o, d_q, dk_pool, dv_pool, softmax_scale,
                     workspace, workspace_bytes, stream, 7);
}

psrl_status_t psrl_bench_bwd_phases(const psrl_plan_t* plan, const void* q, const void* k_pool, const void* v_pool,
                                    int64_t pool_capacity, const void* o, const float* lse, const void* d_o,
                                    void* d_q, void* dk_pool, void* dv_pool, float softmax_scale, void* workspace,
                                    size_t workspace_bytes, void* stream, int phases) {
  return bwd_checked(plan, q, k_pool, v_pool, pool_capacity, o, lse, d_o, d_q, dk_pool, dv_pool, softmax_scale,
                     workspace, workspace_bytes, stream, phases);
}

psrl_status_t psrl_device_status(const void* workspace, void* stream) {
  if (!workspace) return PSRL_ERR_INVALID_ARG;
  int st = 0;
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e == cudaSuccess) e = cudaMemcpy(&st, workspace, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_status(e);
  if (st == 0) return PSRL_OK;
  if (st == PSRL_ERR_TIMEOUT) return PSRL_ERR_TIMEOUT;
  return PSRL_ERR_INTERNAL;
}

int psrl_launch_count(const psrl_plan_t* plan, int backward) {
  if (!plan || !plan->p) return 0;
  const psrl::Plan& P = *plan->p;
  const int merge = (P.dtype == PSRL_BF16 && !P.merge_row.empty()) ? 1 : 0;
  if (!backward) return 1 + merge;
  return 3 + ((P.dtype == PSRL_BF16 && P.n_slabs > 0) ? 1 : 0) + merge;
}

const char* psrl_last_cuda_error(void) { return cudaGetErrorString(psrl::g_last_cuda); }

void psrl_plan_destroy(psrl_plan_t* plan) {
  if (!plan) return;
  delete plan->p;
  delete plan;
}

const char* psrl_status_string(psrl_status_t s) {
  switch (s) {
    case PSRL_OK: return "PSRL_OK";
    case PSRL_ERR_INVALID_ARG: return "PSRL_ERR_INVALID_ARG";
    case PSRL_ERR_BAD_TREE: return "PSRL_ERR_BAD_TREE";
    case PSRL_ERR_BAD_BLOCK_SIZE: return "PSRL_ERR_BAD_BLOCK_SIZE";
    case PSRL_ERR_SHAPE: return "PSRL_ERR_SHAPE";
    case PSRL_ERR_UNSUPPORTED: return "PSRL_ERR_UNSUPPORTED";
    case PSRL_ERR_POOL_FULL: return "PSRL_ERR_POOL_FULL";
    case PSRL_ERR_WORKSPACE: return "PSRL_ERR_WORKSPACE";
    case PSRL_ERR_HOST_OOM: return "PSRL_ERR_HOST_OOM";
    case PSRL_ERR_CUDA: return "PSRL_ERR_CUDA";
    case PSRL_ERR_TIMEOUT: return "PSRL_ERR_TIMEOUT";
    case PSRL_ERR_INTERNAL: return "PSRL_ERR_INTERNAL";
  }
  return "PSRL_ERR_?";
}

}  // extern "C"

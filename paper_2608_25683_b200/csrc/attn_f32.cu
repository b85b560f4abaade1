// fp32 SIMT tree attention, forward and backward.
//
// This is the exact-arithmetic path (fp32 inputs, fp32 products, fp64 running sums, max-abs 1e-5
// against the fp64 definition); tensor cores cannot meet that bound, so the
// kernels are plain CUDA: one warp per (query row, query head) for the forward
// and dQ, one warp per (key slot, KV head) for dK/dV.  Every output element is
// owned by one warp that sums its contributions in block-table order, so the
// results are bitwise reproducible.
//
// Math (paper Sec. 2.5: the sequence-specific mask reproduces per-sequence
// causal attention; Sec. 6: consumer adjoints accumulate on the shared K/V):
//   S_ij = scale q_i.k_j over j in ancestors(seg(i)) + own[0..i];  P = softmax(S)
//   O = P V; LSE = ln sum exp S
//   D_i = dO_i.O_i; dP = dO V^T; dS = P o (dP - D); dQ = scale dS K;
//   dK = scale dS^T Q; dV = P^T dO
#include <cuda_runtime.h>
#include <math_constants.h>

#include "kernels.h"

namespace psrl {
namespace {

constexpr int kWarpsPerBlock = 4;

struct DevPlan {
  const int32_t *seg_len, *seg_q_off, *seg_flags, *seg_first_page, *seg_bs, *seg_desc_q_begin, *seg_desc_q_end;
  const int32_t *page_slot, *page_valid, *page_seg, *page_bs, *bt_off, *bt_pages, *qrow_seg;
  int32_t T_q, n_pages;
};

DevPlan dev_plan(const Plan& P) {
  const int32_t* b = P.dev;
  const DeviceHeader& H = P.hdr;
  DevPlan d;
  d.seg_len = b + H.off_seg_len; d.seg_q_off = b + H.off_seg_q_off; d.seg_flags = b + H.off_seg_flags;
  d.seg_first_page = b + H.off_seg_first_page; d.seg_bs = b + H.off_seg_bs;
  d.seg_desc_q_begin = b + H.off_seg_desc_q_begin; d.seg_desc_q_end = b + H.off_seg_desc_q_end;
  d.page_slot = b + H.off_page_slot; d.page_valid = b + H.off_page_valid; d.page_seg = b + H.off_page_seg;
  d.page_bs = b + H.off_page_bs; d.bt_off = b + H.off_bt_off; d.bt_pages = b + H.off_bt_pages;
  d.qrow_seg = b + H.off_qrow_seg; d.T_q = P.T_q; d.n_pages = P.n_pages;
  return d;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

template <int VEC>
__device__ __forceinline__ void load_vec(float (&r)[VEC], const float* p) {
  if constexpr (VEC == 4) {
    float4 t = *reinterpret_cast<const float4*>(p);
    r[0] = t.x; r[1] = t.y; r[2] = t.z; r[3] = t.w;
  } else {
    float2 t = *reinterpret_cast<const float2*>(p);
    r[0] = t.x; r[1] = t.y;
  }
}
template <int VEC>
__device__ __forceinline__ void store_vec(float* p, const float (&r)[VEC]) {
  if constexpr (VEC == 4) {
    *reinterpret_cast<float4*>(p) = make_float4(r[0], r[1], r[2], r[3]);
  } else {
    *reinterpret_cast<float2*>(p) = make_float2(r[0], r[1]);
  }
}
template <int VEC>
__device__ __forceinline__ float dot(const float (&a)[VEC], const float (&b)[VEC]) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < VEC; ++i) s = fmaf(a[i], b[i], s);
  return s;
}

// ---------------------------------------------------------------- forward / dQ
// MODE 0: forward (O, LSE).  MODE 1: dQ (needs LSE, D, dO).
template <int D, int MODE>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
row_kernel(DevPlan dp, int Hq, int G, int64_t cap, float scale, const float* __restrict__ q,
           const float* __restrict__ kp, const float* __restrict__ vp, float* __restrict__ o_out,
           float* __restrict__ lse_out, const float* __restrict__ lse_in, const float* __restrict__ delta,
           const float* __restrict__ d_o, float* __restrict__ d_q) {
  constexpr int VEC = D / 32;
  const int lane = threadIdx.x & 31;
  const int64_t unit = int64_t(blockIdx.x) * kWarpsPerBlock + (threadIdx.x >> 5);
  if (unit >= int64_t(dp.T_q) * Hq) return;
  const int r = int(unit / Hq), h = int(unit % Hq), hk = h / G;
  const int c = dp.qrow_seg[r];
  const int i = r - dp.seg_q_off[c];
  const int first_page = dp.seg_first_page[c];
  // long sums are kept in fp64 so that the 1e-5 bound holds for thousands of keys
  float qv[VEC], dov[VEC];
  double acc[VEC];
  load_vec<VEC>(qv, q + (int64_t(r) * Hq + h) * D + lane * VEC);
#pragma unroll
  for (int x = 0; x < VEC; ++x) acc[x] = 0.0;
  float m = -CUDART_INF_F, lse = 0.f, dl = 0.f;
  double l = 0.0;
  if (MODE == 1) {
    load_vec<VEC>(dov, d_o + (int64_t(r) * Hq + h) * D + lane * VEC);
    lse = lse_in[int64_t(h) * dp.T_q + r];
    dl = delta[int64_t(h) * dp.T_q + r];
  }
  const float* kbase = kp + int64_t(hk) * cap * D + lane * VEC;
  const float* vbase = vp + int64_t(hk) * cap * D + lane * VEC;
  for (int e = dp.bt_off[c]; e < dp.bt_off[c + 1]; ++e) {
    const int pg = dp.bt_pages[e];
    int valid = dp.page_valid[pg];
    if (dp.page_seg[pg] == c) {
      const int idx0 = (pg - first_page) * dp.page_bs[pg];
      valid = min(valid, i - idx0 + 1);  // causal inside the own segment, diagonal included
      if (valid <= 0) break;
    }
    const int64_t slot0 = dp.page_slot[pg];
    for (int j = 0; j < valid; ++j) {
      float kv[VEC], vv[VEC];
      load_vec<VEC>(kv, kbase + (slot0 + j) * D);
      load_vec<VEC>(vv, vbase + (slot0 + j) * D);
      if (MODE == 0) {
        const float s = warp_sum(dot<VEC>(qv, kv)) * scale;
        const float m_new = fmaxf(m, s);
        const float alpha = expf(m - m_new);
        const float p = expf(s - m_new);
        l = l * double(alpha) + double(p);
#pragma unroll
        for (int x = 0; x < VEC; ++x) acc[x] = acc[x] * double(alpha) + double(p) * double(vv[x]);
        m = m_new;
      } else {
        float s = dot<VEC>(qv, kv), t = dot<VEC>(dov, vv);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          s += __shfl_xor_sync(0xffffffffu, s, off);
          t += __shfl_xor_sync(0xffffffffu, t, off);
        }
        const float p = expf(s * scale - lse);
        const float ds = p * (t - dl);
#pragma unroll
        for (int x = 0; x < VEC; ++x) acc[x] += double(ds) * double(kv[x]);
      }
    }
  }
  if (MODE == 0) {
    float out[VEC];
#pragma unroll
    for (int x = 0; x < VEC; ++x) out[x] = float(acc[x] / l);
    store_vec<VEC>(o_out + (int64_t(r) * Hq + h) * D + lane * VEC, out);
    if (lane == 0) lse_out[int64_t(h) * dp.T_q + r] = float(double(m) + log(l));
  } else {
    float out[VEC];
#pragma unroll
    for (int x = 0; x < VEC; ++x) out[x] = float(acc[x] * double(scale));
    store_vec<VEC>(d_q + (int64_t(r) * Hq + h) * D + lane * VEC, out);
  }
}

// ---------------------------------------------------------------- D = rowsum(dO o O)
template <int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
delta_kernel(int T_q, int Hq, const float* __restrict__ o, const float* __restrict__ d_o,
             float* __restrict__ delta) {
  constexpr int VEC = D / 32;
  const int lane = threadIdx.x & 31;
  const int64_t unit = int64_t(blockIdx.x) * kWarpsPerBlock + (threadIdx.x >> 5);
  if (unit >= int64_t(T_q) * Hq) return;
  const int r = int(unit / Hq), h = int(unit % Hq);
  float a[VEC], b[VEC];
  load_vec<VEC>(a, o + unit * D + lane * VEC);
  load_vec<VEC>(b, d_o + unit * D + lane * VEC);
  const float s = warp_sum(dot<VEC>(a, b));
  if (lane == 0) delta[int64_t(h) * T_q + r] = s;
}

// ---------------------------------------------------------------- dK / dV
// One block per (page, KV head); each warp owns key slots j = warp, warp+4, ...
// A slot beyond page_valid is a pad: its dK/dV rows are written as zeros.
template <int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
dkv_kernel(DevPlan dp, int Hq, int G, int64_t cap, float scale, const float* __restrict__ q,
           const float* __restrict__ kp, const float* __restrict__ vp, const float* __restrict__ lse,
           const float* __restrict__ delta, const float* __restrict__ d_o, float* __restrict__ dkp,
           float* __restrict__ dvp) {
  constexpr int VEC = D / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int pg = blockIdx.x, hk = blockIdx.y;
  const int a = dp.page_seg[pg], bs = dp.page_bs[pg], valid = dp.page_valid[pg];
  const int64_t slot0 = dp.page_slot[pg];
  const int pos0 = (pg - dp.seg_first_page[a]) * bs;
  const int q_off = dp.seg_q_off[a], len = dp.seg_len[a];
  const int dqb = dp.seg_desc_q_begin[a], dqe = dp.seg_desc_q_end[a];
  for (int j = warp; j < bs; j += kWarpsPerBlock) {
    double dk[VEC], dv[VEC];
#pragma unroll
    for (int x = 0; x < VEC; ++x) dk[x] = dv[x] = 0.0;
    const int64_t row = (int64_t(hk) * cap + slot0 + j) * D + lane * VEC;
    if (j < valid) {
      float kv[VEC], vv[VEC];
      load_vec<VEC>(kv, kp + row);
      load_vec<VEC>(vv, vp + row);
      // own segment rows at or after the key, then every row of every descendant
      for (int part = 0; part < 2; ++part) {
        int r0, r1;
        if (part == 0) {
          if (q_off < 0) continue;
          r0 = q_off + pos0 + j;
          r1 = q_off + len;
        } else {
          r0 = dqb;
          r1 = dqe;
        }
        for (int r = r0; r < r1; ++r) {
          for (int g = 0; g < G; ++g) {
            const int h = hk * G + g;
            float qv[VEC], dov[VEC];
            load_vec<VEC>(qv, q + (int64_t(r) * Hq + h) * D + lane * VEC);
            load_vec<VEC>(dov, d_o + (int64_t(r) * Hq + h) * D + lane * VEC);
            float s = dot<VEC>(qv, kv), t = dot<VEC>(dov, vv);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
              s += __shfl_xor_sync(0xffffffffu, s, off);
              t += __shfl_xor_sync(0xffffffffu, t, off);
            }
            const float p = expf(s * scale - lse[int64_t(h) * dp.T_q + r]);
            const float ds = p * (t - delta[int64_t(h) * dp.T_q + r]);
#pragma unroll
            for (int x = 0; x < VEC; ++x) {
              dv[x] += double(p) * double(dov[x]);
              dk[x] += double(ds) * double(qv[x]);
            }
          }
        }
      }
    }
    float dko[VEC], dvo[VEC];
#pragma unroll
    for (int x = 0; x < VEC; ++x) {
      dko[x] = float(dk[x] * double(scale));
      dvo[x] = float(dv[x]);
    }
    store_vec<VEC>(dkp + row, dko);
    store_vec<VEC>(dvp + row, dvo);
  }
}

template <int D>
cudaError_t fwd_impl(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const DevPlan dp = dev_plan(P);
  const int64_t units = int64_t(P.T_q) * P.Hq;
  const unsigned blocks = unsigned((units + kWarpsPerBlock - 1) / kWarpsPerBlock);
  row_kernel<D, 0><<<blocks, kWarpsPerBlock * 32, 0, a.stream>>>(
      dp, P.Hq, P.Hq / P.Hkv, a.pool_capacity, a.scale, static_cast<const float*>(a.q),
      static_cast<const float*>(a.k_pool), static_cast<const float*>(a.v_pool), static_cast<float*>(a.o_out),
      a.lse_out, nullptr, nullptr, nullptr, nullptr);
  return cudaGetLastError();
}

template <int D>
cudaError_t bwd_impl(const AttnArgs& a) {
  const Plan& P = *a.plan;
  const DevPlan dp = dev_plan(P);
  const int64_t units = int64_t(P.T_q) * P.Hq;
  const unsigned blocks = unsigned((units + kWarpsPerBlock - 1) / kWarpsPerBlock);
  const float* q = static_cast<const float*>(a.q);
  const float* k = static_cast<const float*>(a.k_pool);
  const float* v = static_cast<const float*>(a.v_pool);
  const float* d_o = static_cast<const float*>(a.d_o);
  if (units > 0 && (a.phases & 1))
    delta_kernel<D><<<blocks, kWarpsPerBlock * 32, 0, a.stream>>>(P.T_q, P.Hq, static_cast<const float*>(a.o), d_o,
                                                                   a.delta);
  if (units > 0 && (a.phases & 2))
    row_kernel<D, 1><<<blocks, kWarpsPerBlock * 32, 0, a.stream>>>(dp, P.Hq, P.Hq / P.Hkv, a.pool_capacity, a.scale,
                                                                    q, k, v, nullptr, nullptr, a.lse_in, a.delta, d_o,
                                                                    static_cast<float*>(a.d_q));
  dim3 grid(P.n_pages, P.Hkv);
  if (a.phases & 4)
    dkv_kernel<D><<<grid, kWarpsPerBlock * 32, 0, a.stream>>>(dp, P.Hq, P.Hq / P.Hkv, a.pool_capacity, a.scale, q, k, v,
                                                            a.lse_in, a.delta, d_o, static_cast<float*>(a.dk_pool),
                                                            static_cast<float*>(a.dv_pool));
  return cudaGetLastError();
}

}  // namespace

cudaError_t fwd_f32(const AttnArgs& a) { return a.plan->d == 64 ? fwd_impl<64>(a) : fwd_impl<128>(a); }
cudaError_t bwd_f32(const AttnArgs& a) { return a.plan->d == 64 ? bwd_impl<64>(a) : bwd_impl<128>(a); }

}  // namespace psrl

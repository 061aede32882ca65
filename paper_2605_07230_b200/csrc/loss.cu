// The drafter's training loss of Section 4.3, Eq. 4: the soft cross-entropy between the target distribution and
// the drafter's distribution at every position of a target-generated sequence, re-weighted by c where the target's
// hidden states of consecutive positions converge (cosine >= tau_seq, the criterion of Eq. 2).
//
//     L = - sum_k w_k sum_v q_k(v) log p_k(v),   q_k = softmax(target_logits[k]),  p_k = softmax(draft_logits[k])
//
// One CTA per position.  Memory-bound: both logits rows are read from HBM once (the second sweep over a row finds it
// in the L2); 2 * K * V * 4 bytes per call.  - sum_v q(v) log p(v) = lse_p - (sum_v e^(t_v - max t) d_v) / Z_t for
// target logits t and drafter logits d.  A second one-CTA kernel adds the per-position terms in index order
// (no atomics: the total does not depend on scheduling).
#include "cascade_internal.h"

namespace {

constexpr int kLossThreads = 512;

__device__ __forceinline__ float block_reduce(float v, float* red, bool is_max) {
  for (int o = 16; o > 0; o >>= 1) {
    const float x = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, x) : v + x;
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = red[0];
  for (int i = 1; i < kLossThreads / 32; ++i) t = is_max ? fmaxf(t, red[i]) : t + red[i];
  return t;
}

__global__ void __launch_bounds__(kLossThreads) k_drafter_loss(const float* __restrict__ target, const float* __restrict__ draft,
                                                               const float* __restrict__ feat, int K, int V, int h,
                                                               float tau_seq, float c, float* __restrict__ loss,
                                                               float* __restrict__ weight) {
  __shared__ float red[kLossThreads / 32];
  const int k = blockIdx.x;
  const float* t = target + (size_t)k * V;
  const float* d = draft + (size_t)k * V;
  const bool vec = (V & 3) == 0 && ((reinterpret_cast<uintptr_t>(t) | reinterpret_cast<uintptr_t>(d)) & 15u) == 0;
  // sweep 1: the two maxima
  float mt = -INFINITY, md = -INFINITY;
  if (vec) {
    const float4* t4 = reinterpret_cast<const float4*>(t);
    const float4* d4 = reinterpret_cast<const float4*>(d);
    for (int i = threadIdx.x; i < V / 4; i += kLossThreads) {
      const float4 a = t4[i], b = d4[i];
      mt = fmaxf(fmaxf(mt, fmaxf(a.x, a.y)), fmaxf(a.z, a.w));
      md = fmaxf(fmaxf(md, fmaxf(b.x, b.y)), fmaxf(b.z, b.w));
    }
  } else {
    for (int i = threadIdx.x; i < V; i += kLossThreads) {
      mt = fmaxf(mt, t[i]);
      md = fmaxf(md, d[i]);
    }
  }
  mt = block_reduce(mt, red, true);
  md = block_reduce(md, red, true);
  // sweep 2: Z_t, Z_d and sum_v e^(t_v - mt) d_v
  float zt = 0.f, zd = 0.f, cross = 0.f;
  auto term = [&](float a, float b) {
    const float e = __expf(a - mt);
    zt += e;
    zd += __expf(b - md);
    if (e > 0.f) cross += e * b;          // a token of target probability zero adds nothing, whatever the drafter says
  };
  if (vec) {
    const float4* t4 = reinterpret_cast<const float4*>(t);
    const float4* d4 = reinterpret_cast<const float4*>(d);
    for (int i = threadIdx.x; i < V / 4; i += kLossThreads) {
      const float4 a = t4[i], b = d4[i];
      term(a.x, b.x);
      term(a.y, b.y);
      term(a.z, b.z);
      term(a.w, b.w);
    }
  } else {
    for (int i = threadIdx.x; i < V; i += kLossThreads) term(t[i], d[i]);
  }
  zt = block_reduce(zt, red, false);
  zd = block_reduce(zd, red, false);
  cross = block_reduce(cross, red, false);
  // convergence of positions k and k + 1 (Eq. 2's criterion on consecutive target hidden states)
  float w = 1.f;
  if (k + 1 < K) {
    const float* fa = feat + (size_t)k * h;
    const float* fb = fa + h;
    float dot = 0.f, na = 0.f, nb = 0.f;
    for (int i = threadIdx.x; i < h; i += kLossThreads) {
      const float x = fa[i], y = fb[i];
      dot += x * y;
      na += x * x;
      nb += y * y;
    }
    dot = block_reduce(dot, red, false);
    na = block_reduce(na, red, false);
    nb = block_reduce(nb, red, false);
    if (dot / (sqrtf(na) * sqrtf(nb)) >= tau_seq) w = c;
  }
  if (threadIdx.x == 0) {
    const float ce = (md + logf(zd)) - cross / zt;
    loss[k] = w * ce;
    if (weight != nullptr) weight[k] = w;
  }
}

__global__ void __launch_bounds__(256) k_sum_in_order(const float* __restrict__ x, int n, float* __restrict__ out) {
  __shared__ double part[256];
  const int per = (n + 255) / 256, i0 = threadIdx.x * per, i1 = min(n, i0 + per);
  double s = 0.0;
  for (int i = i0; i < i1; ++i) s += (double)x[i];
  part[threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int i = 0; i < 256; ++i) tot += part[i];
    *out = (float)tot;
  }
}

}  // namespace

extern "C" int cascade_drafter_loss(const float* target_logits, const float* draft_logits, const float* feat, int32_t K,
                                    int32_t V, int32_t h, float tau_seq, float c, float* loss_out, float* weight_out,
                                    float* total_out, void* stream) {
  if (target_logits == nullptr || draft_logits == nullptr || feat == nullptr || loss_out == nullptr) return CASCADE_ERR_INVALID_ARG;
  if (K < 1 || V < 1 || h < 1 || !(c > 0.f) || tau_seq != tau_seq) return CASCADE_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  k_drafter_loss<<<K, kLossThreads, 0, s>>>(target_logits, draft_logits, feat, K, V, h, tau_seq, c, loss_out, weight_out);
  CASCADE_CUDA_TRY(cudaGetLastError());
  if (total_out != nullptr) {
    k_sum_in_order<<<1, 256, 0, s>>>(loss_out, K, total_out);
    CASCADE_CUDA_TRY(cudaGetLastError());
  }
  return CASCADE_OK;
}

// Tree-masked attention, plain CUDA-core version for the fp32 workload (small trees and prefixes).
// One CTA per (tree row, query head, CFG row): scores over the visible keys go to shared memory,
// a block-wide softmax follows, then every thread owns some output dimensions.
#include "cascade_internal.h"

namespace {

__global__ void __launch_bounds__(128) k_tree_attn_f32(
    const float* __restrict__ q, const float* __restrict__ kp, const float* __restrict__ vp, int prefix_cap,
    const int32_t* __restrict__ prefix_len, const float* __restrict__ kt, const float* __restrict__ vt,
    const uint64_t* __restrict__ anc, float* __restrict__ out, int T, int Hq, int Hkv, int D, float scale) {
  extern __shared__ float smem[];
  float* s_q = smem;       // [D]
  float* s_w = smem + D;   // [P + T]
  __shared__ float red[4];
  __shared__ float s_bcast;
  const int j = blockIdx.x, head = blockIdx.y, r = blockIdx.z;
  const int hk = head / (Hq / Hkv);
  const int P = prefix_len[r];
  const int n_keys = P + T;
  for (int d = threadIdx.x; d < D; d += blockDim.x) s_q[d] = q[(((size_t)r * T + j) * Hq + head) * D + d];
  __syncthreads();
  const uint64_t* my_anc = anc + (size_t)j * 4;
  float m = -INFINITY;
  for (int i = threadIdx.x; i < n_keys; i += blockDim.x) {
    float s = -INFINITY;
    const float* key = nullptr;
    if (i < P) key = kp + (((size_t)r * prefix_cap + i) * Hkv + hk) * D;
    else if ((my_anc[(i - P) >> 6] >> ((i - P) & 63)) & 1ull) key = kt + (((size_t)r * T + (i - P)) * Hkv + hk) * D;
    if (key != nullptr) {
      float acc = 0.f;
      for (int d = 0; d < D; ++d) acc += s_q[d] * key[d];
      s = acc * scale;
    }
    s_w[i] = s;
    m = fmaxf(m, s);
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) s_bcast = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  __syncthreads();
  m = s_bcast;
  float sum = 0.f;
  for (int i = threadIdx.x; i < n_keys; i += blockDim.x) {
    const float w = s_w[i] == -INFINITY ? 0.f : expf(s_w[i] - m);
    s_w[i] = w;
    sum += w;
  }
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) s_bcast = red[0] + red[1] + red[2] + red[3];
  __syncthreads();
  const float inv = 1.f / s_bcast;
  for (int d = threadIdx.x; d < D; d += blockDim.x) {
    float acc = 0.f;
    for (int i = 0; i < P; ++i) acc += s_w[i] * vp[(((size_t)r * prefix_cap + i) * Hkv + hk) * D + d];
    for (int i = 0; i < T; ++i)
      if (s_w[P + i] != 0.f) acc += s_w[P + i] * vt[(((size_t)r * T + i) * Hkv + hk) * D + d];
    out[(((size_t)r * T + j) * Hq + head) * D + d] = acc * inv;
  }
}

}  // namespace

int launch_tree_attn_f32(cascade_ctx* ctx, const cascade_tree* tree, const float* q, const float* kp,
                         const float* vp, int prefix_cap, const int32_t* prefix_len, const float* kt,
                         const float* vt, float* out, float scale, cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  const size_t smem = (size_t)(sh.D + sh.P_max + tree->T) * sizeof(float);
  if (smem > 200 * 1024) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  if (smem > 48 * 1024)
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(k_tree_attn_f32, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid(tree->T, sh.Hq, 2 * sh.B);
  KernelScope ks(ctx, K_TREE_ATTN_F32, s);
  k_tree_attn_f32<<<grid, 128, smem, s>>>(q, kp, vp, prefix_cap, prefix_len, kt, vt, tree->d_anc, out, tree->T,
                                          sh.Hq, sh.Hkv, sh.D, scale);
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

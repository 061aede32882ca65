// Final RMSNorm of both CFG rows, guidance mix of the normalised states, and the plain fp32 LM head.
//
// The head is linear, so W n_u + s (W n_c - W n_u) = W (n_u + s (n_c - n_u)): the mix is done here on
// the [B*T, h] operand and the product runs once.  For the bf16 path the mixed operand is stored as a
// bf16 high part plus a bf16 remainder (a = hi + lo to ~16 mantissa bits); the tensor-core GEMM adds
// both products into one fp32 accumulator.
#include "cascade_internal.h"
#include "gemm_tc.h"

namespace {

__device__ __forceinline__ float load_elem(const float* p, size_t i) { return p[i]; }
__device__ __forceinline__ float load_elem(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }

__device__ __forceinline__ float block_sum_256(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < 8; ++i) t += red[i];
  return t;
}

template <typename E>
__global__ void __launch_bounds__(256) k_final_norm_mix(const E* __restrict__ hidden, int B, int T, int h,
                                                        const float* __restrict__ gamma, float eps, float s,
                                                        float inv_temp, float* __restrict__ feat,
                                                        float* __restrict__ feat_norm,
                                                        __nv_bfloat16* __restrict__ a_hi,
                                                        __nv_bfloat16* __restrict__ a_lo,
                                                        float* __restrict__ a_f32) {
  __shared__ float red[8];
  const int j = blockIdx.x, b = blockIdx.y;
  const size_t row_c = ((size_t)b * T + j) * h, row_u = ((size_t)(B + b) * T + j) * h;
  float ss_c = 0.f, ss_u = 0.f;
  for (int i = threadIdx.x; i < h; i += 256) {
    const float c = load_elem(hidden, row_c + i), u = load_elem(hidden, row_u + i);
    ss_c += c * c;
    ss_u += u * u;
  }
  ss_c = block_sum_256(ss_c, red);
  ss_u = block_sum_256(ss_u, red);
  const float rc = rsqrtf(ss_c / h + eps), ru = rsqrtf(ss_u / h + eps);
  float nn = 0.f;
  const size_t m = (size_t)b * T + j;
  for (int i = threadIdx.x; i < h; i += 256) {
    const float g = gamma[i];
    const float nc = load_elem(hidden, row_c + i) * rc * g;
    const float nu = load_elem(hidden, row_u + i) * ru * g;
    nn += nc * nc;
    if (feat != nullptr) feat[m * h + i] = nc;
    const float a = (nu + s * (nc - nu)) * inv_temp;
    if (a_hi != nullptr) {
      const __nv_bfloat16 hi = __float2bfloat16_rn(a);
      a_hi[m * h + i] = hi;
      a_lo[m * h + i] = __float2bfloat16_rn(a - __bfloat162float(hi));
    } else {
      a_f32[m * h + i] = a;
    }
  }
  nn = block_sum_256(nn, red);
  if (threadIdx.x == 0 && feat_norm != nullptr) feat_norm[m] = sqrtf(nn);
}

// logits[m][v] = sum_k a[m][k] W[v][k]; a warp per vocabulary row, 8 operand rows per CTA.
__global__ void __launch_bounds__(256) k_head_f32(const float* __restrict__ a, const float* __restrict__ W, int M,
                                                  int V, int h, float* __restrict__ logits) {
  const int v = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (v >= V) return;
  for (int mi = 0; mi < 8; ++mi) {
    const int m = blockIdx.y * 8 + mi;
    if (m >= M) break;
    float acc = 0.f;
    for (int k = lane; k < h; k += 32) acc += a[(size_t)m * h + k] * W[(size_t)v * h + k];
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) logits[(size_t)m * V + v] = acc;
  }
}

// Logits the acceptance rule reads, straight from the operands: for draft node j the logit of tok[j]
// under its parent's row and under its grandparent's row (Algorithm 2: q_x = gtp[x]; Eq. 3 sums).
// One CTA per (node, prompt); 128 threads split the dot products over h.
__global__ void __launch_bounds__(128) k_cand_logits(const __nv_bfloat16* __restrict__ a_hi,
                                                     const __nv_bfloat16* __restrict__ a_lo,
                                                     const __nv_bfloat16* __restrict__ W, int T, int h, int V,
                                                     const int32_t* __restrict__ tok,
                                                     const int32_t* __restrict__ parent,
                                                     float* __restrict__ cand_parent,
                                                     float* __restrict__ cand_gparent) {
  const int j = blockIdx.x, b = blockIdx.y;
  const size_t idx = (size_t)b * T + j;
  __shared__ float red[2][4];
  float dp = 0.f, dg = 0.f;
  const int pi = parent[j];
  const int gp = pi >= 0 ? parent[pi] : -1;
  if (pi >= 0) {
    const int t = tok[idx];
    const __nv_bfloat16* w = W + (size_t)t * h;
    const size_t rp = ((size_t)b * T + pi) * h, rg = ((size_t)b * T + (gp >= 0 ? gp : pi)) * h;
    for (int i = threadIdx.x; i < h; i += 128) {
      const float wv = __bfloat162float(w[i]);
      dp += wv * (__bfloat162float(a_hi[rp + i]) + __bfloat162float(a_lo[rp + i]));
      dg += wv * (__bfloat162float(a_hi[rg + i]) + __bfloat162float(a_lo[rg + i]));
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    dp += __shfl_xor_sync(0xffffffffu, dp, o);
    dg += __shfl_xor_sync(0xffffffffu, dg, o);
  }
  if ((threadIdx.x & 31) == 0) {
    red[0][threadIdx.x >> 5] = dp;
    red[1][threadIdx.x >> 5] = dg;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    cand_parent[idx] = pi >= 0 ? red[0][0] + red[0][1] + red[0][2] + red[0][3] : 0.f;
    cand_gparent[idx] = gp >= 0 ? red[1][0] + red[1][1] + red[1][2] + red[1][3] : 0.f;
  }
}

}  // namespace

int launch_head_bf16(cascade_ctx* ctx, const cascade_tree* tree, const __nv_bfloat16* w_head, const int32_t* tok,
                     float* logits, float* row_lse, float* cand_parent, float* cand_gparent, cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  const int M = sh.B * tree->T;
  if (tok != nullptr) {
    dim3 grid(tree->T, sh.B);
    KernelScope ks(ctx, K_CAND_LOGITS, s);
    k_cand_logits<<<grid, 128, 0, s>>>(ctx->head_a_hi, ctx->head_a_lo, w_head, tree->T, sh.h, sh.V, tok,
                                       tree->d_parent, cand_parent, cand_gparent);
    CASCADE_CUDA_TRY(cudaGetLastError());
  }
  return launch_gemm_tc(ctx, w_head, sh.V, sh.h, ctx->head_a_hi, ctx->head_a_lo, M, logits, sh.V, ctx->head_part,
                        cascade_detail::ceil_div(sh.V, 128), row_lse, K_GEMM_HEAD, s);
}

int launch_final_norm_mix(cascade_ctx* ctx, int T, const void* hidden, const float* gamma, float eps,
                          float cfg_scale, float inv_temperature, float* feat, float* feat_norm,
                          cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  dim3 grid(T, sh.B);
  KernelScope ks(ctx, K_FINAL_NORM_MIX, s);
  if (sh.dtype == CASCADE_BF16)
    k_final_norm_mix<__nv_bfloat16><<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(hidden), sh.B, T, sh.h,
                                                         gamma, eps, cfg_scale, inv_temperature, feat, feat_norm,
                                                         ctx->head_a_hi, ctx->head_a_lo, nullptr);
  else
    k_final_norm_mix<float><<<grid, 256, 0, s>>>(static_cast<const float*>(hidden), sh.B, T, sh.h, gamma, eps,
                                                 cfg_scale, inv_temperature, feat, feat_norm, nullptr, nullptr,
                                                 ctx->head_a_f32);
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

int launch_head_f32(cascade_ctx* ctx, const cascade_tree* tree, const float* w_head, const int32_t* tok,
                    float* logits, float* row_lse, float* cand_parent, float* cand_gparent, cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  const int M = sh.B * tree->T;
  dim3 grid(cascade_detail::ceil_div(sh.V, 8), cascade_detail::ceil_div(M, 8));
  {
    KernelScope ks(ctx, K_HEAD_F32, s);
    k_head_f32<<<grid, 256, 0, s>>>(ctx->head_a_f32, w_head, M, sh.V, sh.h, logits);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return launch_row_stats_from_logits(ctx, tree, logits, tok, row_lse, cand_parent, cand_gparent, s);
}

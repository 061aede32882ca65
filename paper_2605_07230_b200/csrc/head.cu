// Final RMSNorm of both CFG rows, guidance mix of the normalised states, and the plain fp32 LM head.
//
// The head is linear, so W n_u + s (W n_c - W n_u) = W (n_u + s (n_c - n_u)): the mix is done here on
// the [B*T, h] operand and the product runs once.  For the bf16 path the mixed operand is stored as a
// bf16 high part plus a bf16 remainder (a = hi + lo to ~16 mantissa bits), in the staged layout the
// tensor-core GEMM copies straight into shared memory; the GEMM adds both products into one fp32
// accumulator.
#include "cascade_internal.h"
#include "gemm_tc.h"
#include "operand.cuh"

namespace {

// 8 consecutive elements of a row as floats (16-byte loads for bf16, 2 x 16 bytes for fp32)
__device__ __forceinline__ void load8(const float* p, float* v) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float* v) {
  const uint4 r = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

constexpr int kNormThreads = 256;
constexpr int kNormChunks = 4;  // rows of up to 256 * 8 * 4 = 8192 elements stay in registers

__device__ __forceinline__ float block_sum(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < kNormThreads / 32; ++i) t += red[i];
  return t;
}

// One CTA per (tree row, prompt): RMSNorm of the cond and uncond rows, features, guidance mix.
// h is a multiple of 8.  Rows longer than the register budget are read a second time.
template <typename E>
__global__ void __launch_bounds__(kNormThreads) k_final_norm_mix(const E* __restrict__ hidden, int B, int T, int h,
                                                                 const float* __restrict__ gamma, float eps, float s,
                                                                 float inv_temp, float* __restrict__ feat,
                                                                 float* __restrict__ feat_norm,
                                                                 __nv_bfloat16* __restrict__ a_op,
                                                                 const OperandLayout lay, float* __restrict__ a_f32,
                                                                 float* __restrict__ cand_parent,
                                                                 float* __restrict__ cand_gparent,
                                                                 const float* __restrict__ add, int n_add,
                                                                 long long add_stride) {
  __shared__ float red[kNormThreads / 32];
  const int j = blockIdx.x, b = blockIdx.y;
  const size_t m = (size_t)b * T + j;
  const E* row_c = hidden + m * h;
  const E* row_u = hidden + ((size_t)(B + b) * T + j) * h;
  const int n8 = h / 8;
  float c[kNormChunks][8], u[kNormChunks][8];
  float ss_c = 0.f, ss_u = 0.f;
  // 8 elements of the cond and the uncond row, plus whatever projection output has not been added to
  // the residual stream yet
  auto load_pair = [&](int i, float* vc, float* vu) {
    load8(row_c + 8 * i, vc);
    load8(row_u + 8 * i, vu);
    // three slices at a time: their loads are issued before the first is used (one L2 round trip per slice,
    // nine in a row, was most of this kernel's time); added in slice order
    for (int s0 = 0; s0 < n_add; s0 += 3) {
      float tc[3][8], tu[3][8];
#pragma unroll
      for (int q = 0; q < 3; ++q) {
        if (s0 + q < n_add) {
          const float* a0 = add + (size_t)(s0 + q) * add_stride + 8 * (size_t)i;
          load8(a0 + m * h, tc[q]);
          load8(a0 + ((size_t)(B + b) * T + j) * h, tu[q]);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) tc[q][e] = tu[q][e] = 0.f;
        }
      }
#pragma unroll
      for (int q = 0; q < 3; ++q)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          vc[e] += tc[q][e];
          vu[e] += tu[q][e];
        }
    }
  };
#pragma unroll
  for (int k = 0; k < kNormChunks; ++k) {
    const int i = threadIdx.x + k * kNormThreads;
    if (i < n8) {
      load_pair(i, c[k], u[k]);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        ss_c += c[k][e] * c[k][e];
        ss_u += u[k][e] * u[k][e];
      }
    }
  }
  for (int i = threadIdx.x + kNormChunks * kNormThreads; i < n8; i += kNormThreads) {
    float tc[8], tu[8];
    load_pair(i, tc, tu);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      ss_c += tc[e] * tc[e];
      ss_u += tu[e] * tu[e];
    }
  }
  ss_c = block_sum(ss_c, red);
  ss_u = block_sum(ss_u, red);
  const float rc = rsqrtf(ss_c / h + eps), ru = rsqrtf(ss_u / h + eps);
  float nn = 0.f;
  auto emit = [&](int i, const float* vc, const float* vu) {
    float g[8], nc[8], a[8];
    load8(gamma + 8 * i, g);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      nc[e] = vc[e] * rc * g[e];
      const float nu = vu[e] * ru * g[e];
      nn += nc[e] * nc[e];
      a[e] = (nu + s * (nc[e] - nu)) * inv_temp;
    }
    const size_t o = m * h + 8 * (size_t)i;
    if (feat != nullptr) {
      *reinterpret_cast<float4*>(feat + o) = make_float4(nc[0], nc[1], nc[2], nc[3]);
      *reinterpret_cast<float4*>(feat + o + 4) = make_float4(nc[4], nc[5], nc[6], nc[7]);
    }
    if (a_op != nullptr) {
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const __nv_bfloat16 h0 = __float2bfloat16_rn(a[2 * e]), h1 = __float2bfloat16_rn(a[2 * e + 1]);
        const __nv_bfloat16 l0 = __float2bfloat16_rn(a[2 * e] - __bfloat162float(h0));
        const __nv_bfloat16 l1 = __float2bfloat16_rn(a[2 * e + 1] - __bfloat162float(h1));
        hi[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
        lo[e] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
      }
      // GEMM operand in its staged layout: 8 consecutive K elements stay one 16-byte piece
      *reinterpret_cast<uint4*>(a_op + operand_index(lay, (int)m, 8 * i, 0)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *reinterpret_cast<uint4*>(a_op + operand_index(lay, (int)m, 8 * i, 1)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    } else {
      *reinterpret_cast<float4*>(a_f32 + o) = make_float4(a[0], a[1], a[2], a[3]);
      *reinterpret_cast<float4*>(a_f32 + o + 4) = make_float4(a[4], a[5], a[6], a[7]);
    }
  };
#pragma unroll
  for (int k = 0; k < kNormChunks; ++k) {
    const int i = threadIdx.x + k * kNormThreads;
    if (i < n8) emit(i, c[k], u[k]);
  }
  for (int i = threadIdx.x + kNormChunks * kNormThreads; i < n8; i += kNormThreads) {
    float tc[8], tu[8];
    load_pair(i, tc, tu);
    emit(i, tc, tu);
  }
  nn = block_sum(nn, red);
  if (threadIdx.x == 0) {
    if (feat_norm != nullptr) feat_norm[m] = sqrtf(nn);
    if (cand_parent != nullptr) cand_parent[m] = 0.f;
    if (cand_gparent != nullptr) cand_gparent[m] = 0.f;
  }
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

}  // namespace

int launch_head_bf16(cascade_ctx* ctx, const cascade_tree* tree, const __nv_bfloat16* w_head, const int32_t* tok,
                     float* logits, float* cand_parent, float* cand_gparent, cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  GemmEpilogue e;
  e.C = logits;
  e.ldc = sh.V;
  e.part = ctx->head_part;
  e.part_ld = ctx->head_max_tiles;
  if (tok != nullptr) {
    e.tok = tok;
    e.parent = tree->d_parent;
    e.T = tree->T;
    e.n_rows = sh.B * tree->T;
    e.cand_parent = cand_parent;
    e.cand_gparent = cand_gparent;
  }
  // With more than 128 activation rows (several row chunks) the head is no longer a weight stream: every weight tile
  // is used once per chunk, there are hundreds of (tile, chunk) items, and what bounds a 128 x 128 item is the
  // shared-memory fill per UMMA (16 KB of weights + 32 KB of activation pair for eight instructions).  Whole
  // items of 256 weight rows (two accumulators on one activation stage, nothing cut along K, no hand-off) double
  // the tensor work per byte taken in.
  if (operand_layout(sh.B * tree->T, sh.h).n_chunks > 1) e.splits = 1;
  return launch_gemm_tc(ctx, w_head, sh.V, sh.h, ctx->head_a, sh.B * tree->T, e, K_GEMM_HEAD, s);
}

int launch_final_norm_mix(cascade_ctx* ctx, int T, const void* hidden, bool hidden_f32, const PendingAdd& add,
                          const float* gamma, float eps, float cfg_scale, float inv_temperature, float* feat, float* feat_norm,
                          float* cand_parent, float* cand_gparent, cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  dim3 grid(T, sh.B);
  KernelScope ks(ctx, K_FINAL_NORM_MIX, s);
  const bool bf16 = sh.dtype == CASCADE_BF16;
  __nv_bfloat16* a_op = bf16 ? ctx->head_a : nullptr;
  const OperandLayout lay = operand_layout(sh.B * T, sh.h);
  float* a_f32 = bf16 ? nullptr : ctx->head_a_f32;
  if (bf16 && !hidden_f32)
    k_final_norm_mix<__nv_bfloat16><<<grid, kNormThreads, 0, s>>>(static_cast<const __nv_bfloat16*>(hidden), sh.B, T,
                                                                  sh.h, gamma, eps, cfg_scale, inv_temperature, feat,
                                                                  feat_norm, a_op, lay, a_f32, cand_parent, cand_gparent,
                                                                  add.slices, add.n, add.stride);
  else
    k_final_norm_mix<float><<<grid, kNormThreads, 0, s>>>(static_cast<const float*>(hidden), sh.B, T, sh.h, gamma, eps,
                                                          cfg_scale, inv_temperature, feat, feat_norm, a_op, lay, a_f32,
                                                          cand_parent, cand_gparent, add.slices, add.n, add.stride);
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

// The decoder layer around the tree attention (support for the workloads that run the verification
// step through a layer: the paper treats the target model as given, the architecture is the usual
// pre-norm block with rotary embeddings and a SwiGLU MLP).
//
//     a = RMSNorm(x, gamma_attn);  q,k,v = a Wq^T, a Wk^T, a Wv^T;  rotary at prefix_len[r] + depth[j];
//     tree attention;  x += attn Wo^T;  m = RMSNorm(x, gamma_mlp);  x += (silu(m Wg^T) * (m Wu^T)) Wd^T
//
// The projections run on the tensor-core GEMM in sliced mode (K cut into S slices, one output matrix
// per slice); the row-wise kernels here add the S matrices while they do their own work, so no GEMM
// waits for another CTA.  The residual stream x stays fp32; GEMM operands are written as a bf16 high
// part plus a bf16 remainder, in the staged layout the GEMM copies straight into shared memory.
#include "cascade_internal.h"
#include "gemm_tc.h"
#include "operand.cuh"

namespace {

constexpr int kRowThreads = 256;

__device__ __forceinline__ float block_sum(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < kRowThreads / 32; ++i) t += red[i];
  return t;
}

__device__ __forceinline__ float elem_to_float(const float* p, size_t i) { return p[i]; }
__device__ __forceinline__ float elem_to_float(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }

__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 r = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u), __uint_as_float(r.y << 16),
                     __uint_as_float(r.y & 0xffff0000u));
}
__device__ __forceinline__ void add4(float4& a, const float4 b) {
  a.x += b.x;
  a.y += b.y;
  a.z += b.z;
  a.w += b.w;
}
// v + slices[0] + slices[1] + ... in that order, `stride` floats apart.  The loads of four slices are issued before the
// first of them is used: these kernels run few warps per SM, and one L2 round trip per slice (a dependent chain
// of up to nine) was most of their time.
__device__ __forceinline__ float4 add_slices(float4 v, const float* p, int n, long long stride) {
  int s = 0;
  for (; s + 4 <= n; s += 4) {
    const float4 t0 = load4(p + (size_t)s * stride), t1 = load4(p + (size_t)(s + 1) * stride),
                 t2 = load4(p + (size_t)(s + 2) * stride), t3 = load4(p + (size_t)(s + 3) * stride);
    add4(v, t0);
    add4(v, t1);
    add4(v, t2);
    add4(v, t3);
  }
  if (s + 2 <= n) {
    const float4 t0 = load4(p + (size_t)s * stride), t1 = load4(p + (size_t)(s + 1) * stride);
    add4(v, t0);
    add4(v, t1);
    s += 2;
  }
  if (s < n) add4(v, load4(p + (size_t)s * stride));
  return v;
}

// four consecutive operand values of row m, columns k..k+3 (k a multiple of 4): fp32, or the bf16 pair in the
// GEMM's staged layout
__device__ __forceinline__ void put_operand4(__nv_bfloat16* op, const OperandLayout& lay, float* f32, int K, int m, int k,
                                             const float4 a) {
  if (op != nullptr) {
    const float v[4] = {a.x, a.y, a.z, a.w};
    uint32_t h[2], l[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const __nv_bfloat16 h0 = __float2bfloat16_rn(v[2 * i]), h1 = __float2bfloat16_rn(v[2 * i + 1]);
      const __nv_bfloat16 l0 = __float2bfloat16_rn(v[2 * i] - __bfloat162float(h0));
      const __nv_bfloat16 l1 = __float2bfloat16_rn(v[2 * i + 1] - __bfloat162float(h1));
      h[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      l[i] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
    }
    *reinterpret_cast<uint2*>(op + operand_index(lay, m, k, 0)) = make_uint2(h[0], h[1]);
    *reinterpret_cast<uint2*>(op + operand_index(lay, m, k, 1)) = make_uint2(l[0], l[1]);
  } else {
    *reinterpret_cast<float4*>(f32 + (size_t)m * K + k) = a;
  }
}

constexpr int kRowChunks = 8;  // float4 chunks of a row a thread keeps in registers (rows up to 8192 elements)

// One CTA per row m = r * T + j of the CFG pair.  h is a multiple of 4.
//   x[m] (+)= ...: embed != null: x[m] = embed[tok[b, j]]            (first layer)
//                  else          x[m] += sum_s slices[s][m]          (output of the previous projection)
//   operand[m] = RMSNorm(x[m], gamma)                                (skipped when gamma == null)
template <typename E>
__global__ void __launch_bounds__(kRowThreads) k_resid_norm(float* __restrict__ x, int B, int T, int h,
                                                            const E* __restrict__ embed,
                                                            const int32_t* __restrict__ tok,
                                                            const float* __restrict__ slices, int n_slices,
                                                            long long slice_stride, const float* __restrict__ gamma,
                                                            float eps, __nv_bfloat16* __restrict__ a_op,
                                                            const OperandLayout lay, float* __restrict__ a_f32,
                                                            float* __restrict__ x_copy) {
  __shared__ float red[kRowThreads / 32];
  const int m = blockIdx.x;
  const int r = m / T, j = m - r * T, b = r % B;
  float* xr = x + (size_t)m * h;
  const E* er = embed != nullptr ? embed + (size_t)tok[(size_t)b * T + j] * h : nullptr;
  const int n4 = h / 4;
  auto value = [&](int c) {  // element chunk c of the updated row
    float4 v;
    if (er != nullptr) {
      v = load4(er + 4 * c);
    } else {
      v = add_slices(load4(xr + 4 * c), slices + (size_t)m * h + 4 * c, n_slices, slice_stride);
    }
    return v;
  };
  float4 keep[kRowChunks];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < kRowChunks; ++k) {
    const int c = threadIdx.x + k * kRowThreads;
    if (c < n4) {
      keep[k] = value(c);
      ss += keep[k].x * keep[k].x + keep[k].y * keep[k].y + keep[k].z * keep[k].z + keep[k].w * keep[k].w;
      *reinterpret_cast<float4*>(xr + 4 * c) = keep[k];
      if (x_copy != nullptr) *reinterpret_cast<float4*>(x_copy + (size_t)m * h + 4 * c) = keep[k];
    }
  }
  for (int c = threadIdx.x + kRowChunks * kRowThreads; c < n4; c += kRowThreads) {  // longer rows: via memory
    const float4 v = value(c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    *reinterpret_cast<float4*>(xr + 4 * c) = v;
    if (x_copy != nullptr) *reinterpret_cast<float4*>(x_copy + (size_t)m * h + 4 * c) = v;
  }
  if (gamma == nullptr) return;
  ss = block_sum(ss, red);
  const float rs = rsqrtf(ss / h + eps);
  auto emit = [&](int c, const float4 v) {
    const float4 g = load4(gamma + 4 * c);
    put_operand4(a_op, lay, a_f32, h, m, 4 * c, make_float4(v.x * rs * g.x, v.y * rs * g.y, v.z * rs * g.z, v.w * rs * g.w));
  };
#pragma unroll
  for (int k = 0; k < kRowChunks; ++k) {
    const int c = threadIdx.x + k * kRowThreads;
    if (c < n4) emit(c, keep[k]);
  }
  for (int c = threadIdx.x + kRowChunks * kRowThreads; c < n4; c += kRowThreads) emit(c, load4(xr + 4 * c));
}

// q, k, v = sum of the projection's slices; rotary embedding (half-split pairing: (x[i], x[i + D/2]) turned
// by pos * base^(-2i/D)) on q and k at pos = prefix_len[r] + depth[j]; results in the attention's
// element type.  grid (T, R, z): one position per CTA, so its D/2 (cos, sin) pairs are computed once into
// shared memory; the z CTAs of a row share its heads.  D is a multiple of 8.
template <typename E>
__global__ void __launch_bounds__(kRowThreads) k_rope_split(const float* __restrict__ slices, int n_slices,
                                                            long long slice_stride, int T, int Hq, int Hkv, int D,
                                                            const int32_t* __restrict__ prefix_len,
                                                            const int32_t* __restrict__ depth, float rope_base,
                                                            E* __restrict__ q, E* __restrict__ k, E* __restrict__ v) {
  __shared__ float s_cos[128], s_sin[128];  // D <= 256
  const int j = blockIdx.x, r = blockIdx.y;
  const size_t m = (size_t)r * T + j;
  const int n_cols = (Hq + 2 * Hkv) * D, half = D / 2;
  // The angle is formed in double precision: at position 2500 a float angle is off by about 2e-4 rad, which
  // flips the bf16 rounding of one rotated q / k element in ten against an exact evaluation; each flip is a 0.4 %
  // perturbation of that element.  D / 2 angles per CTA, so the cost does not show.
  const double pos = (double)(prefix_len[r] + depth[j]);
  for (int i = threadIdx.x; i < half; i += kRowThreads) {
    const double inv_freq = exp2(-2.0 * (double)i / (double)D * log2((double)rope_base));
    double sn, cs;
    sincos(pos * inv_freq, &sn, &cs);
    s_sin[i] = (float)sn;
    s_cos[i] = (float)cs;
  }
  __syncthreads();
  auto col4 = [&](int c) {
    return add_slices(make_float4(0.f, 0.f, 0.f, 0.f), slices + m * n_cols + c, n_slices, slice_stride);
  };
  auto store4 = [](E* dst, size_t i, const float4 a) {
    if constexpr (sizeof(E) == 2) {
      const __nv_bfloat16 b0 = __float2bfloat16_rn(a.x), b1 = __float2bfloat16_rn(a.y), b2 = __float2bfloat16_rn(a.z),
                          b3 = __float2bfloat16_rn(a.w);
      *reinterpret_cast<uint2*>(dst + i) =
          make_uint2((uint32_t)__bfloat16_as_ushort(b0) | ((uint32_t)__bfloat16_as_ushort(b1) << 16),
                     (uint32_t)__bfloat16_as_ushort(b2) | ((uint32_t)__bfloat16_as_ushort(b3) << 16));
    } else {
      *reinterpret_cast<float4*>(dst + i) = a;
    }
  };
  // rotated pairs of q and k, four pair indices per thread and step
  const int q4 = half / 4;
  for (int t = blockIdx.z * kRowThreads + threadIdx.x; t < (Hq + Hkv) * q4; t += gridDim.z * kRowThreads) {
    const int head = t / q4, i = (t - head * q4) * 4;
    const int c0 = head * D + i;  // q heads first, then k heads: same column order as the projection
    const float4 x1 = col4(c0), x2 = col4(c0 + half);
    const float4 cs = load4(s_cos + i), sn = load4(s_sin + i);
    const float4 y1 = make_float4(x1.x * cs.x - x2.x * sn.x, x1.y * cs.y - x2.y * sn.y, x1.z * cs.z - x2.z * sn.z,
                                  x1.w * cs.w - x2.w * sn.w);
    const float4 y2 = make_float4(x2.x * cs.x + x1.x * sn.x, x2.y * cs.y + x1.y * sn.y, x2.z * cs.z + x1.z * sn.z,
                                  x2.w * cs.w + x1.w * sn.w);
    if (head < Hq) {
      const size_t o = (m * Hq + head) * D + i;
      store4(q, o, y1);
      store4(q, o + half, y2);
    } else {
      const size_t o = (m * Hkv + (head - Hq)) * D + i;
      store4(k, o, y1);
      store4(k, o + half, y2);
    }
  }
  for (int t = blockIdx.z * kRowThreads + threadIdx.x; t < Hkv * D / 4; t += gridDim.z * kRowThreads)
    store4(v, m * Hkv * D + 4 * t, col4((Hq + Hkv) * D + 4 * t));
}

// act = silu(gate) * up from the slices of the fused gate/up projection ([.., 2*ffn]: gate then up).
// ffn is a multiple of 4.
__global__ void __launch_bounds__(kRowThreads) k_swiglu(const float* __restrict__ slices, const SliceMap map,
                                                        long long slice_stride, int ffn,
                                                        __nv_bfloat16* __restrict__ a_op, const OperandLayout lay,
                                                        float* __restrict__ a_f32) {
  const size_t m = blockIdx.y;
  // pieces per projection tile for the (at most kCntTiles) tiles this CTA's gate and up columns fall into
  constexpr int kCntTiles = 16;
  __shared__ int s_cnt[2][kCntTiles];
  const int col0 = blockIdx.x * kRowThreads * 4;
  const int t0g = map.balanced ? col0 / map.tile_cols : 0, t0u = map.balanced ? (ffn + col0) / map.tile_cols : 0;
  if (map.balanced) {
    if (threadIdx.x < 2 * kCntTiles) {
      const int which = threadIdx.x / kCntTiles, i = threadIdx.x % kCntTiles;
      s_cnt[which][i] = slice_count(map, ((which ? t0u : t0g) + i) * map.tile_cols);
    }
    __syncthreads();
  }
  for (int c = blockIdx.x * kRowThreads + threadIdx.x; c < ffn / 4; c += gridDim.x * kRowThreads) {
    float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
    // the gate and the up column lie in different tiles of the projection, which may have been cut into
    // different numbers of pieces (looked up in the table the first threads made)
    const int n_g = map.balanced ? s_cnt[0][(4 * c) / map.tile_cols - t0g] : map.n_slices;
    const int n_u = map.balanced ? s_cnt[1][(ffn + 4 * c) / map.tile_cols - t0u] : map.n_slices;
    // the gate and up loads of up to four slices go out together (a dependent round trip per slice otherwise)
    for (int s0 = 0; s0 < max(n_g, n_u); s0 += 4) {
      float4 tg[4], tu[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float* row = slices + (size_t)(s0 + i) * slice_stride + m * 2 * ffn;
        tg[i] = s0 + i < n_g ? load4(row + 4 * c) : make_float4(0.f, 0.f, 0.f, 0.f);
        tu[i] = s0 + i < n_u ? load4(row + ffn + 4 * c) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        add4(g, tg[i]);
        add4(u, tu[i]);
      }
    }
    put_operand4(a_op, lay, a_f32, ffn, (int)m, 4 * c,
                 make_float4(g.x / (1.f + expf(-g.x)) * u.x, g.y / (1.f + expf(-g.y)) * u.y,
                             g.z / (1.f + expf(-g.z)) * u.z, g.w / (1.f + expf(-g.w)) * u.w));
  }
}

// Plain fp32 projection for the fp32 workload: C[m][n] = sum_k A[m][k] W[n][k]; a warp per weight row.
__global__ void __launch_bounds__(256) k_gemm_f32(const float* __restrict__ A, const float* __restrict__ W, int M,
                                                  int N, int K, float* __restrict__ C) {
  const int n = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (n >= N) return;
  for (int mi = 0; mi < 8; ++mi) {
    const int m = blockIdx.y * 8 + mi;
    if (m >= M) break;
    float acc = 0.f;
    for (int k = lane; k < K; k += 32) acc += A[(size_t)m * K + k] * W[(size_t)n * K + k];
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) C[(size_t)m * N + n] = acc;
  }
}

struct Projection {
  int n_slices;
  long long slice_stride;
  SliceMap map;  // which of the n_slices matrices hold a given column (all of them unless map.balanced)
};

// out slices = operand x W^T for one weight matrix (or several stacked in memory).
int project(cascade_ctx* ctx, const void* W, int N, int K, int M, bool operand_is_attn, int kernel_id, Projection* pr,
            cudaStream_t s, bool consumer_reads_map = false) {
  pr->slice_stride = (long long)M * N;
  pr->map = SliceMap{};
  if (ctx->shape.dtype == CASCADE_BF16) {
    int S = gemm_tc_pick_splits(ctx->sm_count, M, N, K, ctx->layer_max_splits);
    GemmEpilogue e;
    if (consumer_reads_map) {
      // equal ranges of (tile, K block) units per CTA instead of whole (tile, slice) items: no CTA is left with
      // one item while the others have two
      const SliceMap map = gemm_tc_balanced_map(ctx, M, N, K);
      if (map.balanced && map.n_slices <= ctx->layer_max_splits &&
          (long long)map.n_slices * M * N <= ctx->gemm_out_floats) {
        pr->map = map;
        S = map.n_slices;
        e.balanced = 1;
      }
    }
    pr->n_slices = S;
    pr->map.n_slices = S;
    e.C = ctx->gemm_out;
    e.ldc = N;
    e.splits = S;
    e.slice_stride = pr->slice_stride;
    if ((long long)S * M * N > ctx->gemm_out_floats) return CASCADE_ERR_WORKSPACE;
    // the operand is already in the GEMM's staged layout (the attention writes its output that way too)
    return launch_gemm_tc(ctx, (const __nv_bfloat16*)W, N, K,
                          operand_is_attn ? (const __nv_bfloat16*)ctx->attn_out : ctx->act, M, e, kernel_id, s);
  }
  pr->n_slices = 1;
  pr->map.n_slices = 1;
  dim3 grid(cascade_detail::ceil_div(N, 8), cascade_detail::ceil_div(M, 8));
  {
    KernelScope ks(ctx, K_GEMM_F32, s);
    k_gemm_f32<<<grid, 256, 0, s>>>(operand_is_attn ? (const float*)ctx->attn_out : ctx->act_f32, (const float*)W, M, N, K,
                                    ctx->gemm_out);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

template <typename E>
int resid_norm(cascade_ctx* ctx, int T, const void* embed, const int32_t* tok, const Projection* pr, const float* gamma,
               float eps, float* x_copy, int kernel_id, cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  const int M = 2 * sh.B * T;
  const bool bf16 = sh.dtype == CASCADE_BF16;
  KernelScope ks(ctx, kernel_id, s);
  k_resid_norm<E><<<M, kRowThreads, 0, s>>>(ctx->x, sh.B, T, sh.h, (const E*)embed, tok, ctx->gemm_out,
                                            pr ? pr->n_slices : 0, pr ? pr->slice_stride : 0, gamma, eps,
                                            bf16 ? ctx->act : nullptr, operand_layout(M, sh.h), bf16 ? nullptr : ctx->act_f32,
                                            x_copy);
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

template <typename E>
int run_layers_t(cascade_ctx* ctx, const cascade_tree* tree, const cascade_step* st, PendingAdd* pending,
                 cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  const int T = tree->T, R = 2 * sh.B, M = R * T;
  const int qkv_cols = (sh.Hq + 2 * sh.Hkv) * sh.D;
  Projection pr = {0, 0};
  for (int li = 0; li < st->n_layers; ++li) {
    const cascade_layer& L = st->layers[li];
    if (L.gamma_attn == nullptr || L.wq == nullptr || L.wk == nullptr || L.wv == nullptr || L.wo == nullptr ||
        L.gamma_mlp == nullptr || L.w_gate == nullptr || L.w_up == nullptr || L.w_down == nullptr)
      return CASCADE_ERR_INVALID_ARG;
    if (st->prefix_cap > 0 && (L.k_prefix == nullptr || L.v_prefix == nullptr)) return CASCADE_ERR_INVALID_ARG;
    if (((uintptr_t)L.gamma_attn | (uintptr_t)L.gamma_mlp | (uintptr_t)L.wq | (uintptr_t)L.wo | (uintptr_t)L.w_gate |
         (uintptr_t)L.w_down | (uintptr_t)L.k_prefix | (uintptr_t)L.v_prefix) & 15u)
      return CASCADE_ERR_INVALID_ARG;  // vector loads and TMA need 16-byte aligned bases
    // input norm (first layer: from the token embeddings; later: after adding the previous MLP output)
    CASCADE_TRY(resid_norm<E>(ctx, T, li == 0 ? st->embed : nullptr, st->tok, li == 0 ? nullptr : &pr, L.gamma_attn,
                              st->eps, nullptr, li == 0 ? K_EMBED_NORM : K_RESID_NORM, s));
    // q, k, v: one projection when the three matrices are stacked in memory, else three
    const size_t es = sizeof(E);
    const bool stacked = (const char*)L.wk == (const char*)L.wq + (size_t)sh.Hq * sh.D * sh.h * es &&
                         (const char*)L.wv == (const char*)L.wk + (size_t)sh.Hkv * sh.D * sh.h * es;
    if (!stacked) return CASCADE_ERR_UNSUPPORTED_SHAPE;
    CASCADE_TRY(project(ctx, L.wq, qkv_cols, sh.h, M, false, K_GEMM_QKV, &pr, s));
    E* k_rot = st->k_tree_out ? (E*)st->k_tree_out + (size_t)li * M * sh.Hkv * sh.D : (E*)ctx->k_rot;
    E* v_rot = st->v_tree_out ? (E*)st->v_tree_out + (size_t)li * M * sh.Hkv * sh.D : (E*)ctx->v_rot;
    {
      KernelScope ks(ctx, K_ROPE_SPLIT, s);
      const int z = cascade_detail::ceil_div((sh.Hq + sh.Hkv) * sh.D / 8, 2 * kRowThreads);  // ~2 pair groups per thread
      k_rope_split<E><<<dim3(T, R, z < 1 ? 1 : z), kRowThreads, 0, s>>>(ctx->gemm_out, pr.n_slices, pr.slice_stride, T, sh.Hq, sh.Hkv,
                                                         sh.D, st->prefix_len, tree->d_depth, st->rope_base,
                                                         (E*)ctx->q_rot, k_rot, v_rot);
    }
    CASCADE_CUDA_TRY(cudaGetLastError());
    if (sh.dtype == CASCADE_BF16)
      CASCADE_TRY(launch_tree_attn_bf16(ctx, tree, (const __nv_bfloat16*)ctx->q_rot, (const __nv_bfloat16*)L.k_prefix,
                                        (const __nv_bfloat16*)L.v_prefix, st->prefix_cap, st->prefix_len,
                                        (const __nv_bfloat16*)k_rot, (const __nv_bfloat16*)v_rot,
                                        (__nv_bfloat16*)ctx->attn_out, true, st->softmax_scale, s));
    else
      CASCADE_TRY(launch_tree_attn_f32(ctx, tree, (const float*)ctx->q_rot, (const float*)L.k_prefix,
                                       (const float*)L.v_prefix, st->prefix_cap, st->prefix_len, (const float*)k_rot,
                                       (const float*)v_rot, (float*)ctx->attn_out, st->softmax_scale, s));
    // output projection, residual, MLP norm
    CASCADE_TRY(project(ctx, L.wo, sh.h, sh.Hq * sh.D, M, true, K_GEMM_O, &pr, s));
    CASCADE_TRY(resid_norm<E>(ctx, T, nullptr, nullptr, &pr, L.gamma_mlp, st->eps, nullptr, K_RESID_NORM, s));
    // gate and up stacked in memory: one projection
    if ((const char*)L.w_up != (const char*)L.w_gate + (size_t)sh.ffn * sh.h * es) return CASCADE_ERR_UNSUPPORTED_SHAPE;
    CASCADE_TRY(project(ctx, L.w_gate, 2 * sh.ffn, sh.h, M, false, K_GEMM_GATE_UP, &pr, s, true));
    {
      const bool bf16 = sh.dtype == CASCADE_BF16;
      KernelScope ks(ctx, K_SWIGLU, s);
      k_swiglu<<<dim3(cascade_detail::ceil_div(sh.ffn / 4, kRowThreads), M), kRowThreads, 0, s>>>(
          ctx->gemm_out, pr.map, pr.slice_stride, sh.ffn, bf16 ? ctx->act : nullptr, operand_layout(M, sh.ffn),
          bf16 ? nullptr : ctx->act_f32);
    }
    CASCADE_CUDA_TRY(cudaGetLastError());
    CASCADE_TRY(project(ctx, L.w_down, sh.h, sh.ffn, M, false, K_GEMM_DOWN, &pr, s));
  }
  // The last MLP output still has to join the residual stream.  The final norm adds it while it reads
  // x; only a caller that wants the hidden states pays for a pass that writes them.
  if (st->hidden_out == nullptr) {
    pending->slices = ctx->gemm_out;
    pending->n = pr.n_slices;
    pending->stride = pr.slice_stride;
    return CASCADE_OK;
  }
  *pending = PendingAdd{};
  return resid_norm<E>(ctx, T, nullptr, nullptr, &pr, nullptr, st->eps, st->hidden_out, K_RESID_ADD, s);
}

}  // namespace

int run_layers(cascade_ctx* ctx, const cascade_tree* tree, const cascade_step* st, PendingAdd* pending, cudaStream_t s) {
  if (ctx->shape.ffn <= 0 || ctx->x == nullptr) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  if (st->layers == nullptr || st->embed == nullptr || st->prefix_len == nullptr) return CASCADE_ERR_INVALID_ARG;
  if (!(st->rope_base > 1.f) || !(st->softmax_scale > 0.f) || !(st->eps >= 0.f)) return CASCADE_ERR_INVALID_ARG;
  if (st->prefix_cap < 0 || st->prefix_cap > ctx->shape.P_max) return CASCADE_ERR_INVALID_ARG;
  if (ctx->shape.dtype == CASCADE_BF16) return run_layers_t<__nv_bfloat16>(ctx, tree, st, pending, s);
  return run_layers_t<float>(ctx, tree, st, pending, s);
}

// What a decode loop needs between two verification steps: the token that follows the accepted path
// (Algorithm 1's final draw from the target distribution with the rejected proposals removed -- the step
// Algorithm 2 leaves out) and the append of the accepted rows' keys / values to the caches.
#include "cascade_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kMaxLayers = 64;

struct CachePtrs {
  void* k[kMaxLayers];
  void* v[kMaxLayers];
};

// grid (depth_max + 1, R, n_layers): row i of the accepted path of prompt b = r mod B goes to cache position
// prefix_len[r] + i of layer blockIdx.z.  Paths that do not fit set the overflow bit and copy nothing.
template <typename E>
__global__ void __launch_bounds__(kThreads) k_kv_append(CachePtrs caches, const E* __restrict__ k_tree,
                                                        const E* __restrict__ v_tree, int B, int T, int row_elems,
                                                        int depth_max, const int32_t* __restrict__ path_nodes,
                                                        const int32_t* __restrict__ path_len, int prefix_cap,
                                                        const int32_t* __restrict__ prefix_len, int* err) {
  const int i = blockIdx.x, r = blockIdx.y, layer = blockIdx.z, R = 2 * B, b = r % B;
  const int len = path_len[b];
  if (i > len) return;
  const int P = prefix_len[r];
  if (P + len + 1 > prefix_cap) {
    if (threadIdx.x == 0 && i == 0 && layer == 0) atomicOr(err, CASCADE_DEV_ERR_OVERFLOW);
    return;
  }
  const int node = path_nodes[(size_t)b * (depth_max + 1) + i];
  const size_t src = (((size_t)layer * R + r) * T + node) * row_elems;
  const size_t dst = ((size_t)r * prefix_cap + P + i) * row_elems;
  // 16-byte pieces: row_elems * sizeof(E) is a multiple of 16
  const int n16 = row_elems * (int)sizeof(E) / 16;
  const uint4* ks = reinterpret_cast<const uint4*>(k_tree + src);
  const uint4* vs = reinterpret_cast<const uint4*>(v_tree + src);
  uint4* kd = reinterpret_cast<uint4*>(static_cast<E*>(caches.k[layer]) + dst);
  uint4* vd = reinterpret_cast<uint4*>(static_cast<E*>(caches.v[layer]) + dst);
  for (int t = threadIdx.x; t < n16; t += kThreads) {
    kd[t] = ks[t];
    vd[t] = vs[t];
  }
}

__global__ void k_bump_prefix(int B, const int32_t* __restrict__ path_len, int prefix_cap, int32_t* prefix_len) {
  const int r = threadIdx.x + blockIdx.x * blockDim.x;
  if (r >= 2 * B) return;
  const int n = path_len[r % B] + 1;
  if (prefix_len[r] + n <= prefix_cap) prefix_len[r] += n;
}

// One CTA per prompt.  Row = logits of the path's end node.  Without a drafter row: the tokens of that node's
// children (all rejected) get weight zero, the others exp(l - max).  With the drafter's distribution p at the end
// node (draft != null) and at least one rejected child: Algorithm 1's correction step, weight [q - p]+ with
// q = softmax(l) (and plain q if nothing is left of it, i.e. p >= q everywhere).  After a fully accepted path
// (the end node has no children) the weight is q's in both modes.  token = first v with cumsum(weight)[v] >
// u * total.  Every thread owns a contiguous run of the vocabulary; sums in double, runs added in index order,
// so that the order of additions does not move the sample.
__global__ void __launch_bounds__(kThreads) k_bonus_token(const float* __restrict__ logits, int T, int V,
                                                          int depth_max, const int32_t* __restrict__ tok,
                                                          const int32_t* __restrict__ child_begin,
                                                          const int32_t* __restrict__ child_count,
                                                          const int32_t* __restrict__ path_nodes,
                                                          const int32_t* __restrict__ path_len,
                                                          const float* __restrict__ u_bonus,
                                                          const float* __restrict__ draft,
                                                          int32_t* __restrict__ token_out,
                                                          float* __restrict__ mass_out) {
  __shared__ int s_rej[CASCADE_MAX_CHILDREN];
  __shared__ float s_redf[kThreads / 32];
  __shared__ double s_part[kThreads];
  __shared__ double s_total;
  __shared__ float s_max;
  __shared__ int s_token;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int end = path_nodes[(size_t)b * (depth_max + 1) + path_len[b]];
  const int cb = child_begin[end], cc = child_count[end];
  if (tid < cc) s_rej[tid] = tok[(size_t)b * T + cb + tid];
  const float* l = logits + ((size_t)b * T + end) * V;
  float m = -INFINITY;
  for (int i = tid; i < V; i += kThreads) m = fmaxf(m, l[i]);
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((tid & 31) == 0) s_redf[tid >> 5] = m;
  __syncthreads();
  if (tid == 0) {
    float x = s_redf[0];
    for (int i = 1; i < kThreads / 32; ++i) x = fmaxf(x, s_redf[i]);
    s_max = x;
    s_token = V - 1;
  }
  __syncthreads();
  m = s_max;
  const int seg = (V + kThreads - 1) / kThreads, v0 = tid * seg, v1 = min(V, v0 + seg);
  // residual mode needs q itself, i.e. the normaliser of the row, before any weight can be formed
  const float* p_row = (draft != nullptr && cc > 0) ? draft + (size_t)b * V : nullptr;
  double inv_z = 0.0;
  int residual = p_row != nullptr;
  if (residual) {
    double z = 0.0;
    for (int v = v0; v < v1; ++v) z += (double)expf(l[v] - m);
    s_part[tid] = z;
    __syncthreads();
    if (tid == 0) {
      double run = 0.0;
      for (int i = 0; i < kThreads; ++i) run += s_part[i];
      s_total = run;
    }
    __syncthreads();
    inv_z = 1.0 / s_total;
    // is anything left of q above p?  (not when the drafter's row equals the target's)
    double r = 0.0;
    for (int v = v0; v < v1; ++v) r += fmax((double)expf(l[v] - m) * inv_z - (double)p_row[v], 0.0);
    const int any = __syncthreads_or(r > 0.0);
    if (!any) residual = 0;
    __syncthreads();
  }
  auto weight = [&](int v) {
    if (residual) return fmax((double)expf(l[v] - m) * inv_z - (double)p_row[v], 0.0);
    if (p_row != nullptr) return (double)expf(l[v] - m);   // nothing left above p: the target row itself
    for (int c = 0; c < cc; ++c)
      if (s_rej[c] == v) return 0.0;
    return (double)expf(l[v] - m);
  };
  double mine = 0.0;
  for (int v = v0; v < v1; ++v) mine += weight(v);
  s_part[tid] = mine;
  __syncthreads();
  if (tid == 0) {  // exclusive prefix over the 256 runs (serial: 256 adds)
    double run = 0.0;
    for (int i = 0; i < kThreads; ++i) {
      const double x = s_part[i];
      s_part[i] = run;
      run += x;
    }
    s_total = run;
  }
  __syncthreads();
  const double total = s_total;
  const double target = (double)u_bonus[b] * total;
  const double before = s_part[tid];
  if (target >= before && target < before + mine) {
    double acc = before;
    for (int v = v0; v < v1; ++v) {
      acc += weight(v);
      if (acc > target) {
        s_token = v;
        break;
      }
    }
  }
  __syncthreads();
  if (tid == 0) {
    token_out[b] = s_token;
    if (mass_out != nullptr && p_row != nullptr) {
      mass_out[b] = residual ? (float)total : 1.f;   // sum of [q - p]+: the probability mass the correction keeps
    } else if (mass_out != nullptr) {
      // remaining mass = total / sum of all weights; the rejected tokens' weights are added back here
      double all = total;
      for (int c = 0; c < cc; ++c) {
        bool dup = false;
        for (int e = 0; e < c; ++e) dup = dup || s_rej[e] == s_rej[c];
        if (!dup) all += (double)expf(l[s_rej[c]] - m);
      }
      mass_out[b] = (float)(total / all);
    }
  }
}

}  // namespace

extern "C" {

int cascade_kv_append(cascade_ctx* ctx, const cascade_tree* tree, int32_t n_layers, const cascade_layer* layers,
                      const void* k_tree, const void* v_tree, const int32_t* path_nodes, const int32_t* path_len,
                      int32_t prefix_cap, int32_t* prefix_len, void* stream) {
  if (ctx == nullptr || tree == nullptr || layers == nullptr || k_tree == nullptr || v_tree == nullptr ||
      path_nodes == nullptr || path_len == nullptr || prefix_len == nullptr)
    return CASCADE_ERR_INVALID_ARG;
  if (tree->ctx != ctx || n_layers < 1 || prefix_cap < 1 || prefix_cap > ctx->shape.P_max) return CASCADE_ERR_INVALID_ARG;
  if (n_layers > kMaxLayers) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  const cascade_shape& sh = ctx->shape;
  CachePtrs cp;
  for (int i = 0; i < n_layers; ++i) {
    if (layers[i].k_prefix == nullptr || layers[i].v_prefix == nullptr) return CASCADE_ERR_INVALID_ARG;
    if (((uintptr_t)layers[i].k_prefix | (uintptr_t)layers[i].v_prefix) & 15u) return CASCADE_ERR_INVALID_ARG;
    cp.k[i] = layers[i].k_prefix;
    cp.v[i] = layers[i].v_prefix;
  }
  if (((uintptr_t)k_tree | (uintptr_t)v_tree) & 15u) return CASCADE_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  ctx->launches = 0;
  const int row_elems = sh.Hkv * sh.D;
  dim3 grid(tree->depth_max + 1, 2 * sh.B, n_layers);
  {
    KernelScope ks(ctx, K_KV_APPEND, s);
    if (sh.dtype == CASCADE_BF16)
      k_kv_append<__nv_bfloat16><<<grid, kThreads, 0, s>>>(cp, (const __nv_bfloat16*)k_tree, (const __nv_bfloat16*)v_tree,
                                                           sh.B, tree->T, row_elems, tree->depth_max, path_nodes, path_len,
                                                           prefix_cap, prefix_len, ctx->dev_error);
    else
      k_kv_append<float><<<grid, kThreads, 0, s>>>(cp, (const float*)k_tree, (const float*)v_tree, sh.B, tree->T, row_elems,
                                                   tree->depth_max, path_nodes, path_len, prefix_cap, prefix_len,
                                                   ctx->dev_error);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  {
    KernelScope ks(ctx, K_KV_APPEND, s);
    k_bump_prefix<<<cascade_detail::ceil_div(2 * sh.B, 128), 128, 0, s>>>(sh.B, path_len, prefix_cap, prefix_len);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

int cascade_bonus_token(cascade_ctx* ctx, const cascade_tree* tree, const float* logits, const int32_t* tok,
                        const float* draft_row, const int32_t* path_nodes, const int32_t* path_len,
                        const float* u_bonus, int32_t* token_out, float* mass_out, void* stream) {
  if (ctx == nullptr || tree == nullptr || logits == nullptr || tok == nullptr || path_nodes == nullptr ||
      path_len == nullptr || u_bonus == nullptr || token_out == nullptr)
    return CASCADE_ERR_INVALID_ARG;
  if (tree->ctx != ctx) return CASCADE_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  ctx->launches = 0;
  {
    KernelScope ks(ctx, K_BONUS_TOKEN, s);
    k_bonus_token<<<ctx->shape.B, kThreads, 0, s>>>(logits, tree->T, ctx->shape.V, tree->depth_max, tok,
                                                    tree->d_child_begin, tree->d_child_count, path_nodes, path_len,
                                                    u_bonus, draft_row, token_out, mass_out);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

}  // extern "C"

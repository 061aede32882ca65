// Relaxed acceptance (Section 4.1-4.2, Eq. 1-3, Algorithm 2) and path selection.
//
//   k_similarity   one CTA per (pair, prompt): cosine of two feature rows (Section 4.1).
//   k_row_stats    one CTA per (tree row, prompt): log-sum-exp of a logits row and the few logits the
//                  rule reads (used when the caller supplies full logits instead of the LM head's
//                  fused statistics).
//   k_accept       one CTA per prompt: a thread per node builds I_j / C_j and their masses; one
//                  thread then threads the TVD budget through the tree in index order (the order in
//                  which Algorithm 2's walk would meet the nodes), takes the accept tests and picks
//                  the path.
//   k_select_path  path selection alone.
#include "cascade_internal.h"

namespace {

constexpr int kMaxT = CASCADE_MAX_TREE_ROWS;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---- cosine of one pair ----------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_similarity(const float* __restrict__ feat, int T, int dim,
                                                    const float* __restrict__ feat_norm,
                                                    const int32_t* __restrict__ pair_a,
                                                    const int32_t* __restrict__ pair_b, int n_pairs,
                                                    float* __restrict__ scores) {
  const int pair = blockIdx.x, b = blockIdx.y;
  const int ia = pair_a[pair], ib = pair_b[pair];
  const float4* fa = reinterpret_cast<const float4*>(feat + ((size_t)b * T + ia) * dim);
  const float4* fb = reinterpret_cast<const float4*>(feat + ((size_t)b * T + ib) * dim);
  float dot = 0.f, na = 0.f, nb = 0.f;
  for (int i = threadIdx.x; i < dim / 4; i += blockDim.x) {
    const float4 x = fa[i], y = fb[i];
    dot += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
    na += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
    nb += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
  }
  __shared__ float red[3][4];
  dot = warp_sum(dot);
  na = warp_sum(na);
  nb = warp_sum(nb);
  const int w = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    red[0][w] = dot;
    red[1][w] = na;
    red[2][w] = nb;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    dot = red[0][0] + red[0][1] + red[0][2] + red[0][3];
    float norm_a, norm_b;
    if (feat_norm != nullptr) {
      norm_a = feat_norm[(size_t)b * T + ia];
      norm_b = feat_norm[(size_t)b * T + ib];
    } else {
      norm_a = sqrtf(red[1][0] + red[1][1] + red[1][2] + red[1][3]);
      norm_b = sqrtf(red[2][0] + red[2][1] + red[2][2] + red[2][3]);
    }
    scores[(size_t)b * n_pairs + pair] = dot / (norm_a * norm_b);
  }
}

// ---- row statistics from materialised logits ------------------------------------------------------
__global__ void __launch_bounds__(256) k_row_stats(const float* __restrict__ logits, int T, int V,
                                                   const int32_t* __restrict__ tok,
                                                   const int32_t* __restrict__ child_begin,
                                                   const int32_t* __restrict__ child_count,
                                                   float* __restrict__ row_lse, float* __restrict__ cand_parent,
                                                   float* __restrict__ cand_gparent) {
  const int row = blockIdx.x, b = blockIdx.y;
  const float* l = logits + ((size_t)b * T + row) * V;
  __shared__ float red[8];
  __shared__ float s_max;
  float m = -INFINITY;
  for (int i = threadIdx.x; i < V; i += blockDim.x) m = fmaxf(m, l[i]);
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    float x = red[0];
    for (int i = 1; i < 8; ++i) x = fmaxf(x, red[i]);
    s_max = x;
  }
  __syncthreads();
  m = s_max;
  float sum = 0.f;
  for (int i = threadIdx.x; i < V; i += blockDim.x) sum += expf(l[i] - m);
  sum = warp_sum(sum);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float x = 0.f;
    for (int i = 0; i < 8; ++i) x += red[i];
    row_lse[(size_t)b * T + row] = m + logf(x);
    if (row == 0 && tok != nullptr) {
      cand_parent[(size_t)b * T] = 0.f;
      cand_gparent[(size_t)b * T] = 0.f;
    }
  }
  if (tok == nullptr) return;
  // children of `row` read their token under this row; so do its grandchildren
  const int cb = child_begin[row], cc = child_count[row];
  for (int i = threadIdx.x; i < cc; i += blockDim.x) {
    const int c = cb + i;
    cand_parent[(size_t)b * T + c] = l[tok[(size_t)b * T + c]];
    if (row == 0) cand_gparent[(size_t)b * T + c] = 0.f;
    const int gb = child_begin[c], gc = child_count[c];
    for (int k = 0; k < gc; ++k) cand_gparent[(size_t)b * T + gb + k] = l[tok[(size_t)b * T + gb + k]];
  }
}

// ---- path selection (one thread) -------------------------------------------------------------------
__device__ void select_path_serial(int T, int depth_max, const int32_t* parent, const int32_t* depth,
                                   const int32_t* child_begin, const int32_t* child_count,
                                   const uint8_t* accept, const float* tvd, int mode, uint8_t* valid_scratch,
                                   int32_t* path_nodes, int32_t* path_len, float* tvd_used) {
  int end = 0;
  if (mode == CASCADE_SELECT_FIRST_ACCEPT) {
    while (true) {
      const int cb = child_begin[end], cc = child_count[end];
      int nxt = -1;
      for (int i = 0; i < cc; ++i)
        if (accept[cb + i]) {
          nxt = cb + i;
          break;
        }
      if (nxt < 0) break;
      end = nxt;
    }
  } else {
    valid_scratch[0] = 1;
    int best_depth = 0;
    for (int j = 1; j < T; ++j) {
      const uint8_t v = accept[j] && valid_scratch[parent[j]];
      valid_scratch[j] = v;
      if (v && depth[j] > best_depth) {
        best_depth = depth[j];
        end = j;
      }
    }
  }
  const int len = depth[end];
  for (int i = depth_max; i > len; --i) path_nodes[i] = -1;
  for (int i = len, node = end; i >= 0; --i, node = parent[node]) path_nodes[i] = node;
  *path_len = len;
  if (tvd_used != nullptr)
    *tvd_used = tvd == nullptr ? 0.f : (child_count[end] > 0 ? tvd[child_begin[end] + child_count[end] - 1] : tvd[end]);
}

__global__ void k_select_path(int T, int depth_max, const int32_t* __restrict__ parent,
                              const int32_t* __restrict__ depth, const int32_t* __restrict__ child_begin,
                              const int32_t* __restrict__ child_count, const uint8_t* __restrict__ accept,
                              const float* __restrict__ tvd_out, int mode, int32_t* __restrict__ path_nodes,
                              int32_t* __restrict__ path_len, float* __restrict__ tvd_used) {
  __shared__ int32_t s_parent[kMaxT], s_depth[kMaxT], s_cb[kMaxT], s_cc[kMaxT];
  __shared__ uint8_t s_accept[kMaxT], s_valid[kMaxT];
  __shared__ float s_tvd[kMaxT];
  const int b = blockIdx.x;
  for (int j = threadIdx.x; j < T; j += blockDim.x) {
    s_parent[j] = parent[j];
    s_depth[j] = depth[j];
    s_cb[j] = child_begin[j];
    s_cc[j] = child_count[j];
    s_accept[j] = accept[(size_t)b * T + j];
    s_tvd[j] = tvd_out ? tvd_out[(size_t)b * T + j] : 0.f;
  }
  __syncthreads();
  if (threadIdx.x == 0)
    select_path_serial(T, depth_max, s_parent, s_depth, s_cb, s_cc, s_accept, tvd_out ? s_tvd : nullptr, mode,
                       s_valid, path_nodes + (size_t)b * (depth_max + 1), path_len + b,
                       tvd_used ? tvd_used + b : nullptr);
}

// index of the unordered sibling pair (x < y) among k siblings, lexicographic order
__device__ __forceinline__ int sib_pair_index(int x, int y, int k) { return x * k - x * (x + 1) / 2 + (y - x - 1); }

// ---- the rule ----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kMaxT) k_accept(
    int T, int depth_max, int n_pairs, const int32_t* __restrict__ parent, const int32_t* __restrict__ depth,
    const int32_t* __restrict__ child_begin, const int32_t* __restrict__ child_count,
    const int32_t* __restrict__ sib_base, const float* __restrict__ scores, const float* __restrict__ row_lse,
    const float* __restrict__ cand_parent, const float* __restrict__ cand_gparent, const int32_t* __restrict__ tok,
    const float* __restrict__ draft_p, const float* __restrict__ uniforms, cascade_params prm,
    uint8_t* __restrict__ accept, float* __restrict__ q_relaxed, float* __restrict__ tvd_out,
    int32_t* __restrict__ near_count, int select_mode, int32_t* __restrict__ path_nodes,
    int32_t* __restrict__ path_len, float* __restrict__ tvd_used) {
  __shared__ int32_t s_parent[kMaxT], s_depth[kMaxT], s_cb[kMaxT], s_cc[kMaxT], s_tok[kMaxT];
  __shared__ float s_q[kMaxT];    // mass of tok[j] under its parent's row
  __shared__ float s_qg[kMaxT];   // mass of tok[j] under its grandparent's row
  __shared__ float s_lse[kMaxT], s_mI[kMaxT], s_mC[kMaxT], s_p[kMaxT], s_u[kMaxT], s_qR[kMaxT], s_tvd[kMaxT];
  __shared__ uint8_t s_has[kMaxT];   // bit 0: I_j non-empty, bit 1: C_j non-empty
  __shared__ uint8_t s_near[kMaxT];
  __shared__ uint8_t s_accept[kMaxT], s_valid[kMaxT];

  const int b = blockIdx.x, j = threadIdx.x;
  const size_t row0 = (size_t)b * T;
  const float* sc = scores + (size_t)b * n_pairs;
  if (j < T) {
    s_parent[j] = parent[j];
    s_depth[j] = depth[j];
    s_cb[j] = child_begin[j];
    s_cc[j] = child_count[j];
    s_tok[j] = tok[row0 + j];
    s_lse[j] = row_lse[row0 + j];
    s_p[j] = draft_p[row0 + j];
    s_u[j] = uniforms[row0 + j];
  }
  __syncthreads();
  if (j < T) {
    float q = 0.f, qg = 0.f;
    if (j >= 1) {
      const int pi = s_parent[j];
      q = expf(cand_parent[row0 + j] - s_lse[pi]);
      if (s_parent[pi] >= 0) qg = expf(cand_gparent[row0 + j] - s_lse[s_parent[pi]]);
    }
    s_q[j] = q;
    s_qg[j] = qg;
  }
  __syncthreads();
  if (j >= 1 && j < T) {
    const int pi = s_parent[j];
    const int cb = s_cb[pi], k = s_cc[pi], me = j - cb;
    const int my_tok = s_tok[j];
    uint32_t imask = 0, near = 0;
    float mI = 0.f, mC = 0.f;
    if (prm.flags & CASCADE_USE_I) {
      const int base = sib_base[pi];
      for (int s = 0; s < k; ++s) {
        if (s == me) continue;
        const float c = sc[base + (s < me ? sib_pair_index(s, me, k) : sib_pair_index(me, s, k))];
        if (fabsf(c - prm.tau_pos) < CASCADE_NEAR) near |= 1;
        if (c >= prm.tau_pos) {
          const int t = s_tok[cb + s];
          bool fresh = t != my_tok;
          for (int e = 0; e < s && fresh; ++e)
            if (((imask >> e) & 1u) && s_tok[cb + e] == t) fresh = false;
          if (fresh) mI += s_q[cb + s];
          imask |= 1u << s;
        }
      }
    }
    uint32_t cmask = 0;
    if (prm.flags & CASCADE_USE_C) {
      const int kb = s_cb[j], kk = s_cc[j];
      const bool self_dist = (prm.flags & CASCADE_CONV_DIST_SELF) != 0;
      for (int s = 0; s < kk; ++s) {
        const int c_node = kb + s;
        const float c = sc[c_node - 1];  // edge (parent[c_node] -> c_node) is pair c_node - 1
        if (fabsf(c - prm.tau_seq) < CASCADE_NEAR) near |= 1;
        if (c >= prm.tau_seq) {
          const int t = s_tok[c_node];
          bool fresh = t != my_tok;
          for (int e = 0; e < k && fresh; ++e)
            if (((imask >> e) & 1u) && s_tok[cb + e] == t) fresh = false;
          for (int e = 0; e < s && fresh; ++e)
            if (((cmask >> e) & 1u) && s_tok[kb + e] == t) fresh = false;
          if (fresh) mC += self_dist ? s_q[c_node] : s_qg[c_node];
          cmask |= 1u << s;
        }
      }
    }
    s_mI[j] = mI;
    s_mC[j] = mC;
    s_has[j] = (imask ? 1 : 0) | (cmask ? 2 : 0);
    s_near[j] = (uint8_t)near;
  }
  __syncthreads();
  if (j == 0) {
    // Budget threading in index order.  Algorithm 2 reaches node i only after accepting i's ancestors
    // and rejecting i's earlier siblings, so its running total on arrival is the total left by the
    // parent (first child) or by the previous sibling.
    s_tvd[0] = 0.f;
    s_qR[0] = 0.f;
    s_accept[0] = 1;
    s_near[0] = 0;
    int n_near = 0;
    for (int i = 1; i < T; ++i) {
      const int pi = s_parent[i];
      float t = (i == s_cb[pi]) ? s_tvd[pi] : s_tvd[i - 1];
      float qR = s_q[i];
      uint8_t near = s_near[i];
      if (s_has[i] & 1) {
        const float m = s_mI[i];
        if (fabsf(t + m - prm.tvd_budget) < CASCADE_NEAR) near |= 2;
        if (t + m <= prm.tvd_budget) {
          qR += m;
          t += m;
        }
      }
      if (s_has[i] & 2) {
        const float m = s_mC[i];
        if (fabsf(t + m - prm.tvd_budget) < CASCADE_NEAR) near |= 2;
        if (t + m <= prm.tvd_budget) {
          qR += m;
          t += m;
        }
      }
      s_tvd[i] = t;
      s_qR[i] = qR;
      uint8_t a = 0;
      const float p = s_p[i];
      if (p > 0.f) {
        const float ratio = qR / p;
        a = s_u[i] < fminf(1.f, ratio) ? 1 : 0;
        if (fabsf(ratio - s_u[i]) < CASCADE_NEAR) near |= 4;
      }
      s_accept[i] = a;
      s_near[i] = near;
      n_near += near ? 1 : 0;
    }
    if (near_count != nullptr) near_count[b] = n_near;
    if (path_nodes != nullptr)
      select_path_serial(T, depth_max, s_parent, s_depth, s_cb, s_cc, s_accept, s_tvd, select_mode, s_valid,
                         path_nodes + (size_t)b * (depth_max + 1), path_len + b, tvd_used ? tvd_used + b : nullptr);
  }
  __syncthreads();
  if (j < T) {
    accept[row0 + j] = s_accept[j];
    if (q_relaxed != nullptr) q_relaxed[row0 + j] = s_qR[j];
    if (tvd_out != nullptr) tvd_out[row0 + j] = s_tvd[j];
  }
}

}  // namespace

int launch_similarity(cascade_ctx* ctx, const cascade_tree* tree, const float* feat, int feat_dim,
                      const float* feat_norm, float* scores, cudaStream_t s) {
  if (tree->n_pairs == 0) return CASCADE_OK;
  dim3 grid(tree->n_pairs, ctx->shape.B);
  {
    KernelScope ks(ctx, K_SIMILARITY, s);
    k_similarity<<<grid, 128, 0, s>>>(feat, tree->T, feat_dim, feat_norm, tree->d_pair_a, tree->d_pair_b,
                                      tree->n_pairs, scores);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

int launch_row_stats_from_logits(cascade_ctx* ctx, const cascade_tree* tree, const float* logits,
                                 const int32_t* tok, float* row_lse, float* cand_parent,
                                 float* cand_gparent, cudaStream_t s) {
  dim3 grid(tree->T, ctx->shape.B);
  {
    KernelScope ks(ctx, K_ROW_STATS, s);
    k_row_stats<<<grid, 256, 0, s>>>(logits, tree->T, ctx->shape.V, tok, tree->d_child_begin, tree->d_child_count,
                                     row_lse, cand_parent, cand_gparent);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

int launch_accept(cascade_ctx* ctx, const cascade_tree* tree, const float* scores, const float* row_lse,
                  const float* cand_parent, const float* cand_gparent, const int32_t* tok,
                  const float* draft_p, const float* uniforms, const cascade_params* prm, uint8_t* accept,
                  float* q_relaxed, float* tvd_out, int32_t* near_count, int select_mode, int32_t* path_nodes,
                  int32_t* path_len, float* tvd_used, cudaStream_t s) {
  KernelScope ks(ctx, K_ACCEPT, s);
  k_accept<<<ctx->shape.B, kMaxT, 0, s>>>(tree->T, tree->depth_max, tree->n_pairs, tree->d_parent, tree->d_depth,
                                          tree->d_child_begin, tree->d_child_count, tree->d_sib_base, scores,
                                          row_lse, cand_parent, cand_gparent, tok, draft_p, uniforms, *prm, accept,
                                          q_relaxed, tvd_out, near_count, select_mode, path_nodes, path_len,
                                          tvd_used);
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

int launch_select_path(cascade_ctx* ctx, const cascade_tree* tree, const uint8_t* accept,
                       const float* tvd_out, int mode, int32_t* path_nodes, int32_t* path_len,
                       float* tvd_used, cudaStream_t s) {
  KernelScope ks(ctx, K_SELECT_PATH, s);
  k_select_path<<<ctx->shape.B, 128, 0, s>>>(tree->T, tree->depth_max, tree->d_parent, tree->d_depth,
                                             tree->d_child_begin, tree->d_child_count, accept, tvd_out, mode,
                                             path_nodes, path_len, tvd_used);
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

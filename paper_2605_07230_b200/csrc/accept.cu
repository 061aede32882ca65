// Relaxed acceptance (Section 4.1-4.2, Eq. 1-3, Algorithm 2) and path selection.
//
//   k_tail         the tail of a verification step in one launch.  CTAs 0..n_pairs-1 of a prompt each
//                  take the cosine of one (node, node) feature pair (Section 4.1); the next CTAs fold the
//                  LM head's per-tile softmax partials into the log-sum-exp of each logits row (a warp
//                  per row); the CTA of a prompt that finishes last then runs the acceptance rule and
//                  picks the path.  Any of the three parts can be switched off, which gives the
//                  stand-alone entry points.
//   k_row_stats    one CTA per (tree row, prompt): log-sum-exp of a logits row and the few logits the
//                  rule reads (used when the caller supplies full logits instead of the LM head's
//                  fused statistics).
//   k_select_path  path selection alone.
//
// The rule itself (accept_block) is one CTA per prompt with a thread per node:
//   1. q_j, and the mass of tok[j] under the grandparent's row;
//   2. I_j / C_j and their masses (distinct tokens only);
//   3. the TVD budget is threaded through the tree one level at a time: a thread per parent walks its
//      children in order, which is the order Algorithm 2's walk would meet them, so every node gets the
//      running total the walk would hold on arriving there;
//   4. accept tests, one per thread;
//   5. path selection on bit masks: a node lies on an all-accepted path iff its packed
//      ancestor-or-self mask is covered by the accept mask.
#include "cascade_internal.h"

namespace {

constexpr int kMaxT = CASCADE_MAX_TREE_ROWS;
constexpr int kTailThreads = 256;
constexpr int kMaxPairsSmem = kMaxT * (CASCADE_MAX_CHILDREN + 1) / 2 + kMaxT;
static_assert(kTailThreads == kMaxT, "one thread per tree row");

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

struct TreeDev {
  int T, depth_max, n_pairs;
  int pairs_stride;     // row length of the scores arrays (= n_pairs unless the tree was built on the device)
  const int32_t* meta;  // device-built tree: meta[0] = its pair count (the host does not know it); else null
  const int32_t *parent, *depth, *child_begin, *child_count, *sib_base, *pair_a, *pair_b;
  const uint64_t* anc;
};
__device__ __forceinline__ int pair_count(const TreeDev& tr) { return tr.meta != nullptr ? tr.meta[0] : tr.n_pairs; }

struct AcceptIO {
  const float* scores;        // [B, n_pairs]
  const float* row_lse;       // [B, T]
  const float* cand_parent;   // [B, T]
  const float* cand_gparent;  // [B, T]
  const int32_t* tok;
  const float* draft_p;
  const float* uniforms;
  cascade_params prm;
  uint8_t* accept;
  float* q_relaxed;
  float* tvd_out;
  int32_t* near_count;
  int select_mode;
  int32_t* path_nodes;  // null: no path selection
  int32_t* path_len;
  float* tvd_used;
};

struct TailArgs {
  // cosines
  const float* feat;
  int feat_dim;
  const float* feat_norm;
  float* scores_out;
  int n_pair_blocks;  // CTAs per prompt that take cosines (each strides over the pair list)
  // row log-sum-exp from the LM head's partials
  const float2* part;
  int part_ld, n_tiles, n_lse_blocks;
  float* row_lse_out;
  // the rule
  int do_accept;
  unsigned int* counters;  // one per prompt, zero between launches
};

// index of the unordered sibling pair (x < y) among k siblings, lexicographic order
__device__ __forceinline__ int sib_pair_index(int x, int y, int k) { return x * k - x * (x + 1) / 2 + (y - x - 1); }

// ---- the rule: whole CTA (kTailThreads threads), one prompt ------------------------------------------
__device__ void accept_block(const TreeDev& tr, const AcceptIO& io, int b) {
  __shared__ int32_t s_parent[kMaxT], s_depth[kMaxT], s_cb[kMaxT], s_cc[kMaxT], s_tok[kMaxT], s_sib[kMaxT];
  __shared__ float s_q[kMaxT];    // mass of tok[j] under its parent's row
  __shared__ float s_qg[kMaxT];   // mass of tok[j] under its grandparent's row
  __shared__ float s_lse[kMaxT], s_mI[kMaxT], s_mC[kMaxT], s_qR[kMaxT], s_tvd[kMaxT];
  __shared__ uint8_t s_has[kMaxT];   // bit 0: I_j non-empty, bit 1: C_j non-empty
  __shared__ uint8_t s_near[kMaxT];
  __shared__ uint8_t s_accept[kMaxT];
  __shared__ float s_scores[kMaxPairsSmem];
  __shared__ uint32_t s_mask[2][kMaxT / 32];  // [0] accept bits, [1] "first accepted among its siblings" bits
  __shared__ uint32_t s_best[kTailThreads / 32];

  const int T = tr.T, j = threadIdx.x;
  const size_t row0 = (size_t)b * T;
  const cascade_params prm = io.prm;
  const int n_pairs = min(pair_count(tr), tr.pairs_stride);
  for (int i = j; i < n_pairs; i += kTailThreads) s_scores[i] = __ldcg(io.scores + (size_t)b * tr.pairs_stride + i);
  // every global read of this block is issued here, in one round trip
  float my_p = 0.f, my_u = 1.f, my_cp = 0.f, my_cg = 0.f;
  uint64_t my_anc[kMaxT / 64] = {0, 0, 0, 0};
  if (j < T) {
    s_parent[j] = tr.parent[j];
    s_depth[j] = tr.depth[j];
    s_cb[j] = tr.child_begin[j];
    s_cc[j] = tr.child_count[j];
    s_sib[j] = tr.sib_base[j];
    s_tok[j] = io.tok[row0 + j];
    s_lse[j] = __ldcg(io.row_lse + row0 + j);
    my_p = io.draft_p[row0 + j];
    my_u = io.uniforms[row0 + j];
    my_cp = __ldcg(io.cand_parent + row0 + j);
    my_cg = __ldcg(io.cand_gparent + row0 + j);
#pragma unroll
    for (int w = 0; w < kMaxT / 64; ++w) my_anc[w] = tr.anc[(size_t)j * 4 + w];
  }
  __syncthreads();
  // 1. target mass of each drafted token under its parent's (and grandparent's) distribution
  if (j < T) {
    float q = 0.f, qg = 0.f;
    if (j >= 1) {
      const int pi = s_parent[j];
      q = expf(my_cp - s_lse[pi]);
      if (s_parent[pi] >= 0) qg = expf(my_cg - s_lse[s_parent[pi]]);
    }
    s_q[j] = q;
    s_qg[j] = qg;
  }
  __syncthreads();
  // 2. interchangeable siblings (Eq. 1) and convergent children (Eq. 2) with their masses (Eq. 3)
  if (j >= 1 && j < T) {
    const int pi = s_parent[j];
    const int cb = s_cb[pi], k = s_cc[pi], me = j - cb;
    const int my_tok = s_tok[j];
    uint32_t imask = 0, near = 0;
    float mI = 0.f, mC = 0.f;
    if (prm.flags & CASCADE_USE_I) {
      const int base = s_sib[pi];
      for (int s = 0; s < k; ++s) {
        if (s == me) continue;
        const float c = s_scores[base + (s < me ? sib_pair_index(s, me, k) : sib_pair_index(me, s, k))];
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
        const float c = s_scores[c_node - 1];  // edge (parent[c_node] -> c_node) is pair c_node - 1
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
  if (j == 0) {
    s_tvd[0] = 0.f;
    s_qR[0] = 0.f;
    s_near[0] = 0;
  }
  __syncthreads();
  // 3. budget threading, one level per round.  Algorithm 2 reaches node i only after accepting i's
  // ancestors and rejecting i's earlier siblings, so its running total on arrival is the total left by
  // the parent (first child) or by the previous sibling.
  for (int d = 0; d < tr.depth_max; ++d) {
    if (j < T && s_depth[j] == d && s_cc[j] > 0) {
      float t = s_tvd[j];
      const int cb = s_cb[j], cc = s_cc[j];
      // four children at a time: their data is read first (independent shared-memory loads), the
      // running total then moves through registers only
      for (int base = 0; base < cc; base += 4) {
        float q4[4], mI4[4], mC4[4];
        uint32_t has4[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = cb + min(base + u, cc - 1);
          q4[u] = s_q[i];
          mI4[u] = s_mI[i];
          mC4[u] = s_mC[i];
          has4[u] = s_has[i];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (base + u < cc) {
            const int i = cb + base + u;
            float qR = q4[u];
            uint32_t near = 0;
            if (has4[u] & 1u) {
              const float m = mI4[u];
              if (fabsf(t + m - prm.tvd_budget) < CASCADE_NEAR) near |= 2;
              if (t + m <= prm.tvd_budget) {
                qR += m;
                t += m;
              }
            }
            if (has4[u] & 2u) {
              const float m = mC4[u];
              if (fabsf(t + m - prm.tvd_budget) < CASCADE_NEAR) near |= 2;
              if (t + m <= prm.tvd_budget) {
                qR += m;
                t += m;
              }
            }
            s_tvd[i] = t;
            s_qR[i] = qR;
            if (near) s_near[i] |= (uint8_t)near;
          }
        }
      }
    }
    __syncthreads();
  }
  // 4. accept tests (Algorithm 1's test on the relaxed probability)
  uint8_t a = 0, near = 0;
  if (j == 0) {
    a = 1;
  } else if (j < T) {
    near = s_near[j];
    if (my_p > 0.f) {
      const float ratio = s_qR[j] / my_p;
      a = my_u < fminf(1.f, ratio) ? 1 : 0;
      if (fabsf(ratio - my_u) < CASCADE_NEAR) near |= 4;
    }
  }
  if (j < T) {
    s_accept[j] = a;
    io.accept[row0 + j] = a;
    if (io.q_relaxed != nullptr) io.q_relaxed[row0 + j] = s_qR[j];
    if (io.tvd_out != nullptr) io.tvd_out[row0 + j] = s_tvd[j];
  }
  const uint32_t acc_bits = __ballot_sync(0xffffffffu, a != 0);
  if ((j & 31) == 0) s_mask[0][j >> 5] = acc_bits;
  const int n_near = __syncthreads_count(near != 0);
  if (j == 0 && io.near_count != nullptr) io.near_count[b] = n_near;
  if (io.path_nodes == nullptr) return;
  // 5. path selection
  bool first = a != 0;
  if (j >= 1 && j < T && first) {
    for (int i = s_cb[s_parent[j]]; i < j; ++i)
      if (s_accept[i]) first = false;   // an earlier sibling was accepted: Algorithm 2 never looks at j
  }
  const uint32_t first_bits = __ballot_sync(0xffffffffu, first);
  if ((j & 31) == 0) s_mask[1][j >> 5] = first_bits;
  __syncthreads();
  const uint32_t* cover = s_mask[io.select_mode == CASCADE_SELECT_FIRST_ACCEPT ? 1 : 0];
  uint32_t key = 0;  // (depth, smallest index first) of a node whose whole path is covered
  if (j < T) {
    bool on_path = true;
#pragma unroll
    for (int w = 0; w < kMaxT / 64; ++w) {
      const uint64_t need = my_anc[w];
      const uint64_t have = (uint64_t)cover[2 * w] | ((uint64_t)cover[2 * w + 1] << 32);
      if (need & ~have) on_path = false;
    }
    if (on_path) key = ((uint32_t)s_depth[j] << 16) | (uint32_t)(0xFFFF - j);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
  if ((j & 31) == 0) s_best[j >> 5] = key;
  __syncthreads();
  if (j == 0) {
    for (int w = 1; w < kTailThreads / 32; ++w) key = max(key, s_best[w]);
    const int end = 0xFFFF - (int)(key & 0xFFFFu);
    const int len = s_depth[end];
    int32_t* nodes = io.path_nodes + (size_t)b * (tr.depth_max + 1);
    for (int i = tr.depth_max; i > len; --i) nodes[i] = -1;
    for (int i = len, node = end; i >= 0; --i, node = s_parent[node]) nodes[i] = node;
    io.path_len[b] = len;
    if (io.tvd_used != nullptr) io.tvd_used[b] = s_cc[end] > 0 ? s_tvd[s_cb[end] + s_cc[end] - 1] : s_tvd[end];
  }
}

// ---- tail of the step ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTailThreads) k_tail(const TreeDev tr, const TailArgs ta, const AcceptIO io) {
  const int b = blockIdx.y, blk = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_pair_blocks = ta.feat != nullptr ? ta.n_pair_blocks : 0;
  if (blk < n_pair_blocks) {
    // cosines: one pair per CTA when the host knows the pair count, a strided share of the list otherwise
    __shared__ float red[3][kTailThreads / 32];
    const int n_pairs = min(pair_count(tr), tr.pairs_stride);
    for (int pi = blk; pi < n_pairs; pi += n_pair_blocks) {
      const int ia = tr.pair_a[pi], ib = tr.pair_b[pi];
      const float4* fa = reinterpret_cast<const float4*>(ta.feat + ((size_t)b * tr.T + ia) * ta.feat_dim);
      const float4* fb = reinterpret_cast<const float4*>(ta.feat + ((size_t)b * tr.T + ib) * ta.feat_dim);
      float dot = 0.f, na = 0.f, nb = 0.f;
      for (int i = threadIdx.x; i < ta.feat_dim / 4; i += kTailThreads) {
        const float4 x = fa[i], y = fb[i];
        dot += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
        na += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
        nb += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
      }
      dot = warp_sum(dot);
      na = warp_sum(na);
      nb = warp_sum(nb);
      __syncthreads();  // the previous pair's sums have been read
      if (lane == 0) {
        red[0][warp] = dot;
        red[1][warp] = na;
        red[2][warp] = nb;
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        dot = na = nb = 0.f;
        for (int w = 0; w < kTailThreads / 32; ++w) {
          dot += red[0][w];
          na += red[1][w];
          nb += red[2][w];
        }
        float norm_a, norm_b;
        if (ta.feat_norm != nullptr) {
          norm_a = ta.feat_norm[(size_t)b * tr.T + ia];
          norm_b = ta.feat_norm[(size_t)b * tr.T + ib];
        } else {
          norm_a = sqrtf(na);
          norm_b = sqrtf(nb);
        }
        ta.scores_out[(size_t)b * tr.pairs_stride + pi] = dot / (norm_a * norm_b);
      }
    }
  } else if (blk < n_pair_blocks + ta.n_lse_blocks) {
    // log-sum-exp of one logits row per warp from the per-tile (max, sum of exp) partials
    const int row = (blk - n_pair_blocks) * (kTailThreads / 32) + warp;
    if (row < tr.T) {
      const float2* pr = ta.part + ((size_t)b * tr.T + row) * ta.part_ld;
      // 16 partials per lane per round, all loads of a round in flight together
      float mx = -INFINITY, sum = 0.f;
      for (int t0 = 0; t0 < ta.n_tiles; t0 += 32 * 16) {
        float2 ms[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int t = t0 + i * 32 + lane;
          ms[i] = t < ta.n_tiles ? __ldcg(&pr[t]) : make_float2(-INFINITY, 0.f);
        }
        float m2 = mx;
#pragma unroll
        for (int i = 0; i < 16; ++i) m2 = fmaxf(m2, ms[i].x);
        if (m2 != -INFINITY) {
          sum *= __expf(mx - m2);
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (ms[i].x != -INFINITY) sum += ms[i].y * __expf(ms[i].x - m2);
        }
        mx = m2;
      }
      const float m_all = warp_max(mx);
      sum = warp_sum(mx == -INFINITY ? 0.f : sum * __expf(mx - m_all));
      mx = m_all;
      if (lane == 0) ta.row_lse_out[(size_t)b * tr.T + row] = mx + logf(sum);
    }
  }
  if (!ta.do_accept) return;
  // the CTA of this prompt that finishes last runs the rule
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int ticket = atomicAdd(ta.counters + b, 1u);
    s_last = ticket == gridDim.x - 1;
    if (s_last) ta.counters[b] = 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  accept_block(tr, io, b);
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
  // 16 bytes per lane where the row allows it (V is a multiple of 8; the base may not be aligned)
  const bool vec = (reinterpret_cast<uintptr_t>(l) & 15u) == 0 && (V & 3) == 0;
  const float4* l4 = reinterpret_cast<const float4*>(l);
  float m = -INFINITY;
  if (vec) {
#pragma unroll 4
    for (int i = threadIdx.x; i < V / 4; i += blockDim.x) {
      const float4 x = l4[i];
      m = fmaxf(fmaxf(m, fmaxf(x.x, x.y)), fmaxf(x.z, x.w));
    }
  } else {
    for (int i = threadIdx.x; i < V; i += blockDim.x) m = fmaxf(m, l[i]);
  }
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
  if (vec) {
#pragma unroll 4
    for (int i = threadIdx.x; i < V / 4; i += blockDim.x) {
      const float4 x = l4[i];
      sum += (expf(x.x - m) + expf(x.y - m)) + (expf(x.z - m) + expf(x.w - m));
    }
  } else {
    for (int i = threadIdx.x; i < V; i += blockDim.x) sum += expf(l[i] - m);
  }
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

// ---- path selection alone (one thread per prompt) ------------------------------------------------------
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
  if (threadIdx.x != 0) return;
  int end = 0;
  if (mode == CASCADE_SELECT_FIRST_ACCEPT) {
    while (true) {
      const int cb = s_cb[end], cc = s_cc[end];
      int nxt = -1;
      for (int i = 0; i < cc; ++i)
        if (s_accept[cb + i]) {
          nxt = cb + i;
          break;
        }
      if (nxt < 0) break;
      end = nxt;
    }
  } else {
    s_valid[0] = 1;
    int best_depth = 0;
    for (int j = 1; j < T; ++j) {
      const uint8_t v = s_accept[j] && s_valid[s_parent[j]];
      s_valid[j] = v;
      if (v && s_depth[j] > best_depth) {
        best_depth = s_depth[j];
        end = j;
      }
    }
  }
  const int len = s_depth[end];
  int32_t* nodes = path_nodes + (size_t)b * (depth_max + 1);
  for (int i = depth_max; i > len; --i) nodes[i] = -1;
  for (int i = len, node = end; i >= 0; --i, node = s_parent[node]) nodes[i] = node;
  path_len[b] = len;
  if (tvd_used != nullptr)
    tvd_used[b] = tvd_out == nullptr ? 0.f : (s_cc[end] > 0 ? s_tvd[s_cb[end] + s_cc[end] - 1] : s_tvd[end]);
}

TreeDev tree_dev(const cascade_tree* tree) {
  TreeDev t;
  t.T = tree->T;
  t.depth_max = tree->depth_max;
  t.n_pairs = tree->n_pairs;
  t.pairs_stride = tree->n_pairs;
  t.meta = tree->device_built ? tree->d_meta : nullptr;
  t.parent = tree->d_parent;
  t.depth = tree->d_depth;
  t.child_begin = tree->d_child_begin;
  t.child_count = tree->d_child_count;
  t.sib_base = tree->d_sib_base;
  t.pair_a = tree->d_pair_a;
  t.pair_b = tree->d_pair_b;
  t.anc = tree->d_anc;
  return t;
}

}  // namespace

int launch_tail(cascade_ctx* ctx, const cascade_tree* tree, const TailWork& w, cudaStream_t s) {
  TailArgs ta = {};
  AcceptIO io = {};
  const int B = ctx->shape.B;
  if (w.feat != nullptr && tree->n_pairs > 0) {
    ta.feat = w.feat;
    ta.feat_dim = w.feat_dim;
    ta.feat_norm = w.feat_norm;
    ta.scores_out = w.scores;
    // a tree built on the device has an unknown number of pairs (n_pairs is then the row length it may fill):
    // a fixed number of CTAs shares the list
    ta.n_pair_blocks = tree->device_built ? (tree->n_pairs < 128 ? tree->n_pairs : 128) : tree->n_pairs;
  }
  if (w.part != nullptr) {
    ta.part = w.part;
    ta.part_ld = w.part_ld;
    ta.n_tiles = w.n_tiles;
    ta.n_lse_blocks = cascade_detail::ceil_div(tree->T, kTailThreads / 32);
    ta.row_lse_out = w.row_lse;
  }
  ta.do_accept = w.prm != nullptr;
  ta.counters = ctx->tail_counters;
  if (ta.do_accept) {
    io.scores = w.scores;
    io.row_lse = w.row_lse;
    io.cand_parent = w.cand_parent;
    io.cand_gparent = w.cand_gparent;
    io.tok = w.tok;
    io.draft_p = w.draft_p;
    io.uniforms = w.uniforms;
    io.prm = *w.prm;
    io.accept = w.accept;
    io.q_relaxed = w.q_relaxed;
    io.tvd_out = w.tvd_out;
    io.near_count = w.near_count;
    io.select_mode = w.select_mode;
    io.path_nodes = w.path_nodes;
    io.path_len = w.path_len;
    io.tvd_used = w.tvd_used;
  }
  int blocks = (ta.feat != nullptr ? ta.n_pair_blocks : 0) + ta.n_lse_blocks;
  if (blocks == 0) {
    if (!ta.do_accept) return CASCADE_OK;
    blocks = 1;  // nothing to prepare: a single CTA per prompt runs the rule
  }
  dim3 grid(blocks, B);
  {
    KernelScope ks(ctx, w.kernel_id, s);
    k_tail<<<grid, kTailThreads, 0, s>>>(tree_dev(tree), ta, io);
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

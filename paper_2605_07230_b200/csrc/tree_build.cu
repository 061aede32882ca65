// The draft-tree descriptor built on the device from a device-resident parent[] (drafters that grow a different
// tree every step -- the dynamic trees of Section 2's related work -- without a host round trip): what
// cascade_tree_create computes on the host, by one CTA with a thread per tree row.
//
//   validated first, nothing is written before:  parent[0] = -1;  0 <= parent[j] < j;  depth never decreases with
//   the index (breadth-first order);  parent never decreases (sibling groups contiguous);  at most
//   CASCADE_MAX_CHILDREN children per node;  depth <= depth_cap;  pairs <= pairs_cap
//   then: depth, child ranges, first sibling pair of every parent, the pair list (edge (parent[j], j) at index
//   j - 1, then the unordered sibling pairs of each parent in order), the packed ancestor-or-self mask, and the
//   pair count in meta[0] (the host never learns it: consumers read it from there).
// A tree that fails a check sets bit CASCADE_DEV_ERR_BAD_TREE of the context's error word, and a neutral
// descriptor is installed instead (every row a leaf below the root, no pairs), so that whatever is enqueued next
// with the new row count keeps every index in range; its results mean nothing until a valid tree is installed.
#include "cascade_internal.h"

namespace {

constexpr int kMaxT = CASCADE_MAX_TREE_ROWS;

struct TreeOut {
  int32_t *parent, *depth, *child_begin, *child_count, *sib_base, *pair_a, *pair_b, *meta;
  uint64_t* anc;
};

__global__ void __launch_bounds__(kMaxT) k_build_tree(int T, int depth_cap, int pairs_cap,
                                                      const int32_t* __restrict__ parent_in, TreeOut o, int* err) {
  __shared__ int32_t s_parent[kMaxT], s_depth[kMaxT], s_cb[kMaxT], s_cc[kMaxT], s_sib[kMaxT];
  __shared__ int s_bad, s_pairs;
  const int j = threadIdx.x;
  if (j == 0) s_bad = 0;
  s_cb[j] = 0;
  s_cc[j] = 0;
  __syncthreads();
  int p = -1;
  if (j < T) {
    p = parent_in[j];
    if (j == 0 ? p != -1 : (p < 0 || p >= j)) s_bad = 1;
    s_parent[j] = p;
  }
  __syncthreads();
  // every barrier below is reached by all threads; the work between them is predicated
  const bool walk = s_bad == 0 && j < T;   // parent indices are all smaller than their rows: walks to the root end
  int d = 0;
  uint64_t a[4] = {0, 0, 0, 0};            // ancestor-or-self mask, kept in registers until the checks are through
  if (walk) {
    for (int i = j; i >= 0; i = s_parent[i]) {
      a[i >> 6] |= 1ull << (i & 63);
      if (i != j) ++d;
    }
    s_depth[j] = d;
    if (d > depth_cap) s_bad = 1;
  }
  __syncthreads();
  if (walk && j >= 1) {
    if (d < s_depth[j - 1]) s_bad = 1;                      // breadth-first order
    if (j >= 2 && p < s_parent[j - 1]) s_bad = 1;           // sibling groups contiguous
    if (j == 1 || p != s_parent[j - 1]) s_cb[p] = j;        // first child of p
  }
  __syncthreads();
  if (walk && j >= 1 && (j == T - 1 || s_parent[j + 1] != p)) {   // last child of p
    s_cc[p] = j - s_cb[p] + 1;
    if (s_cc[p] > CASCADE_MAX_CHILDREN) s_bad = 1;
  }
  __syncthreads();
  if (j == 0 && s_bad == 0) {
    int n = T - 1;
    for (int q = 0; q < T; ++q) {
      s_sib[q] = n;
      n += s_cc[q] * (s_cc[q] - 1) / 2;
    }
    s_pairs = n;
    if (n > pairs_cap) s_bad = 1;
  }
  __syncthreads();
  const bool ok = s_bad == 0;
  if (ok && j < T) {
    o.parent[j] = p;
    o.depth[j] = d;
    o.child_begin[j] = s_cb[j];
    o.child_count[j] = s_cc[j];
    o.sib_base[j] = s_sib[j];
#pragma unroll
    for (int w = 0; w < 4; ++w) o.anc[(size_t)j * 4 + w] = a[w];
    if (j >= 1) {
      o.pair_a[j - 1] = p;
      o.pair_b[j - 1] = j;
    }
    int at = s_sib[j];
    const int cb = s_cb[j], k = s_cc[j];
    for (int x = 0; x < k; ++x)
      for (int y = x + 1; y < k; ++y) {
        o.pair_a[at] = cb + x;
        o.pair_b[at++] = cb + y;
      }
    if (j == 0) {
      o.meta[0] = s_pairs;
      o.meta[1] = s_depth[T - 1];
      o.meta[2] = 1;
    }
  }
  if (!ok) {
    if (j == 0) {
      atomicOr(err, CASCADE_DEV_ERR_BAD_TREE);
      o.meta[0] = 0;
      o.meta[1] = T > 1 ? 1 : 0;
      o.meta[2] = 0;
    }
    if (j < T) {
      o.parent[j] = j == 0 ? -1 : 0;
      o.depth[j] = j == 0 ? 0 : 1;
      o.child_begin[j] = 0;
      o.child_count[j] = 0;
      o.sib_base[j] = 0;
      uint64_t n[4] = {1ull, 0, 0, 0};    // the root and the row itself
      n[j >> 6] |= 1ull << (j & 63);
#pragma unroll
      for (int w = 0; w < 4; ++w) o.anc[(size_t)j * 4 + w] = n[w];
    }
  }
}

}  // namespace

int launch_build_tree(cascade_ctx* ctx, cascade_tree* tree, int T, int depth_cap, int pairs_cap,
                      const int32_t* parent_dev, cudaStream_t s) {
  TreeOut o;
  o.parent = tree->d_parent;
  o.depth = tree->d_depth;
  o.child_begin = tree->d_child_begin;
  o.child_count = tree->d_child_count;
  o.sib_base = tree->d_sib_base;
  o.pair_a = tree->d_pair_a;
  o.pair_b = tree->d_pair_b;
  o.meta = tree->d_meta;
  o.anc = tree->d_anc;
  {
    KernelScope ks(ctx, K_BUILD_TREE, s);
    k_build_tree<<<1, kMaxT, 0, s>>>(T, depth_cap, pairs_cap, parent_dev, o, ctx->dev_error);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

// cascade_accept_static: similarity scores + relaxed acceptance + path selection for callers that
// cannot allocate device memory.  It needs no context and no tree object (both of which come from
// cudaMalloc): the few hundred kilobytes the tail kernel wants besides its inputs and outputs -- the
// draft tree's device-side descriptor, the cosine scores and the per-prompt "last CTA" counters -- live
// in one file-scope __device__ array that every GPU loading the library carries until the process ends.
#include <cstring>
#include <mutex>
#include <vector>

#include "cascade_internal.h"

namespace {

constexpr int kMaxB = CASCADE_STATIC_MAX_PROMPTS;
constexpr int kMaxT = CASCADE_MAX_TREE_ROWS;
constexpr int kMaxPairs = kMaxT * (CASCADE_MAX_CHILDREN + 1) / 2 + kMaxT;

// Fixed layout of the scratch array (every region 256-byte aligned).
struct Layout {
  static constexpr size_t kInts = 5 * (size_t)kMaxT + 2 * (size_t)kMaxPairs;  // parent, depth, child_begin,
                                                                               // child_count, sib_base, pair_a, pair_b
  static constexpr size_t off_ints = 0;
  static constexpr size_t off_anc = (off_ints + kInts * 4 + 255) / 256 * 256;
  static constexpr size_t off_counters = (off_anc + (size_t)kMaxT * 4 * 8 + 255) / 256 * 256;
  static constexpr size_t off_scores = (off_counters + (size_t)kMaxB * 4 + 255) / 256 * 256;
  static constexpr size_t total = (off_scores + (size_t)kMaxB * kMaxPairs * 4 + 255) / 256 * 256;
};

static __device__ __align__(256) unsigned char g_static_scratch[Layout::total];

// In host code the array's name is only a handle for the runtime, never a device address: the address
// each device gave it is looked up once per device and remembered here.
constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

int scratch_address(unsigned char** out) {
  int dev = 0;
  CASCADE_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    CASCADE_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return CASCADE_OK;
}

}  // namespace

extern "C" int cascade_accept_static(int32_t B, int32_t T, const int32_t* parent, const float* feat, int32_t feat_dim,
                                     const float* feat_norm, const float* row_lse, const float* cand_parent,
                                     const float* cand_gparent, const int32_t* tok, const float* draft_p,
                                     const float* uniforms, const cascade_params* params, int32_t select_mode,
                                     uint8_t* accept, float* q_relaxed, float* tvd_out, int32_t* near_count,
                                     int32_t* path_nodes, int32_t* path_len, float* tvd_used, void* stream) {
  if (parent == nullptr || feat == nullptr || row_lse == nullptr || cand_parent == nullptr ||
      cand_gparent == nullptr || tok == nullptr || draft_p == nullptr || uniforms == nullptr || params == nullptr ||
      accept == nullptr || path_nodes == nullptr || path_len == nullptr)
    return CASCADE_ERR_INVALID_ARG;
  if (B < 1 || T < 1 || feat_dim < 4 || feat_dim % 4 != 0) return CASCADE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(feat) & 15u) != 0) return CASCADE_ERR_INVALID_ARG;
  if (B > kMaxB || T > kMaxT) return CASCADE_ERR_UNSUPPORTED_SHAPE;  // beyond what the static array holds
  if (!(params->tvd_budget >= 0.f) || params->tau_pos != params->tau_pos || params->tau_seq != params->tau_seq ||
      (params->flags & ~(CASCADE_USE_I | CASCADE_USE_C | CASCADE_CONV_DIST_SELF)))
    return CASCADE_ERR_INVALID_ARG;
  if (select_mode != CASCADE_SELECT_LONGEST && select_mode != CASCADE_SELECT_FIRST_ACCEPT)
    return CASCADE_ERR_INVALID_ARG;

  // the tree's descriptor, built on the host exactly as the tree object would hold it
  if (parent[0] != -1) return CASCADE_ERR_BAD_TREE;
  std::vector<int32_t> ints(Layout::kInts, 0);
  int32_t* h_parent = ints.data();
  int32_t* h_depth = h_parent + kMaxT;
  int32_t* h_cb = h_depth + kMaxT;
  int32_t* h_cc = h_cb + kMaxT;
  int32_t* h_sib = h_cc + kMaxT;
  int32_t* h_pa = h_sib + kMaxT;
  int32_t* h_pb = h_pa + kMaxPairs;
  int depth_max = 0;
  h_parent[0] = -1;
  for (int j = 1; j < T; ++j) {
    const int p = parent[j];
    if (p < 0 || p >= j) return CASCADE_ERR_BAD_TREE;
    h_parent[j] = p;
    h_depth[j] = h_depth[p] + 1;
    if (h_depth[j] < h_depth[j - 1]) return CASCADE_ERR_BAD_TREE;  // breadth-first order
    if (j > 1 && p < parent[j - 1]) return CASCADE_ERR_BAD_TREE;   // sibling groups contiguous
    if (h_cc[p] == 0) h_cb[p] = j;
    if (++h_cc[p] > CASCADE_MAX_CHILDREN) return CASCADE_ERR_UNSUPPORTED_SHAPE;
    depth_max = h_depth[j];
  }
  int n_pairs = 0;
  for (int j = 1; j < T; ++j) {  // edge (parent[j], j) is pair j - 1
    h_pa[n_pairs] = parent[j];
    h_pb[n_pairs++] = j;
  }
  for (int p = 0; p < T; ++p) {  // then the sibling pairs of each parent
    h_sib[p] = n_pairs;
    for (int x = 0; x < h_cc[p]; ++x)
      for (int y = x + 1; y < h_cc[p]; ++y) {
        if (n_pairs >= kMaxPairs) return CASCADE_ERR_UNSUPPORTED_SHAPE;
        h_pa[n_pairs] = h_cb[p] + x;
        h_pb[n_pairs++] = h_cb[p] + y;
      }
  }
  std::vector<uint64_t> anc((size_t)kMaxT * 4, 0);
  for (int j = 0; j < T; ++j)
    for (int i = j; i >= 0; i = h_parent[i]) anc[(size_t)j * 4 + (i >> 6)] |= 1ull << (i & 63);

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The copies below read host memory that lives only until this call returns: a stream that is recording
  // would replay them later from memory that is gone, so it is refused.
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess) {
    (void)cudaGetLastError();
    return CASCADE_ERR_CUDA;
  }
  if (capturing != cudaStreamCaptureStatusNone) return CASCADE_ERR_INVALID_ARG;
  unsigned char* base = nullptr;
  CASCADE_TRY(scratch_address(&base));
  // The array still holds the previous call's descriptor and scores: everything read below is rewritten
  // here, and the counters (which the kernel expects at zero) are cleared.
  CASCADE_CUDA_TRY(cudaMemcpyAsync(base + Layout::off_ints, ints.data(), Layout::kInts * 4, cudaMemcpyHostToDevice, s));
  CASCADE_CUDA_TRY(cudaMemcpyAsync(base + Layout::off_anc, anc.data(), anc.size() * 8, cudaMemcpyHostToDevice, s));
  CASCADE_CUDA_TRY(cudaMemsetAsync(base + Layout::off_counters, 0, (size_t)kMaxB * 4, s));

  // Stand-ins for the context and tree objects, pointing into the static array (nothing is allocated).
  cascade_ctx ctx;
  ctx.shape = {};
  ctx.shape.B = B;
  ctx.tail_counters = reinterpret_cast<unsigned int*>(base + Layout::off_counters);
  cascade_tree tree;
  tree.ctx = &ctx;
  tree.T = T;
  tree.depth_max = depth_max;
  tree.n_pairs = n_pairs;
  int32_t* d_ints = reinterpret_cast<int32_t*>(base + Layout::off_ints);
  tree.d_parent = d_ints;
  tree.d_depth = d_ints + kMaxT;
  tree.d_child_begin = d_ints + 2 * kMaxT;
  tree.d_child_count = d_ints + 3 * kMaxT;
  tree.d_sib_base = d_ints + 4 * kMaxT;
  tree.d_pair_a = d_ints + 5 * kMaxT;
  tree.d_pair_b = d_ints + 5 * kMaxT + kMaxPairs;
  tree.d_anc = reinterpret_cast<uint64_t*>(base + Layout::off_anc);

  TailWork w;
  w.kernel_id = K_TAIL;
  w.feat = feat;
  w.feat_dim = feat_dim;
  w.feat_norm = feat_norm;
  w.scores = reinterpret_cast<float*>(base + Layout::off_scores);
  w.row_lse = const_cast<float*>(row_lse);
  w.prm = params;
  w.cand_parent = cand_parent;
  w.cand_gparent = cand_gparent;
  w.tok = tok;
  w.draft_p = draft_p;
  w.uniforms = uniforms;
  w.accept = accept;
  w.q_relaxed = q_relaxed;
  w.tvd_out = tvd_out;
  w.near_count = near_count;
  w.select_mode = select_mode;
  w.path_nodes = path_nodes;
  w.path_len = path_len;
  w.tvd_used = tvd_used;
  return launch_tail(&ctx, &tree, w, s);
}

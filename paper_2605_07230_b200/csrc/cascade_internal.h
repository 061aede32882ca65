// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <vector>

#include "cascade.h"

#define CASCADE_CUDA_TRY(expr)                 \
  do {                                         \
    cudaError_t _e = (expr);                   \
    if (_e != cudaSuccess) {                   \
      cascade_detail::note_cuda_error(_e);     \
      return CASCADE_ERR_CUDA;                 \
    }                                          \
  } while (0)

#define CASCADE_TRY(expr)        \
  do {                           \
    int _s = (expr);             \
    if (_s != CASCADE_OK) return _s; \
  } while (0)

namespace cascade_detail {
void note_cuda_error(cudaError_t e);
inline int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
}  // namespace cascade_detail

// Kernel ids for the per-kernel timing table.
enum KernelId : int {
  K_TREE_ATTN = 0, K_TREE_ATTN_F32, K_FINAL_NORM_MIX, K_GEMM_HEAD, K_HEAD_F32, K_ROW_STATS,
  K_ROW_LSE, K_SIMILARITY, K_ACCEPT, K_TAIL, K_SELECT_PATH, K_EMBED_NORM, K_GEMM_QKV, K_ROPE_SPLIT, K_GEMM_O,
  K_RESID_NORM, K_GEMM_GATE_UP, K_SWIGLU, K_GEMM_DOWN, K_GEMM_F32, K_RESID_ADD, K_KV_APPEND, K_BONUS_TOKEN,
  K_FILTER_LOGITS, K_WAIT_PROBE, K_BUILD_TREE, K_KERNEL_ID_END
};
static_assert(K_KERNEL_ID_END <= CASCADE_KERNEL_COUNT, "timing table too small");

struct TimedLaunch {
  int id;
  cudaEvent_t start, stop;
};

// Bits of the device error word.
enum : int { CASCADE_DEV_ERR_WAIT = 1, CASCADE_DEV_ERR_OVERFLOW = 2, CASCADE_DEV_ERR_BAD_TREE = 4 };

struct cascade_ctx {
  cascade_shape shape;
  int device = 0;
  int sm_count = 148;
  int launches = 0;  // kernels enqueued by the call in progress / last call

  // one device allocation, carved into the regions below
  char* ws = nullptr;
  int64_t ws_bytes = 0;

  int* dev_error = nullptr;  // device error word
  int* host_error = nullptr;  // pinned mirror
  bool timing = false;
  unsigned long long wait_limit_ns = 2000000000ull;  // limit of every bounded device-side wait (cascade_set_wait_limit)
  // cudaFuncSetAttribute is per device and a context is bound to one device: what has been set is kept here
  int gemm_smem_configured[6] = {0, 0, 0, 0, 0, 0};
  bool attn_configured = false, filter_configured = false;
  std::vector<TimedLaunch> timed;        // event pairs recorded since the last read
  std::vector<cudaEvent_t> event_pool;   // spare events
  void* tmap_cache = nullptr; // TMA tensor maps built so far (tmap.cu)
  float* gemm_scratch = nullptr;         // tensor-core GEMM: partial accumulators of tiles split between CTAs
  unsigned int* gemm_flags = nullptr;    // one hand-off flag per CTA (zero between launches)

  // tree attention: a KV split must keep at least this many 128-key tiles (merging splits has a fixed cost)
  int attn_min_tiles_per_split = 3;

  // LM head
  int head_m_pad = 0;             // B*T_max rounded up to 128
  __nv_bfloat16* head_a = nullptr;     // the head's activation operand (B*T x h) in the GEMM's staged layout
  int head_max_tiles = 0;
  float2* head_part = nullptr;    // [head_max_tiles][head_m_pad] (tile max, tile sum of exp)
  float* head_a_f32 = nullptr;    // [B*T_max][h] mixed operand (fp32 path)
  unsigned int* tail_counters = nullptr;  // [B] CTAs-finished counters of the tail kernel (zero between launches)

  // intermediates used when the caller passes NULL
  float* feat = nullptr;        // [B,T,h]
  float* feat_norm = nullptr;   // [B,T]
  float* row_lse = nullptr;     // [B,T]
  float* cand_parent = nullptr;   // [B,T]
  float* cand_gparent = nullptr;  // [B,T]
  float* scores = nullptr;      // [B,max_pairs]
  float* q_relaxed = nullptr;   // [B,T]
  float* tvd_out = nullptr;     // [B,T]
  int max_pairs = 0;

  // decoder layer activations (allocated when ffn > 0)
  float* x = nullptr;            // [R*T][h] residual stream, fp32
  __nv_bfloat16* act = nullptr;  // GEMM operand (R*T x max(h,ffn)) in the GEMM's staged layout (bf16 pair)
  float* act_f32 = nullptr;      // [R*T][max(h,ffn)] GEMM operand (fp32 path)
  float* gemm_out = nullptr;     // [slices][R*T][N] fp32 projection results, one matrix per K slice
  int64_t gemm_out_floats = 0;
  int layer_max_splits = 16;
  void* q_rot = nullptr;         // [R,T,Hq,D] elem
  void* k_rot = nullptr;         // [R,T,Hkv,D] elem
  void* v_rot = nullptr;
  void* attn_out = nullptr;      // fp32 path: [R,T,Hq,D] float; bf16 path: the output projection's operand
                                 // (R*T x Hq*D, bf16 pair) in the GEMM's staged layout

  // staging for the host-buffer entry point
  // host-buffer entry: one block for the step's inputs (tok | draft_p | uniforms) and one for its results
  // (accept | path_nodes | path_len), each moved with a single copy through a pinned host block
  char* st_in = nullptr;
  char* st_out = nullptr;
  char* host_stage = nullptr;   // pinned: inputs, then results
  // host-buffer entry: the step recorded as a CUDA graph once the same call has been seen twice
  struct HostGraph {
    std::vector<unsigned char> key;
    const cascade_tree* tree = nullptr;  // the descriptor the recorded kernels read (dropped with it)
    cudaGraphExec_t exec = nullptr;
    int state = 0;     // 0: key seen once, 1: graph ready, -1: recording failed for this key
    int launches = 0;
    uint64_t last_use = 0;
  };
  std::vector<HostGraph> host_graphs;  // a few entries: callers alternate between a few step structures
  uint64_t host_graph_clock = 0;
  int64_t st_in_bytes = 0, st_out_bytes = 0;
};

struct cascade_tree {
  cascade_ctx* ctx = nullptr;
  int T = 0, depth_max = 0, n_pairs = 0;
  uint64_t uid = 0;      // process-wide unique number of this descriptor's current contents (new at every update)
  std::vector<int32_t> parent, depth, child_begin, child_count, pair_a, pair_b, sib_base;
  // device copies
  char* dev = nullptr;
  int32_t* d_parent = nullptr;
  int32_t* d_depth = nullptr;
  int32_t* d_child_begin = nullptr;  // first child index (children are contiguous)
  int32_t* d_child_count = nullptr;
  int32_t* d_sib_base = nullptr;     // index in the pair list of the first sibling pair among node's children
  int32_t* d_pair_a = nullptr;
  int32_t* d_pair_b = nullptr;
  uint64_t* d_anc = nullptr;         // [T][4] ancestor-or-self bitmask
  int32_t* d_meta = nullptr;         // [4] written by the device-side builder: pair count, depth, valid
  // true after cascade_tree_update_device: the host then knows only T and the caller's bounds -- depth_max is the
  // depth bound, n_pairs the pair bound (the row length of scores arrays) -- and its mirrors of the arrays are stale
  bool device_built = false;
};

// Brackets one kernel launch with events when timing is on; always counts the launch.
struct KernelScope {
  cascade_ctx* ctx;
  cudaStream_t stream;
  cudaEvent_t stop = nullptr;
  KernelScope(cascade_ctx* c, int id, cudaStream_t s) : ctx(c), stream(s) {
    c->launches++;
    if (!c->timing) return;
    cudaEvent_t ev[2];
    for (auto& e : ev) {
      if (!c->event_pool.empty()) {
        e = c->event_pool.back();
        c->event_pool.pop_back();
      } else if (cudaEventCreate(&e) != cudaSuccess) {
        (void)cudaGetLastError();
        return;
      }
    }
    cudaEventRecord(ev[0], s);
    stop = ev[1];
    c->timed.push_back({id, ev[0], ev[1]});
  }
  ~KernelScope() {
    if (stop != nullptr) cudaEventRecord(stop, stream);
  }
};

// ---- kernel launchers (each returns a CASCADE_* status and bumps ctx->launches) -------------------

// accept.cu
// One launch of the tail kernel: any of (cosines, row log-sum-exp from the head's partials, the rule).
struct TailWork {
  int kernel_id = K_TAIL;
  // cosines of the tree's pair list (skipped when feat == nullptr); written to `scores`
  const float* feat = nullptr;
  int feat_dim = 0;
  const float* feat_norm = nullptr;
  float* scores = nullptr;      // [B, n_pairs]: output of the cosines, input of the rule
  // row log-sum-exp from per-tile partials (skipped when part == nullptr); written to `row_lse`
  const float2* part = nullptr;
  int part_ld = 0, n_tiles = 0;
  float* row_lse = nullptr;     // [B, T]: output of the fold, input of the rule
  // the rule (skipped when prm == nullptr) and path selection (skipped when path_nodes == nullptr)
  const cascade_params* prm = nullptr;
  const float* cand_parent = nullptr;
  const float* cand_gparent = nullptr;
  const int32_t* tok = nullptr;
  const float* draft_p = nullptr;
  const float* uniforms = nullptr;
  uint8_t* accept = nullptr;
  float* q_relaxed = nullptr;
  float* tvd_out = nullptr;
  int32_t* near_count = nullptr;
  int select_mode = 0;
  int32_t* path_nodes = nullptr;
  int32_t* path_len = nullptr;
  float* tvd_used = nullptr;
};
int launch_tail(cascade_ctx* ctx, const cascade_tree* tree, const TailWork& w, cudaStream_t s);
int launch_row_stats_from_logits(cascade_ctx* ctx, const cascade_tree* tree, const float* logits,
                                 const int32_t* tok, float* row_lse, float* cand_parent,
                                 float* cand_gparent, cudaStream_t s);
int launch_select_path(cascade_ctx* ctx, const cascade_tree* tree, const uint8_t* accept,
                       const float* tvd_out, int mode, int32_t* path_nodes, int32_t* path_len,
                       float* tvd_used, cudaStream_t s);

// attn_f32.cu / attn_bf16.cu
int launch_tree_attn_f32(cascade_ctx* ctx, const cascade_tree* tree, const float* q, const float* kp,
                         const float* vp, int prefix_cap, const int32_t* prefix_len, const float* kt,
                         const float* vt, float* out, float scale, cudaStream_t s);
int launch_tree_attn_bf16(cascade_ctx* ctx, const cascade_tree* tree, const __nv_bfloat16* q,
                          const __nv_bfloat16* kp, const __nv_bfloat16* vp, int prefix_cap,
                          const int32_t* prefix_len, const __nv_bfloat16* kt, const __nv_bfloat16* vt,
                          __nv_bfloat16* out, bool out_as_operand, float scale, cudaStream_t s);

// head.cu (norm + mix producers, fp32 head) / gemm_tc.cu (tcgen05 GEMM)
// cand_parent / cand_gparent (may be null) are cleared here; the head fills the entries that exist.
// Top-k / nucleus truncation of n_rows rows of V logits in place (filter.cu); counts the launch it makes.
int launch_filter_logits(cascade_ctx* ctx, float* logits, int n_rows, int top_k, float top_p, int32_t* kept_count,
                         cudaStream_t s);

// Output matrices of a sliced projection that still have to be added to the residual stream.
struct PendingAdd {
  const float* slices = nullptr;  // [n][R*T][h]
  int n = 0;
  long long stride = 0;
};
// hidden_f32: the hidden states are fp32 whatever the context's element type (the residual stream); `add`
// (fp32 hidden only) is added to them on the fly.
int launch_final_norm_mix(cascade_ctx* ctx, int T, const void* hidden, bool hidden_f32, const PendingAdd& add,
                          const float* gamma, float eps,
                          float cfg_scale, float inv_temperature, float* feat, float* feat_norm,
                          float* cand_parent, float* cand_gparent, cudaStream_t s);
int launch_head_f32(cascade_ctx* ctx, const cascade_tree* tree, const float* w_head, const int32_t* tok,
                    float* logits, float* row_lse, float* cand_parent, float* cand_gparent, cudaStream_t s);
// bf16 head: logits (optional), per-tile softmax partials into the context, gathered candidate logits.
// The row log-sum-exp is folded from the partials by launch_tail.
int launch_head_bf16(cascade_ctx* ctx, const cascade_tree* tree, const __nv_bfloat16* w_head,
                     const int32_t* tok, float* logits, float* cand_parent, float* cand_gparent, cudaStream_t s);

// tree_build.cu: the descriptor's device arrays from a device-resident parent[]
int launch_build_tree(cascade_ctx* ctx, cascade_tree* tree, int T, int depth_cap, int pairs_cap,
                      const int32_t* parent_dev, cudaStream_t s);

// layer.cu: the decoder layers of a verification step; leaves the residual stream in ctx->x.
// `pending`: the last MLP output, still to be added to ctx->x by whoever reads it next (empty if the
// caller asked for the hidden states, in which case they are complete in ctx->x).
int run_layers(cascade_ctx* ctx, const cascade_tree* tree, const cascade_step* st, PendingAdd* pending, cudaStream_t s);

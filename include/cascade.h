/*
 * cascade.h -- C ABI of the B200 (sm_100a) tree-verification library for CASCADE
 * ("CASCADE: Context-Aware Relaxation for Speculative Image Decoding").
 *
 * One verification step of tree-based speculative image decoding: the target model looks at a draft
 * token tree in one pass (Section 3, "tree decoding"), and the relaxed acceptance rule of Section 4
 * (Eq. 1-3, Algorithm 2) decides which root-to-node path of draft tokens is kept.
 *
 * Conventions
 *   - Every function returns an int status: CASCADE_OK (0) or a negative CASCADE_ERR_* code.  Nothing
 *     throws or aborts.  All arguments are validated on the host before anything is launched, so a bad
 *     argument never reaches the device.
 *   - Pointers are DEVICE pointers unless the parameter is documented "host".  The caller owns every
 *     data buffer; the library owns only what cascade_create / cascade_tree_create return, until the
 *     matching destroy call.
 *   - Work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL = default stream)
 *     and is asynchronous: outputs are valid after the stream has been synchronised.
 *   - A context is bound to the device that was current at cascade_create and holds scratch memory
 *     that its calls share: calls on ONE context must not overlap on the GPU (use one stream, or one
 *     context per stream).
 *   - Tensors are dense, row-major, innermost index last.  "elem" is the context's dtype
 *     (float for CASCADE_F32, bf16 bit patterns for CASCADE_BF16).
 *   - Notation: B prompts; R = 2B rows of the classifier-free-guidance pair, cond rows 0..B-1 then
 *     uncond rows B..2B-1; T tree rows INCLUDING the root row 0 (the pending, last-emitted token whose
 *     key/value is not yet in the cache); P prefix (KV cache) length; h hidden size; Hq/Hkv query/kv
 *     heads; D head size; V image-token vocabulary.
 */
#ifndef CASCADE_H_
#define CASCADE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------------------------------ */
#define CASCADE_OK 0
#define CASCADE_ERR_INVALID_ARG (-1)       /* null pointer, non-positive size, value out of range     */
#define CASCADE_ERR_BAD_TREE (-2)          /* parent[] is not a BFS-ordered tree with grouped siblings (from
                                              cascade_check: found by cascade_tree_update_device)        */
#define CASCADE_ERR_WORKSPACE (-3)         /* device allocation of the context's scratch failed        */
#define CASCADE_ERR_UNSUPPORTED_SHAPE (-4) /* shape outside what the kernels handle (see cascade_shape) */
#define CASCADE_ERR_CUDA (-5)              /* a CUDA runtime / driver call failed                      */
#define CASCADE_ERR_TIMEOUT (-6)           /* a bounded device-side wait gave up (see cascade_check)   */
#define CASCADE_ERR_OVERFLOW (-7)          /* cascade_kv_append: a cache has no room (see cascade_check) */

/* ---- enums ------------------------------------------------------------------------------------- */
#define CASCADE_F32 0
#define CASCADE_BF16 1

/* cascade_params.flags */
#define CASCADE_USE_I 1u          /* Eq. 1: add the mass of interchangeable siblings                     */
#define CASCADE_USE_C 2u          /* Eq. 2: add the mass of convergent children                          */
#define CASCADE_CONV_DIST_SELF 4u /* Eq. 3 read literally: a child's mass is taken under the candidate's
                                     own row; default (flag clear) follows Algorithm 2, which reads it
                                     from the same distribution as the candidate's own probability       */

/* cascade_select_path mode */
#define CASCADE_SELECT_LONGEST 0      /* deepest node whose whole path is accepted, smallest index first */
#define CASCADE_SELECT_FIRST_ACCEPT 1 /* Algorithm 2's walk: first accepted child at every level         */

/* A score this close to its threshold is counted in near_count (decisions there are not stable under
 * rounding). */
#define CASCADE_NEAR 1e-3f

#define CASCADE_MAX_TREE_ROWS 256   /* T  <= 256                                            */
#define CASCADE_MAX_CHILDREN 32     /* children of one node <= 32                           */

typedef struct cascade_ctx cascade_ctx;
typedef struct cascade_tree cascade_tree;

/* Fixed sizes of a context.  Supported: D in {64,128}; Hq a multiple of Hkv; h a multiple of 64;
 * V a multiple of 8; T_max <= CASCADE_MAX_TREE_ROWS; B >= 1.  ffn may be 0 if no decoder layer is
 * run through cascade_verify_step (otherwise a multiple of 8). */
typedef struct {
  int32_t dtype; /* CASCADE_F32 or CASCADE_BF16: element type of q/k/v, hidden states and weights */
  int32_t B;
  int32_t T_max;
  int32_t P_max; /* largest prefix length any call will use                                      */
  int32_t h, Hq, Hkv, D, V;
  int32_t ffn;
} cascade_shape;

/* Relaxation parameters (Section 4.1: tau_pos gates Eq. 1, tau_seq gates Eq. 2; Eq. 3 / Algorithm 2:
 * tvd_budget is the total-variation budget of one verification step, 0.5 in the paper). */
typedef struct {
  float tau_pos;
  float tau_seq;
  float tvd_budget;
  uint32_t flags; /* CASCADE_USE_I | CASCADE_USE_C [| CASCADE_CONV_DIST_SELF] */
} cascade_params;

/* ---- life cycle -------------------------------------------------------------------------------- */

/* Create a context on the current device and allocate its scratch (split-KV partial results,
 * activation staging, softmax partials).  *out is set only on success. */
int cascade_create(cascade_ctx** out, const cascade_shape* shape);
int cascade_destroy(cascade_ctx* ctx);

/* Bytes of device scratch the context holds. */
int64_t cascade_workspace_bytes(const cascade_ctx* ctx);

/* Reads the context's device-side error word (set when a bounded wait inside a kernel ran out) after
 * synchronising `stream`.  Returns CASCADE_OK, CASCADE_ERR_TIMEOUT, CASCADE_ERR_BAD_TREE, CASCADE_ERR_OVERFLOW or
 * CASCADE_ERR_CUDA, and clears the word. */
int cascade_check(cascade_ctx* ctx, void* stream);

/* Number of kernels the most recent call on this context enqueued. */
int cascade_last_launch_count(const cascade_ctx* ctx);

/* Failure detection.  Every wait inside a kernel (on an mbarrier, on another CTA's flag) gives up after a
 * limit, records it in the context's error word and leaves through the kernel's normal teardown, so a wait
 * that can never end costs the limit, not the device; cascade_check then returns CASCADE_ERR_TIMEOUT and the
 * context stays usable.  cascade_set_wait_limit changes the limit for later calls on this context
 * (nanoseconds, >= 1000; default 2 s).
 * cascade_wait_probe is a self-test of that path: it enqueues one small kernel whose only CTA waits on a
 * barrier nothing will ever arrive on (no copy in flight), with the context's limit.  waited_ns (DEVICE
 * uint32, may be NULL) receives how long the wait lasted.  After the stream has been synchronised,
 * cascade_check reports CASCADE_ERR_TIMEOUT. */
int cascade_set_wait_limit(cascade_ctx* ctx, int64_t limit_ns);
int cascade_wait_probe(cascade_ctx* ctx, uint32_t* waited_ns, void* stream);

const char* cascade_strerror(int status);

/* Per-kernel device timing (measurement aid, off by default).  While enabled, every kernel a call on
 * this context enqueues is bracketed by a pair of CUDA events on the caller's stream.
 * cascade_timing_read synchronises those events, ADDS the elapsed milliseconds and launch counts per
 * kernel id into ms_total / launches (HOST arrays of CASCADE_KERNEL_COUNT entries, caller-zeroed) and
 * forgets the recorded events.  cascade_kernel_name(id) names an id (NULL if out of range). */
#define CASCADE_KERNEL_COUNT 32
int cascade_timing_enable(cascade_ctx* ctx, int32_t on);
int cascade_timing_read(cascade_ctx* ctx, float* ms_total, int32_t* launches);
const char* cascade_kernel_name(int32_t id);

/* The draft tree (the static tree mask of Section 3; Algorithm 2 input `tree`).
 * parent: HOST array of T entries, parent[0] = -1, 0 <= parent[j] < j, rows in BFS order (depth never
 * decreases with the index) and the children of one parent contiguous.  Builds the device-side
 * descriptor: depth, packed ancestor-or-self bitmask (T x 4 uint64 words), child ranges, and the list
 * of (node, node) pairs whose cosine the acceptance rule reads (every parent->child edge, then every
 * unordered sibling pair).  Returns CASCADE_ERR_BAD_TREE if the ordering rules do not hold. */
int cascade_tree_create(cascade_ctx* ctx, int32_t T, const int32_t* parent, cascade_tree** out);
int cascade_tree_destroy(cascade_tree* tree);

/* A new draft tree in an existing descriptor (drafters that grow a different tree every step): same rules
 * and errors as cascade_tree_create, T <= the context's T_max.  Nothing is allocated; the descriptor is
 * rebuilt on the host and copied to the device on `stream` (the source is pageable host memory, so the copy
 * is staged before the call returns), and calls that use the tree must be enqueued after it on that stream.
 * An invalid tree returns its error and leaves the descriptor as it was.  Host-side queries
 * (cascade_tree_rows / depth / num_pairs / pairs) answer for the new tree as soon as the call returns. */
int cascade_tree_update(cascade_tree* tree, int32_t T, const int32_t* parent, void* stream);
/* The same, from a parent[] that is already in DEVICE memory, without a host round trip (drafters that decide
 * the tree's shape on the device each step: the dynamic trees that Section 2 contrasts with the static mask).
 * One small kernel on `stream` checks the rules of cascade_tree_create and writes the descriptor.  The host
 * cannot see the tree, so the caller states bounds that sizes depend on:
 *   T          rows (host value; grids and row counts of every later call come from it), <= T_max;
 *   depth_cap  the tree is at most this deep; path_nodes arrays of later calls have depth_cap + 1 entries per
 *              prompt and cascade_tree_depth returns it;
 *   pairs_cap  at most this many (node, node) pairs (edges + sibling pairs); scores arrays of later calls have
 *              pairs_cap entries per prompt and cascade_tree_num_pairs returns it; <= 0: the context's maximum.
 * A parent[] that breaks a rule or a bound is found on the device: cascade_check then returns
 * CASCADE_ERR_BAD_TREE, and the descriptor is left holding a neutral tree of T rows (every row a childless leaf
 * below the root, no pairs), so that calls already enqueued behind it stay within their buffers; their results
 * are meaningless.  Nothing is allocated; the host-side mirrors are not refreshed (cascade_tree_pairs and
 * cascade_tree_download fetch from the device with blocking copies). */
int cascade_tree_update_device(cascade_tree* tree, int32_t T, int32_t depth_cap, int32_t pairs_cap,
                               const int32_t* parent_dev, void* stream);
/* Copies the descriptor's device arrays to HOST arrays (blocking copies; synchronise the stream of a pending
 * update first): parent, depth, child_begin, child_count [T] int32 and the packed ancestor-or-self mask
 * anc [T][4] uint64 (bit i of row j set iff i is j or an ancestor of j).  Any pointer may be NULL. */
int cascade_tree_download(const cascade_tree* tree, int32_t* parent, int32_t* depth, int32_t* child_begin,
                          int32_t* child_count, uint64_t* anc);
int32_t cascade_tree_rows(const cascade_tree* tree);      /* T                                     */
int32_t cascade_tree_depth(const cascade_tree* tree);     /* deepest level                         */
int32_t cascade_tree_num_pairs(const cascade_tree* tree); /* edges + sibling pairs                 */
/* Copies the pair list to HOST arrays of cascade_tree_num_pairs entries (for inspecting scores). */
int cascade_tree_pairs(const cascade_tree* tree, int32_t* pair_a, int32_t* pair_b);

/* ---- (a) tree-masked attention ----------------------------------------------------------------- */
/* Section 3: all draft-tree rows are verified by the target "via a parallel forward pass".  For every
 * row r of the CFG pair, head and tree row j:
 *     out[r,j,head,:] = sum_i softmax_i(softmax_scale * <q[r,j,head,:], k_i>) v_i
 * over the keys row j may see: cache entries 0..prefix_len[r]-1 and the tree rows that are j itself or
 * one of its ancestors.  Query head `head` reads kv head head / (Hq / Hkv).
 *   q        [R,T,Hq,D] elem          k_tree, v_tree [R,T,Hkv,D] elem
 *   k_prefix, v_prefix [R,prefix_cap,Hkv,D] elem; rows at or beyond prefix_len[r] are never used
 *   prefix_len [R] int32, device; 0 <= prefix_len[r] <= min(prefix_cap, P_max)
 *   out      [R,T,Hq,D] elem
 * Softmax and accumulation are fp32.  Base addresses must be 16-byte aligned. */
int cascade_tree_attn(cascade_ctx* ctx, const cascade_tree* tree, const void* q, const void* k_prefix,
                      const void* v_prefix, int32_t prefix_cap, const int32_t* prefix_len,
                      const void* k_tree, const void* v_tree, void* out, float softmax_scale,
                      void* stream);

/* ---- (b) final norm + LM head + classifier-free guidance + vocabulary softmax statistics ------- */
/* Section 4.2 names the final projection, O(hV), as the dominant cost of verification; the guidance
 * scale is the experimental setting of App. D.2 (3.0, or 5.0 for Janus-Pro).  For prompt b, tree row j:
 *     n_x      = hidden_x * rsqrt(mean(hidden_x^2) + eps) * rms_gamma         x in {cond, uncond}
 *     logits   = (W n_u + cfg_scale * (W n_c - W n_u)) / temperature
 *     feat     = n_c                 (the target hidden state F of Section 4.1 that feeds the head)
 *     row_lse  = log sum_v exp(logits[v])
 *     cand_parent[b,j]  = logits[b, parent[j], tok[b,j]]              (0 for the root)
 *     cand_gparent[b,j] = logits[b, parent[parent[j]], tok[b,j]]      (0 where there is none)
 *   hidden [R,T,h] elem; rms_gamma [h] float; w_head [V,h] elem; tok [B,T] int32 in [0,V)
 *   logits_out [B,T,V] float or NULL; feat_out [B,T,h] float; feat_norm_out [B,T] float (||feat||_2);
 *   row_lse_out [B,T] float; cand_parent_out, cand_gparent_out [B,T] float (both NULL if tok is NULL).
 * The guidance mix is applied to the normalised hidden states before the product (the head is
 * linear), and that operand is carried as a bf16 high part plus a bf16 remainder so the result keeps
 * fp32-level accuracy.  temperature > 0. */
int cascade_lm_head_cfg(cascade_ctx* ctx, const cascade_tree* tree, const void* hidden,
                        const float* rms_gamma, float eps, const void* w_head, float cfg_scale,
                        float temperature, const int32_t* tok, float* logits_out, float* feat_out,
                        float* feat_norm_out, float* row_lse_out, float* cand_parent_out,
                        float* cand_gparent_out, void* stream);

/* ---- (c) relaxed acceptance -------------------------------------------------------------------- */
/* Cosines of Section 4.1 for the tree's pair list: scores_out[b,i] = cos(feat[b,pair_a[i]],
 * feat[b,pair_b[i]]).  feat [B,T,feat_dim] float; feat_norm [B,T] float or NULL (then computed here).
 * Passing logits as feat (feat_dim = V) gives the logit-space variant of App. B. */
int cascade_similarity(cascade_ctx* ctx, const cascade_tree* tree, const float* feat, int32_t feat_dim,
                       const float* feat_norm, float* scores_out, void* stream);

/* Eq. 1-3 and Algorithm 2 for every draft node at once.  For node j >= 1 with parent pi,
 * g = softmax(logits[b,pi,:]):
 *     q_j  = g[tok_j]
 *     I_j  = siblings s of j with cos(F_j,F_s) >= tau_pos ; C_j = children c of j with cos >= tau_seq
 *     mI_j = mass under g of the distinct tokens of I_j other than tok_j
 *     mC_j = mass (under g, or under softmax(logits[b,j,:]) with CASCADE_CONV_DIST_SELF) of the distinct
 *            tokens of C_j not equal to tok_j and not already in mI_j
 *     running total t: the first child of pi starts from tvd_out[pi], a later sibling from the previous
 *     sibling's tvd_out (what Algorithm 2's curr_TVD holds when its walk arrives at j);
 *     each set is added whole, I first, only if non-empty and t + mass <= tvd_budget;
 *     accept[j] = uniforms[j] < min(1, q_relaxed[j] / draft_p[j]);  draft_p <= 0 rejects; accept[0] = 1.
 * Inputs: scores [B,num_pairs] float from cascade_similarity; row_lse, cand_parent, cand_gparent [B,T]
 * float as produced by cascade_lm_head_cfg -- or pass logits [B,T,V] float (then those three may be
 * NULL and are derived from logits); tok [B,T] int32; draft_p [B,T] float (the drafter's probability of
 * tok[j] under its parent's context: Algorithm 2 input D); uniforms [B,T] float in [0,1) (Algorithm 2's
 * random(), made an input so results are reproducible).
 * Outputs: accept [B,T] uint8; q_relaxed, tvd_out [B,T] float; near_count [B] int32 = number of nodes
 * with a cosine, a budget comparison or the accept test within CASCADE_NEAR of its threshold (any of
 * the last three may be NULL). */
int cascade_relaxed_accept(cascade_ctx* ctx, const cascade_tree* tree, const float* scores,
                           const float* logits, const float* row_lse, const float* cand_parent,
                           const float* cand_gparent, const int32_t* tok, const float* draft_p,
                           const float* uniforms, const cascade_params* params, uint8_t* accept,
                           float* q_relaxed, float* tvd_out, int32_t* near_count, void* stream);

/* ---- (d) path selection ------------------------------------------------------------------------ */
/* Algorithm 2 keeps, level by level, the first accepted candidate (CASCADE_SELECT_FIRST_ACCEPT);
 * CASCADE_SELECT_LONGEST returns the deepest node all of whose ancestors are accepted.
 *   accept [B,T] uint8; tvd_out [B,T] float or NULL
 *   path_nodes [B, depth+1] int32: root..end node, unused entries -1  (depth = cascade_tree_depth)
 *   path_len [B] int32: number of accepted draft tokens (alpha of Algorithm 2)
 *   tvd_used [B] float or NULL: the running total where the walk stops (needs tvd_out). */
int cascade_select_path(cascade_ctx* ctx, const cascade_tree* tree, const uint8_t* accept,
                        const float* tvd_out, int32_t mode, int32_t* path_nodes, int32_t* path_len,
                        float* tvd_used, void* stream);

/* ---- the whole step ---------------------------------------------------------------------------- */

/* One pre-norm decoder layer (the workload's architecture; the paper treats the target as given):
 * a = RMSNorm(x, gamma_attn); q,k,v = a Wq^T, a Wk^T, a Wv^T; rotary (half-split pairing) at position
 * prefix_len[r] + depth[j]; tree attention; x += attn Wo^T; m = RMSNorm(x, gamma_mlp);
 * x += (silu(m Wg^T) * (m Wu^T)) Wd^T.  Matrices are [out_features, in_features] elem.  wq, wk, wv must be
 * stacked in memory in this order (wk = wq + Hq*D*h elements, wv = wk + Hkv*D*h), and so must w_gate, w_up
 * (w_up = w_gate + ffn*h): each group runs as one projection; CASCADE_ERR_UNSUPPORTED_SHAPE otherwise.
 * The bf16 path needs D = 128. */
typedef struct {
  const float* gamma_attn; /* [h] */
  const void* wq;          /* [Hq*D, h]  */
  const void* wk;          /* [Hkv*D, h] */
  const void* wv;          /* [Hkv*D, h] */
  const void* wo;          /* [h, Hq*D]  */
  const float* gamma_mlp;  /* [h] */
  const void* w_gate;      /* [ffn, h] */
  const void* w_up;        /* [ffn, h] */
  const void* w_down;      /* [h, ffn] */
  void* k_prefix;          /* [R, prefix_cap, Hkv, D] this layer's cache: read by cascade_verify_step, */
  void* v_prefix;          /* written (rows at and beyond prefix_len) by cascade_kv_append              */
} cascade_layer;

/* All arguments of one verification step.  Pointers are device pointers except `layers`, a HOST
 * array of n_layers structs (whose members are device pointers). */
typedef struct {
  /* model */
  int32_t n_layers;            /* >= 0.  0: skip the decoder layers, `hidden_in` is the head's input */
  const cascade_layer* layers; /* host array */
  const void* embed;           /* [V,h] elem, token embedding (n_layers > 0)                         */
  const float* gamma_final;    /* [h]                                                                */
  const void* w_head;          /* [V,h] elem                                                         */
  int32_t prefix_cap;
  const int32_t* prefix_len;   /* [R]                                                                */
  float eps, rope_base, softmax_scale, cfg_scale, temperature;
  /* step inputs */
  const int32_t* tok;          /* [B,T] */
  const float* draft_p;        /* [B,T] */
  const float* uniforms;       /* [B,T] */
  const void* hidden_in;       /* [R,T,h] elem, used when n_layers == 0                              */
  /* stand-alone attention inputs, used when n_layers == 0 and q != NULL: piece (a) runs on them in
   * the same enqueue and writes attn_out */
  const void* q;               /* [R,T,Hq,D]  */
  const void* k_tree;          /* [R,T,Hkv,D] */
  const void* v_tree;
  const void* k_prefix;        /* [R,prefix_cap,Hkv,D] */
  const void* v_prefix;
  void* attn_out;              /* [R,T,Hq,D] elem */
  /* rule */
  cascade_params params;
  int32_t select_mode;
  /* outputs */
  uint8_t* accept;             /* [B,T] */
  int32_t* path_nodes;         /* [B,depth+1] */
  int32_t* path_len;           /* [B] */
  float* q_relaxed;            /* [B,T] or NULL */
  float* tvd_out;              /* [B,T] or NULL */
  float* tvd_used;             /* [B] or NULL */
  int32_t* near_count;         /* [B] or NULL */
  /* optional intermediates, NULL to skip the store */
  float* logits;               /* [B,T,V] */
  float* feat;                 /* [B,T,h] */
  float* scores;               /* [B,num_pairs] */
  float* row_lse;              /* [B,T] */
  float* hidden_out;           /* [R,T,h] float: residual stream entering the final norm (n_layers>0) */
  void* k_tree_out;            /* [n_layers,R,T,Hkv,D] elem: rotated keys / values of the tree rows, */
  void* v_tree_out;            /*   what a caller appends to the cache for the accepted path          */
  /* truncation of the target distribution before the rule (see cascade_filter_logits; Appendix D.1):
   * top_k > 0 and/or 0 < top_p < 1 switch it on, which needs `logits` (they are truncated in place and the
   * row statistics are taken from them); zero in both fields (a zeroed struct): off */
  int32_t top_k;
  float top_p;
} cascade_step;

/* Runs pieces (a)-(d) (and the decoder layers, if any) as one enqueue on `stream`. */
int cascade_verify_step(cascade_ctx* ctx, const cascade_tree* tree, const cascade_step* step, void* stream);

/* Same step with the per-step inputs and results in HOST memory (pageable or pinned): tok, draft_p, uniforms
 * [B,T] are gathered into the context's pinned block and copied to the device in one transfer, accept [B,T],
 * path_nodes [B,depth+1] and path_len [B] come back in one transfer, and the call returns after the stream
 * has been synchronised, the results in the caller's arrays.  The corresponding pointers inside `step` are
 * ignored (the context's own staging buffers are used); everything else in `step` is read as in
 * cascade_verify_step.  Like all calls on one context, these must not overlap.  When the same call (same
 * step contents, tree and stream) is repeated on a stream that can be recorded (not the legacy default
 * stream), the library records its copies and launches as a CUDA graph at the second call and replays it
 * afterwards; results are the same either way. */
int cascade_verify_step_host(cascade_ctx* ctx, const cascade_tree* tree, const cascade_step* step,
                             const int32_t* tok_host, const float* draft_p_host, const float* uniforms_host,
                             uint8_t* accept_host, int32_t* path_nodes_host, int32_t* path_len_host,
                             void* stream);

/* ---- between two steps of a decode loop --------------------------------------------------------- */
/* The token after the accepted path: Algorithm 1's last step, which Algorithm 2 leaves out.  For prompt b,
 * end = last node of its path, q = softmax(logits[b, end, :]).  Two rules:
 *   draft_row != NULL (the drafter's full distribution p at the end node, [B,V] float, row b for prompt b):
 *     Algorithm 1's correction step -- if a child of end was rejected, the token is drawn from [q - p]+
 *     normalised; after a fully accepted draft (end has no children), from q.  Should nothing of q lie above p
 *     (p = q), q is used.  mass_out[b] = sum of [q - p]+ (1 where q was used).
 *   draft_row == NULL (a tree drafter that keeps only the probabilities of its proposals): the tokens of end's
 *     children (all rejected, whichever selection mode chose the path) get probability zero, the rest of q is
 *     renormalised.  mass_out[b] = the probability mass that remains.
 * token_out[b] is the inverse-CDF sample at u_bonus[b]: the first v whose cumulative weight exceeds
 * u_bonus[b] * (total weight).
 *   logits [B,T,V] float (as stored by cascade_lm_head_cfg / cascade_verify_step); tok [B,T] int32;
 *   path_nodes [B,depth+1], path_len [B] from cascade_select_path; u_bonus [B] float in [0,1);
 *   token_out [B] int32; mass_out [B] float or NULL. */
int cascade_bonus_token(cascade_ctx* ctx, const cascade_tree* tree, const float* logits, const int32_t* tok,
                        const float* draft_row, const int32_t* path_nodes, const int32_t* path_len,
                        const float* u_bonus, int32_t* token_out, float* mass_out, void* stream);

/* Appends the keys / values of the accepted path's tree rows (root row first: the pending token, then the
 * accepted drafts) to the caches of n_layers layers, for both CFG rows of every prompt, at positions
 * prefix_len[r] .. prefix_len[r] + path_len[b], and adds path_len[b] + 1 to prefix_len[r] (device array,
 * updated in place).  The tree rows were rotated at exactly these positions by cascade_verify_step.
 *   layers: HOST array of n_layers structs; only k_prefix / v_prefix are used, and those caches
 *           ([R, prefix_cap, Hkv, D] elem) are written here.
 *   k_tree, v_tree [n_layers,R,T,Hkv,D] elem: cascade_step.k_tree_out / v_tree_out of the step.
 * A path that does not fit into prefix_cap is not appended and raises CASCADE_ERR_OVERFLOW at the next
 * cascade_check.  n_layers <= 64. */
int cascade_kv_append(cascade_ctx* ctx, const cascade_tree* tree, int32_t n_layers, const cascade_layer* layers,
                      const void* k_tree, const void* v_tree, const int32_t* path_nodes, const int32_t* path_len,
                      int32_t prefix_cap, int32_t* prefix_len, void* stream);

/* ---- truncation of the target distribution ------------------------------------------------------- */
/* Top-k / nucleus truncation of target logits, in place (the sampling settings of the paper's experiments,
 * Appendix D.1: temperature 1, top-p 1.0, top-k 2000; the paper states the numbers, the truncations are
 * the usual ones).  Per row of V logits:
 *   top_k (0 < top_k < V; 0 or >= V: off): keep the tokens whose logit is >= the top_k-th largest logit of the
 *     row -- tokens tied with it stay together, so more than top_k can remain;
 *   top_p (< 1; 1: off), on the distribution renormalised over what top-k kept: keep a token iff the
 *     probability of the tokens with a strictly larger logit is < top_p (ties stay together).
 * A dropped token's logit becomes -inf: cascade_relaxed_accept (with these logits), cascade_bonus_token and
 * any softmax over the row then give it probability zero and renormalise the rest.
 *   logits [n_rows, V] float, DEVICE, read and written (V from the context's shape; rows are independent,
 *          e.g. the [B,T,V] logits of cascade_lm_head_cfg with n_rows = B*T);
 *   kept_count [n_rows] int32 DEVICE or NULL: how many tokens of each row remain.
 * Both thresholds are exact (a radix descent over the logits' bit patterns; the nucleus sums probabilities
 * in 40-bit fixed point, so the result does not depend on the order of the additions).
 * Errors: CASCADE_ERR_INVALID_ARG (null pointers, n_rows < 1, top_k < 0, top_p outside (0, 1]). */
int cascade_filter_logits(cascade_ctx* ctx, float* logits, int32_t n_rows, int32_t top_k, float top_p,
                          int32_t* kept_count, void* stream);

/* ---- the drafter's training loss (outside the verification step) ---------------------------------- */
/* Section 4.3, Eq. 4: the soft cross-entropy between the target distribution and the drafter's at every position k
 * of a target-generated sequence, weighted by c (2 in the paper's experiments, Appendix D.1) where the target's
 * hidden states of positions k and k+1 satisfy the convergence criterion of Eq. 2 (cosine >= tau_seq), by 1 elsewhere
 * and at the last position:
 *     loss_out[k] = - w_k * sum_v softmax(target_logits[k])[v] * log softmax(draft_logits[k])[v]
 *   target_logits, draft_logits [K,V] float; feat [K,h] float (target hidden states); DEVICE pointers.
 *   loss_out [K] float; weight_out [K] float or NULL (w_k); total_out [1] float or NULL (sum of loss_out, added in
 *   index order).  No context is needed and nothing is allocated; two kernels on `stream`.
 * Only the forward value is computed (the gradient with respect to draft_logits[k] is w_k (p_k - q_k), which a
 * training framework forms from its own softmax).  Errors: CASCADE_ERR_INVALID_ARG (null pointers, sizes < 1,
 * c <= 0, NaN threshold). */
int cascade_drafter_loss(const float* target_logits, const float* draft_logits, const float* feat, int32_t K, int32_t V,
                         int32_t h, float tau_seq, float c, float* loss_out, float* weight_out, float* total_out,
                         void* stream);

/* ---- acceptance without any device allocation --------------------------------------------------- */
/* The paper has no counterpart to this entry point; it exists for deployment.  Some callers of this
 * library may not allocate device memory at all: a plug-in running inside a serving process that
 * handed its whole memory budget to one arena at start-up, code that runs after the host has frozen
 * allocation (for instance to keep addresses stable), or a process whose allocator hooks forbid
 * cudaMalloc.  cascade_create and cascade_tree_create call cudaMalloc, so such callers cannot use the
 * entry points above.  This one needs neither object: similarity scores (Section 4.1), relaxed acceptance
 * (Eq. 1-3, Algorithm 2) and path selection, as cascade_similarity + cascade_relaxed_accept +
 * cascade_select_path compute them, with all device-side scratch (the tree descriptor, the cosine
 * scores, the per-prompt finished-CTA counters) in one static device array of the library
 * (about 0.7 MB, held by every GPU that loads the library until the process exits).
 *   B <= CASCADE_STATIC_MAX_PROMPTS, T <= CASCADE_MAX_TREE_ROWS; larger sizes return
 *   CASCADE_ERR_UNSUPPORTED_SHAPE and nothing is launched.
 *   parent [T]: HOST array, same rules as cascade_tree_create.  Everything else: device pointers with the
 *   meaning they have in cascade_similarity / cascade_relaxed_accept / cascade_select_path
 *   (feat [B,T,feat_dim] float, 16-byte aligned; feat_norm [B,T] or NULL; row_lse, cand_parent,
 *   cand_gparent [B,T]; tok, draft_p, uniforms [B,T]; outputs accept [B,T], path_nodes [B,depth+1],
 *   path_len [B]; q_relaxed, tvd_out, near_count, tvd_used may be NULL).
 * The call allocates nothing on the device: it copies the tree descriptor into the static array (from
 * temporary host memory that is gone when the call returns), clears the counters and enqueues one kernel on
 * `stream`.  A stream that is being captured is refused (CASCADE_ERR_INVALID_ARG, nothing is enqueued): the
 * copies read host memory of this call only.  The first call on a device also looks up the device address of
 * the array (cudaGetSymbolAddress).
 * All calls on a device share the one array and it keeps the last call's contents: two calls whose
 * work overlaps on the GPU (different streams) race; serialise them. */
#define CASCADE_STATIC_MAX_PROMPTS 32
int cascade_accept_static(int32_t B, int32_t T, const int32_t* parent, const float* feat, int32_t feat_dim,
                          const float* feat_norm, const float* row_lse, const float* cand_parent,
                          const float* cand_gparent, const int32_t* tok, const float* draft_p,
                          const float* uniforms, const cascade_params* params, int32_t select_mode,
                          uint8_t* accept, float* q_relaxed, float* tvd_out, int32_t* near_count,
                          int32_t* path_nodes, int32_t* path_len, float* tvd_used, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CASCADE_H_ */

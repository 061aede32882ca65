#pragma once
#include "cascade_internal.h"

// What the tensor-core GEMM does with a finished tile (all members optional).
struct GemmEpilogue {
  float* C = nullptr;      // [M][ldc] fp32 result
  int ldc = 0;
  int accumulate = 0;      // 1: C += result (residual add), 0: C = result
  // splits = 0: the kernel balances (tile, K block) work over the SMs and adds the pieces of a tile
  // itself.  splits = S >= 1: K is cut into S slices and slice s writes its own matrix
  // C + s * slice_stride; the consumer adds the S matrices (no waiting inside the kernel; S > 1 needs C,
  // no accumulate, no part).
  int splits = 0;
  int64_t slice_stride = 0;
  // balanced = 1 (with splits = the value gemm_tc_balanced_map returned): the flattened (tile, K block) list is
  // cut into one equally long range per CTA as in the splits = 0 mode, but every piece of a tile goes to an output
  // matrix of its own (the piece's number within the tile) instead of being handed to the tile's owner; tiles
  // have different numbers of pieces, which the consumer takes from the SliceMap.
  int balanced = 0;
  float2* part = nullptr;  // per-(row, 128-wide tile) softmax partials (max, sum of exp): part[m * part_ld + tile]
  int part_ld = 0;
  // gather of the logits the acceptance rule reads (needs part): for idx = b * T + j,
  // cand_parent[idx] = C[b * T + parent[j]][tok[idx]], cand_gparent[idx] likewise for the grandparent
  const int32_t* tok = nullptr;
  const int32_t* parent = nullptr;
  int T = 0, n_rows = 0;
  float* cand_parent = nullptr;
  float* cand_gparent = nullptr;
};

// C[m][n] = sum_k (a_hi[m][k] + a_lo[m][k]) * W[n][k] on the tensor cores (see gemm_tc.cu).
// W [N][K] bf16 row-major; A: the M x K activation operand (bf16 high part + bf16 remainder) in the staged
// layout of operand.cuh; K a multiple of 64.  Uses the context's split-tile scratch: calls on one context
// must not overlap.
int launch_gemm_tc(cascade_ctx* ctx, const __nv_bfloat16* W, int N, int K, const __nv_bfloat16* A, int M,
                   const GemmEpilogue& epi, int kernel_id, cudaStream_t s);
// How a balanced launch spread its tiles' pieces over the output matrices: the columns [t * tile_cols,
// (t + 1) * tile_cols) of the result have slice_count(map, t) valid matrices (0, 1, ...).
struct SliceMap {
  int balanced = 0;   // 0: every column has `n_slices` matrices
  int n_slices = 0;   // matrices to add (balanced: the most pieces any tile has)
  int q = 0, r = 0, n_kb = 0, tile_cols = 1;
};
#ifdef __CUDACC__
// CTA whose range holds unit u (ranges: CTA c starts at c * q + min(c, r))
__device__ __forceinline__ int slice_map_cta(const SliceMap& m, int u) {
  const int big = m.r * (m.q + 1);
  return u < big ? u / (m.q + 1) : m.r + (u - big) / m.q;
}
__device__ __forceinline__ int slice_count(const SliceMap& m, int col) {
  if (!m.balanced) return m.n_slices;
  const int t = col / m.tile_cols;
  return slice_map_cta(m, (t + 1) * m.n_kb - 1) - slice_map_cta(m, t * m.n_kb) + 1;
}
#endif
// The map of the launch launch_gemm_tc(ctx, W, N, K, ., M, epi with balanced = 1, ...) would make (one row chunk
// only: M <= 128); map.n_slices is the value to pass as epi.splits.  map.balanced = 0 if the mode does not apply.
SliceMap gemm_tc_balanced_map(const cascade_ctx* ctx, int M, int N, int K);
// Floats of scratch the split-tile hand-off needs for a device with `sm_count` SMs.
int64_t gemm_tc_scratch_floats(int sm_count);
// Number of K slices (splits >= 1) that keeps the SMs evenly busy for an [N][K] weight matrix.
int gemm_tc_pick_splits(int sm_count, int M, int N, int K, int max_splits);

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
// Floats of scratch the split-tile hand-off needs for a device with `sm_count` SMs.
int64_t gemm_tc_scratch_floats(int sm_count);
// Number of K slices (splits >= 1) that keeps the SMs evenly busy for an [N][K] weight matrix.
int gemm_tc_pick_splits(int sm_count, int M, int N, int K, int max_splits);

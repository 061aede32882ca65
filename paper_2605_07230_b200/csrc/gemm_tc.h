#pragma once
#include "cascade_internal.h"

// C[m][n] = sum_k (a_hi[m][k] + a_lo[m][k]) * W[n][k] on the tensor cores (see gemm_tc.cu).
// W [N][K] bf16, a_hi/a_lo [M][K] bf16, K a multiple of 64.  C (fp32, row stride ldc) may be null.
// With part != null the kernel also writes per-(row, 128-wide tile) softmax partials to
// part[m * part_ld + tile] and row-wise log-sum-exp over n to lse[m].
int launch_gemm_tc(cascade_ctx* ctx, const __nv_bfloat16* W, int N, int K, const __nv_bfloat16* a_hi,
                   const __nv_bfloat16* a_lo, int M, float* C, int ldc, float2* part, int part_ld, float* lse,
                   int kernel_id, cudaStream_t s);

// Weight-streaming skinny GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
//     C[m][n] = sum_k (Ahi[m][k] + Alo[m][k]) * W[n][k]        m < M (few rows), n < N (many rows)
//
// This is the LM head (W = [V,h], the O(hV) projection that Section 4.2 of the paper names as the
// dominant cost of verification) and every other projection of the decoder layer.  With M of the
// order of the draft-tree size the product is bound by streaming W from HBM once, so the kernel is
// organised around that stream:
//   * the WEIGHT rows sit on the UMMA M dimension (128 per tile) and the activation rows on the UMMA
//     N dimension (NB = M rounded up to 16, <= 256), so no tensor-core work is spent on padding a
//     small M up to 128;
//   * persistent CTAs (one per SM) walk the weight tiles; a TMA producer warp keeps a ring of
//     [W 128x64 | Ahi NBx64 | Alo NBx64] bf16 stages (128-byte swizzle) in flight, a single thread
//     issues the UMMAs (two per 16-wide K step: the high part and the remainder of the activation
//     operand accumulate into the same fp32 TMEM accumulator), and four epilogue warps drain one of
//     two TMEM accumulators while the next tile is being accumulated into the other;
//   * epilogue: TMEM lane = weight row n, column = activation row m.  Optional store of C (coalesced
//     over n), and optional per-(m, tile) softmax partials (max, sum of exp) which the last CTA to
//     finish folds into row-wise log-sum-exp -- the vocabulary softmax statistic the acceptance rule
//     needs (Algorithm 2, gtp = softmax(logits)) without re-reading the logits.
// Every mbarrier wait is bounded; on expiry the CTA records an error word and leaves through the
// normal teardown (TMEM is freed).
#include "cascade_internal.h"
#include "gemm_tc.h"
#include "ptx.cuh"
#include "tmap.h"

namespace {

constexpr int kThreads = 192;       // warp 0: TMA, warp 1: UMMA issue + TMEM alloc, warps 2-5: epilogue
constexpr int kTileN = 128;         // weight rows per tile (UMMA M)
constexpr int kBK = 64;             // K elements per stage (one 128-byte swizzle span)
constexpr int kMaxStages = 8;
constexpr int kStRow = 136;         // staging row stride (floats): 136 = 8 mod 32 keeps reads conflict-free
constexpr int kWBytes = kTileN * kBK * 2;

struct GemmArgs {
  int M, N, K, NB, n_ntiles, n_mchunks, stages, tmem_cols;
  float* C;
  int ldc;
  float2* part;
  int part_ld;
  float* lse;
  unsigned int* counter;
  int* err;
};

__device__ __forceinline__ void combine_ms(float& m, float& s, float mo, float so) {
  const float nm = fmaxf(m, mo);
  if (nm == -INFINITY) {
    s = 0.f;
    return;
  }
  s = s * __expf(m - nm) + so * __expf(mo - nm);
  m = nm;
}

__global__ void __launch_bounds__(kThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_hi,
          const __grid_constant__ CUtensorMap tm_lo, const GemmArgs p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tmem_full[2], tmem_empty[2];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort, s_last;
  __shared__ float st[16 * kStRow];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const int a_bytes = p.NB * kBK * 2;
  const int stage_bytes = kWBytes + 2 * a_bytes;
  const int n_kb = p.K / kBK;
  const int n_tiles = p.n_ntiles * p.n_mchunks;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      ptx::mbar_init(&full_bar[i], 1);
      ptx::mbar_init(&empty_bar[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&tmem_full[i], 1);
      ptx::mbar_init(&tmem_empty[i], 128);
    }
    s_abort = 0;
    s_last = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_w);
    ptx::prefetch_tmap(&tm_hi);
    ptx::prefetch_tmap(&tm_lo);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&s_tmem_base, (uint32_t)p.tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x) {
        const int n0 = (tile / p.n_mchunks) * kTileN, m0 = (tile % p.n_mchunks) * p.NB;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % p.stages;
          const uint32_t ph = (it / p.stages) & 1u;
          if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1u, abort_flag, p.err)) break;
          uint8_t* stage = smem + (size_t)s * stage_bytes;
          ptx::mbar_arrive_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
          ptx::tma_load_2d(stage, &tm_w, kb * kBK, n0, &full_bar[s]);
          ptx::tma_load_2d(stage + kWBytes, &tm_hi, kb * kBK, m0, &full_bar[s]);
          ptx::tma_load_2d(stage + kWBytes + a_bytes, &tm_lo, kb * kBK, m0, &full_bar[s]);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- UMMA issue ----------------
    if (lane == 0) {
      const uint32_t idesc = ptx::umma_idesc_bf16(kTileN, p.NB);
      uint32_t it = 0, ti = 0;
      for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x, ++ti) {
        const uint32_t acc = ti & 1u, aph = (ti >> 1) & 1u;
        if (!ptx::mbar_wait(&tmem_empty[acc], aph ^ 1u, abort_flag, p.err)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * (uint32_t)p.NB;
        bool ok = true;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % p.stages;
          const uint32_t ph = (it / p.stages) & 1u;
          if (!ptx::mbar_wait(&full_bar[s], ph, abort_flag, p.err)) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t w_addr = smem_base + (uint32_t)s * stage_bytes;
          const uint32_t hi_addr = w_addr + kWBytes, lo_addr = hi_addr + a_bytes;
#pragma unroll
          for (int ks = 0; ks < kBK / 16; ++ks) {
            const uint64_t wd = ptx::umma_desc_sw128(w_addr + ks * 32);
            ptx::umma_bf16(d_tmem, wd, ptx::umma_desc_sw128(hi_addr + ks * 32), idesc, (kb | ks) != 0);
            ptx::umma_bf16(d_tmem, wd, ptx::umma_desc_sw128(lo_addr + ks * 32), idesc, 1u);
          }
          ptx::umma_commit(&empty_bar[s]);  // stage reusable once these UMMAs have read it
        }
        if (!ok) break;
        ptx::umma_commit(&tmem_full[acc]);
      }
    }
  } else {
    // ---------------- epilogue (128 threads) ----------------
    const int quad = warp & 3;                  // TMEM lane quadrant this warp may read
    const int vl = quad * 32 + lane;            // weight row within the tile
    const int eid = (warp - 2) * 32 + lane;     // 0..127
    const int st_m = eid >> 3, st_part = eid & 7;
    uint32_t ti = 0;
    for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x, ++ti) {
      const uint32_t acc = ti & 1u, aph = (ti >> 1) & 1u;
      const int n_tile = tile / p.n_mchunks;
      const int n = n_tile * kTileN + vl, m0 = (tile % p.n_mchunks) * p.NB;
      if (!ptx::mbar_wait(&tmem_full[acc], aph, abort_flag, p.err)) break;
      ptx::tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * (uint32_t)p.NB;
      for (int c0 = 0; c0 < p.NB; c0 += 16) {
        float v[16];
        ptx::tmem_ld16(t_addr + c0, v);
        if (p.C != nullptr && n < p.N) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int m = m0 + c0 + i;
            if (m < p.M) p.C[(size_t)m * p.ldc + n] = v[i];
          }
        }
        if (p.part != nullptr) {
          ptx::named_bar_sync(1, 128);  // the previous chunk has been read
#pragma unroll
          for (int i = 0; i < 16; ++i) st[i * kStRow + vl] = (n < p.N) ? v[i] : -INFINITY;
          ptx::named_bar_sync(1, 128);
          float mx = -INFINITY;
#pragma unroll
          for (int i = 0; i < 16; ++i) mx = fmaxf(mx, st[st_m * kStRow + st_part + 8 * i]);
          float sum = 0.f;
          if (mx != -INFINITY) {
#pragma unroll
            for (int i = 0; i < 16; ++i) sum += __expf(st[st_m * kStRow + st_part + 8 * i] - mx);
          }
#pragma unroll
          for (int o = 1; o < 8; o <<= 1) {
            const float mo = __shfl_xor_sync(0xffffffffu, mx, o), so = __shfl_xor_sync(0xffffffffu, sum, o);
            combine_ms(mx, sum, mo, so);
          }
          const int m = m0 + c0 + st_m;
          if (st_part == 0 && m < p.M) p.part[(size_t)m * p.part_ld + n_tile] = make_float2(mx, sum);
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tmem_empty[acc]);
    }
    __threadfence();
  }
  __syncwarp();
  __syncthreads();
  if (*abort_flag) __nanosleep(500000);  // let copies still in flight land before the CTA goes away
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
  if (p.part == nullptr) return;
  // ---------------- last CTA folds the tile partials into row-wise log-sum-exp ----------------
  if (threadIdx.x == 0) {
    const unsigned int ticket = atomicAdd(p.counter, 1u);
    s_last = (ticket == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int m = warp; m < p.M; m += kThreads / 32) {
    float mx = -INFINITY, sum = 0.f;
    for (int t = lane; t < p.n_ntiles; t += 32) {
      const float2 ms = __ldcg(&p.part[(size_t)m * p.part_ld + t]);
      combine_ms(mx, sum, ms.x, ms.y);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float mo = __shfl_xor_sync(0xffffffffu, mx, o), so = __shfl_xor_sync(0xffffffffu, sum, o);
      combine_ms(mx, sum, mo, so);
    }
    if (lane == 0) p.lse[m] = mx + logf(sum);
  }
  if (threadIdx.x == 0) *p.counter = 0u;
}

}  // namespace

int launch_gemm_tc(cascade_ctx* ctx, const __nv_bfloat16* W, int N, int K, const __nv_bfloat16* a_hi,
                   const __nv_bfloat16* a_lo, int M, float* C, int ldc, float2* part, int part_ld, float* lse,
                   int kernel_id, cudaStream_t s) {
  if (K % kBK != 0 || M < 1 || N < 1) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  GemmArgs a;
  a.M = M;
  a.N = N;
  a.K = K;
  a.NB = M <= 256 ? (int)cascade_detail::align_up(M, 16) : 128;
  a.n_ntiles = cascade_detail::ceil_div(N, kTileN);
  a.n_mchunks = cascade_detail::ceil_div(M, a.NB);
  const int stage_bytes = kWBytes + 2 * a.NB * kBK * 2;
  const int budget = 227 * 1024 - 12 * 1024 - 1024;  // static shared + alignment slack
  a.stages = budget / stage_bytes;
  if (a.stages > kMaxStages) a.stages = kMaxStages;
  if (a.stages < 2) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  a.tmem_cols = 32;
  while (a.tmem_cols < 2 * a.NB) a.tmem_cols *= 2;
  a.C = C;
  a.ldc = ldc;
  a.part = part;
  a.part_ld = part_ld;
  a.lse = lse;
  a.counter = ctx->gemm_counter;
  a.err = ctx->dev_error;
  if (part != nullptr && (lse == nullptr || part_ld < a.n_ntiles)) return CASCADE_ERR_INVALID_ARG;
  const CUtensorMap* tw = get_tmap_2d_bf16(ctx, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, kTileN, kBK);
  const CUtensorMap* thi = get_tmap_2d_bf16(ctx, a_hi, (uint64_t)M, (uint64_t)K, (uint64_t)K, (uint32_t)a.NB, kBK);
  const CUtensorMap* tlo = get_tmap_2d_bf16(ctx, a_lo, (uint64_t)M, (uint64_t)K, (uint64_t)K, (uint32_t)a.NB, kBK);
  if (tw == nullptr || thi == nullptr || tlo == nullptr) return CASCADE_ERR_CUDA;
  const int smem = a.stages * stage_bytes + 1024;
  static int configured_smem = 0;
  if (smem > configured_smem) {
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured_smem = smem;
  }
  const int n_tiles = a.n_ntiles * a.n_mchunks;
  const int grid = n_tiles < ctx->sm_count ? n_tiles : ctx->sm_count;
  {
    KernelScope ks(ctx, kernel_id, s);
    k_gemm_tc<<<grid, kThreads, smem, s>>>(*tw, *thi, *tlo, a);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

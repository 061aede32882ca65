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
//   * the work is the flattened list of (weight tile, K block) units, cut into one contiguous,
//     equally long range per CTA (one CTA per SM), so every SM streams the same number of weight
//     bytes whatever the number of tiles.  A CTA whose range starts inside a tile adds its partial
//     accumulator to a scratch slot and raises a flag; the CTA that holds the tile's first K block
//     reaches that tile last, adds the partials of the CTAs after it in index order (deterministic)
//     and runs the epilogue.  The launch is cooperative, so all CTAs are resident; the wait is bounded;
//   * a TMA producer thread keeps a ring of [W 128 x BK | Ahi NB x BK | Alo NB x BK] bf16 stages
//     (128-byte swizzle) in flight, one thread issues the UMMAs (the high part and the remainder of the
//     activation operand accumulate into the same fp32 TMEM accumulator), and four epilogue warps
//     drain one of two TMEM accumulators while the next tile is being accumulated into the other.
//     The producer and issue loops are kept to a few dozen instructions per stage: a single thread
//     retires an instruction every few cycles, and at 16 KB of weights per round trip that latency,
//     not HBM, was the limit;
//   * epilogue: TMEM lane = weight row n, column = activation row m.  Optional store of (or addition
//     into) C, coalesced over n; optional per-(m, tile) softmax partials (max, sum of exp) and gather
//     of the few logits the acceptance rule reads (Algorithm 2: q_x = gtp[x]).
// Every mbarrier / flag wait is bounded; on expiry the CTA records an error word and leaves through
// the normal teardown (TMEM is freed).
#include "cascade_internal.h"
#include "gemm_tc.h"
#include "ptx.cuh"
#include "tmap.h"

namespace {

constexpr int kThreads = 192;       // warp 0: TMA, warp 1: UMMA issue + TMEM alloc, warps 2-5: epilogue
constexpr int kTileN = 128;         // weight rows per tile (UMMA M)
constexpr int kSpan = 64;           // K elements per 128-byte swizzle span
constexpr int kMaxStages = 8;
constexpr int kStRow = 136;         // staging row stride (floats): 136 = 8 mod 32 keeps reads conflict-free
constexpr int kWSpanBytes = kTileN * kSpan * 2;

struct GemmArgs {
  int M, N, NB, n_mchunks, n_kb, stages, tmem_cols;
  long long units;      // n_tiles * n_kb
  GemmEpilogue epi;
  float* sk_scratch;    // [grid][NB][128] partial accumulators of split tiles
  unsigned int* sk_flags;
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

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned int* p, unsigned int v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// One contiguous piece of a CTA's range: K blocks [kb0, kb1) of `tile`.
struct Segment {
  int tile, kb0, kb1;
};
struct SegmentWalk {
  long long u, u_end;
  int n_kb;
  __device__ SegmentWalk(const GemmArgs& p) : n_kb(p.n_kb) {
    u = (long long)blockIdx.x * p.units / gridDim.x;
    u_end = (long long)(blockIdx.x + 1) * p.units / gridDim.x;
  }
  __device__ bool next(Segment& s) {
    if (u >= u_end) return false;
    s.tile = (int)(u / n_kb);
    s.kb0 = (int)(u - (long long)s.tile * n_kb);
    const long long left = u_end - u;
    s.kb1 = left < (long long)(n_kb - s.kb0) ? s.kb0 + (int)left : n_kb;
    u += s.kb1 - s.kb0;
    return true;
  }
};

template <int kSpans>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_a, const GemmArgs p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tmem_full[2], tmem_empty[2];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  __shared__ float st[16 * kStRow];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const int a_span_bytes = 2 * p.NB * kSpan * 2;  // hi block then lo block of one span
  const int stage_bytes = kSpans * (kWSpanBytes + a_span_bytes);

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
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_w);
    ptx::prefetch_tmap(&tm_a);
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
      int s = 0;
      uint32_t ph = 0;
      const int stages = p.stages, n_mchunks = p.n_mchunks, NB = p.NB;
      SegmentWalk walk(p);
      Segment sg;
      bool ok = true;
      while (ok && walk.next(sg)) {
        const int n0 = (sg.tile / n_mchunks) * kTileN, m0 = (sg.tile % n_mchunks) * NB;
        for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
          if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1u, abort_flag, p.err)) {
            ok = false;
            break;
          }
          uint8_t* stage = smem + s * stage_bytes;
          ptx::mbar_arrive_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
#pragma unroll
          for (int q = 0; q < kSpans; ++q)
            ptx::tma_load_2d(stage + q * kWSpanBytes, &tm_w, (kb * kSpans + q) * kSpan, n0, &full_bar[s]);
#pragma unroll
          for (int q = 0; q < kSpans; ++q)
            ptx::tma_load_3d(stage + kSpans * kWSpanBytes + q * a_span_bytes, &tm_a, (kb * kSpans + q) * kSpan, m0, 0,
                             &full_bar[s]);
          if (++s == stages) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- UMMA issue ----------------
    if (lane == 0) {
      const uint32_t idesc = ptx::umma_idesc_bf16(kTileN, p.NB);
      const int stages = p.stages;
      const uint32_t lo_off = (uint32_t)(p.NB * kSpan * 2) >> 4;  // descriptor units of 16 bytes
      int s = 0;
      uint32_t ph = 0, seg_i = 0;
      SegmentWalk walk(p);
      Segment sg;
      bool ok = true;
      while (ok && walk.next(sg)) {
        const uint32_t acc = seg_i & 1u, aph = (seg_i >> 1) & 1u;
        ++seg_i;
        if (!ptx::mbar_wait(&tmem_empty[acc], aph ^ 1u, abort_flag, p.err)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * (uint32_t)p.NB;
        uint32_t accumulate = 0;
        for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
          if (!ptx::mbar_wait(&full_bar[s], ph, abort_flag, p.err)) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t w_addr = smem_base + (uint32_t)(s * stage_bytes);
          const uint32_t a_addr = w_addr + kSpans * kWSpanBytes;
#pragma unroll
          for (int q = 0; q < kSpans; ++q) {
            const uint64_t wd0 = ptx::umma_desc_sw128(w_addr + q * kWSpanBytes);
            const uint64_t ad0 = ptx::umma_desc_sw128(a_addr + q * a_span_bytes);
#pragma unroll
            for (int ks = 0; ks < kSpan / 16; ++ks) {
              // advancing 16 K elements = 32 bytes = 2 descriptor units inside the swizzle span
              ptx::umma_bf16(d_tmem, wd0 + 2 * ks, ad0 + 2 * ks, idesc, accumulate);
              accumulate = 1u;
              ptx::umma_bf16(d_tmem, wd0 + 2 * ks, ad0 + lo_off + 2 * ks, idesc, 1u);
            }
          }
          ptx::umma_commit(&empty_bar[s]);  // stage reusable once these UMMAs have read it
          if (++s == stages) {
            s = 0;
            ph ^= 1u;
          }
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
    const GemmEpilogue& e = p.epi;
    const int NB = p.NB;
    uint32_t seg_i = 0;
    SegmentWalk walk(p);
    Segment sg;
    while (walk.next(sg)) {
      const uint32_t acc = seg_i & 1u, aph = (seg_i >> 1) & 1u;
      ++seg_i;
      const int n_tile = sg.tile / p.n_mchunks;
      const int n = n_tile * kTileN + vl, m0 = (sg.tile % p.n_mchunks) * NB;
      const bool contributor = sg.kb0 > 0;
      const bool owner_of_split = sg.kb0 == 0 && sg.kb1 < p.n_kb;
      int n_contrib = 0;
      if (owner_of_split) {
        // the CTAs after this one whose range starts inside this tile each hold one partial of it
        const long long tile_end = (long long)(sg.tile + 1) * p.n_kb;
        for (int c = blockIdx.x + 1; c < (int)gridDim.x && (long long)c * p.units / gridDim.x < tile_end; ++c) ++n_contrib;
        if (eid == 0) {
          for (int i = 1; i <= n_contrib && !*abort_flag; ++i) {
            const unsigned int* f = p.sk_flags + blockIdx.x + i;
            if (ld_acquire(f) != 0u) continue;
            const uint64_t t0 = ptx::global_timer_ns();
            uint32_t polls = 0;
            while (ld_acquire(f) == 0u) {
              if ((++polls & 63u) == 0 && ptx::global_timer_ns() - t0 > ptx::kWaitLimitNs) {
                *abort_flag = 1;
                atomicOr(p.err, 1);
                break;
              }
            }
          }
        }
        ptx::named_bar_sync(1, 128);
      }
      if (*abort_flag) break;
      if (!ptx::mbar_wait(&tmem_full[acc], aph, abort_flag, p.err)) break;
      ptx::tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * (uint32_t)NB;
      for (int c0 = 0; c0 < NB; c0 += 16) {
        float v[16];
        ptx::tmem_ld16(t_addr + c0, v);
        if (contributor) {
          float* slot = p.sk_scratch + ((size_t)blockIdx.x * NB + c0) * kTileN + vl;
#pragma unroll
          for (int i = 0; i < 16; ++i) slot[(size_t)i * kTileN] = v[i];
          continue;
        }
        for (int k = 1; k <= n_contrib; ++k) {
          const float* slot = p.sk_scratch + ((size_t)(blockIdx.x + k) * NB + c0) * kTileN + vl;
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] += __ldcg(slot + (size_t)i * kTileN);
        }
        if (e.C != nullptr && n < p.N) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int m = m0 + c0 + i;
            if (m < p.M) {
              float* dst = e.C + (size_t)m * e.ldc + n;
              *dst = e.accumulate ? *dst + v[i] : v[i];
            }
          }
        }
        if (e.part != nullptr) {
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
          if (st_part == 0 && m < p.M) e.part[(size_t)m * e.part_ld + n_tile] = make_float2(mx, sum);
          if (e.tok != nullptr) {
            // logits the acceptance rule reads: tok[idx] under its parent's and grandparent's rows
            for (int idx = eid; idx < e.n_rows; idx += 128) {
              const int ln = e.tok[idx] - n_tile * kTileN;
              if ((unsigned)ln >= (unsigned)kTileN) continue;
              const int b = idx / e.T, j = idx - b * e.T;
              const int pi = e.parent[j];
              if (pi < 0) continue;
              int col = b * e.T + pi - m0 - c0;
              if ((unsigned)col < 16u) e.cand_parent[idx] = st[col * kStRow + ln];
              const int gp = e.parent[pi];
              if (gp < 0) continue;
              col = b * e.T + gp - m0 - c0;
              if ((unsigned)col < 16u) e.cand_gparent[idx] = st[col * kStRow + ln];
            }
          }
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tmem_empty[acc]);
      if (contributor) {
        __threadfence();
        ptx::named_bar_sync(1, 128);
        if (eid == 0) st_release(p.sk_flags + blockIdx.x, 1u);
      } else if (n_contrib > 0) {
        ptx::named_bar_sync(1, 128);  // every thread has read the partials
        if (eid == 0)
          for (int k = 1; k <= n_contrib; ++k) p.sk_flags[blockIdx.x + k] = 0u;  // ready for the next launch
      }
    }
  }
  __syncwarp();
  __syncthreads();
  if (*abort_flag) __nanosleep(500000);  // let copies still in flight land before the CTA goes away
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

}  // namespace

int64_t gemm_tc_scratch_floats(int sm_count) { return (int64_t)sm_count * 256 * kTileN; }

int launch_gemm_tc(cascade_ctx* ctx, const __nv_bfloat16* W, int N, int K, const __nv_bfloat16* a_hi,
                   int64_t lo_offset, int M, const GemmEpilogue& epi, int kernel_id, cudaStream_t s) {
  if (K % 8 != 0 || M < 1 || N < 1 || lo_offset % 8 != 0) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  if (epi.part != nullptr && epi.part_ld < cascade_detail::ceil_div(N, kTileN)) return CASCADE_ERR_INVALID_ARG;
  if (epi.tok != nullptr && (epi.part == nullptr || epi.parent == nullptr || epi.cand_parent == nullptr ||
                             epi.cand_gparent == nullptr || epi.T < 1))
    return CASCADE_ERR_INVALID_ARG;
  GemmArgs a;
  a.M = M;
  a.N = N;
  a.NB = M <= 256 ? (int)cascade_detail::align_up(M, 16) : 128;
  a.n_mchunks = cascade_detail::ceil_div(M, a.NB);
  a.epi = epi;
  a.sk_scratch = ctx->gemm_scratch;
  a.sk_flags = ctx->gemm_flags;
  a.err = ctx->dev_error;
  const int budget = 227 * 1024 - 12 * 1024 - 1024;  // static shared + alignment slack
  // two swizzle spans per stage when at least three such stages fit, else one
  const int stage1 = kWSpanBytes + 2 * a.NB * kSpan * 2;
  const int spans = (budget / (2 * stage1) >= 3) ? 2 : 1;
  const int stage_bytes = spans * stage1;
  a.stages = budget / stage_bytes;
  if (a.stages > kMaxStages) a.stages = kMaxStages;
  if (a.stages < 2) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  a.n_kb = cascade_detail::ceil_div(K, kSpan * spans);
  const int n_tiles = cascade_detail::ceil_div(N, kTileN) * a.n_mchunks;
  a.units = (long long)n_tiles * a.n_kb;
  a.tmem_cols = 32;
  while (a.tmem_cols < 2 * a.NB) a.tmem_cols *= 2;
  const CUtensorMap* tw = get_tmap_2d_bf16(ctx, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, kTileN, kSpan);
  const uint64_t ad[3] = {(uint64_t)K, (uint64_t)M, 2};
  const uint64_t as[2] = {(uint64_t)K, (uint64_t)lo_offset};
  const uint32_t ab[3] = {kSpan, (uint32_t)a.NB, 2};
  const CUtensorMap* ta = get_tmap_bf16(ctx, a_hi, 3, ad, as, ab);
  if (tw == nullptr || ta == nullptr) return CASCADE_ERR_CUDA;
  const int smem = a.stages * stage_bytes + 1024;
  auto kern = spans == 2 ? k_gemm_tc<2> : k_gemm_tc<1>;
  static int configured_smem[2] = {0, 0};
  if (smem > configured_smem[spans - 1]) {
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured_smem[spans - 1] = smem;
  }
  long long grid = a.units < ctx->sm_count ? a.units : ctx->sm_count;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: the split-tile hand-off waits on peers
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  {
    KernelScope ks(ctx, kernel_id, s);
    CASCADE_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, *tw, *ta, a));
  }
  return CASCADE_OK;
}

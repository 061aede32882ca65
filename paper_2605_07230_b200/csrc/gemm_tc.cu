// Weight-streaming skinny GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
//     C[m][n] = sum_k (Ahi[m][k] + Alo[m][k]) * W[n][k]        m < M (few rows), n < N (many rows)
//
// This is the LM head (W = [V,h], the O(hV) projection that Section 4.2 of the paper names as the
// dominant cost of verification) and every other projection of the decoder layer.  With M of the
// order of the draft-tree size the product is bound by streaming W from HBM once, so the kernel is
// organised around that stream:
//   * the WEIGHT rows sit on the UMMA M dimension and the activation rows on the UMMA N dimension
//     (NB = M rounded up to 16, <= 128), so no tensor-core work is spent on padding a small M up to
//     128.  A work tile is 128 weight rows (kHalves = 1; the kernel also takes 256-row tiles, two
//     accumulators on one activation stage);
//   * two ways of spreading the work over the SMs (one CTA per SM):
//       contiguous (splits = 0): the flattened list of (tile, K block) units is cut into one equally
//         long range per CTA, so every SM streams the same number of weight bytes whatever the number
//         of tiles.  A CTA whose range starts inside a tile writes its partial accumulator to a
//         scratch slot and raises a flag; the CTA that holds the tile's first K block reaches that tile
//         last, adds the partials of the CTAs after it in index order (deterministic; they were
//         produced earlier, so they are summed into spare TMEM columns while this CTA's own UMMAs run) and
//         runs the epilogue.  The launch is cooperative, so all CTAs are resident; the wait is bounded;
//       sliced (splits = S): K is cut into S slices, work item (tile, slice) writes its own output
//         matrix and the consumer adds the S matrices.  Nothing waits inside the kernel; this is for
//         weight matrices with so few tiles that each would be cut many times;
//   * a TMA producer thread keeps a ring of [W rows x 64 | Ahi NB x 64 | Alo NB x 64] bf16 stages
//     (128-byte swizzle) in flight -- the weights by tiled TMA loads, the activations, which their
//     producers already store in the staged layout (operand.cuh), by one contiguous bulk copy --, one thread issues the UMMAs (the high part and the remainder of the
//     activation operand accumulate into the same fp32 TMEM accumulator), and four epilogue warps
//     drain one of two TMEM accumulator sets while the next tile is being accumulated into the other.
//     The producer and issue loops are kept to a few dozen instructions per stage: a single thread
//     retires an instruction every few cycles, and that latency, not HBM, is the limit otherwise;
//   * epilogue: TMEM lane = weight row n (within a 128-row tile), column = activation row m.  Optional
//     store of (or addition into) C, coalesced over n; optional per-(m, tile) softmax partials
//     (max, sum of exp) and gather of the few logits the acceptance rule reads (Algorithm 2:
//     q_x = gtp[x]).
// Every mbarrier / flag wait is bounded; on expiry the CTA records an error word and leaves through
// the normal teardown (TMEM is freed).
#include "cascade_internal.h"
#include "gemm_tc.h"
#include "operand.cuh"
#include "ptx.cuh"
#include "tmap.h"

namespace {

constexpr int kThreads = 192;       // warp 0: TMA, warp 1: UMMA issue + TMEM alloc, warps 2-5: epilogue
constexpr int kLeanThreads = 320;   // ... warps 2-9: epilogue of the sliced projections
constexpr int kTileN = 128;         // weight rows per accumulator (UMMA M)
constexpr int kSpan = 64;           // K elements per stage (one 128-byte swizzle span)
constexpr int kMaxStages = 8;
constexpr int kGatherCap = 128;     // candidate logits one 128-row tile can serve from the shared list
constexpr int kStCols = 32;         // activation rows staged per softmax round
constexpr int kStRow = 132;         // floats per staged activation row: 4 runs of 33 (32 weight rows + 1 pad)
constexpr int kTileWBytes = kTileN * kSpan * 2;

struct GemmArgs {
  int M, N, NB, n_mchunks, n_kb, stages, tmem_cols;
  const __nv_bfloat16* A;  // activation operand in the staged layout of operand.cuh
  long long a_chunk_elems; // elements of one row chunk of A (all its K blocks)
  int stash;               // 1: TMEM has room for a third accumulator set (partials of split tiles)
  int combine;             // 1: one UMMA per K step over both parts of the operand (N = 2 NB), parts added in the epilogue
  int acc_cols;            // TMEM columns of one accumulator set
  long long units;         // n_tiles * n_kb
  int unit_q, unit_r;      // units = grid * unit_q + unit_r: CTA c starts at unit c * unit_q + min(c, unit_r)
  int n_tiles;
  int splits;              // 0: contiguous ranges with in-kernel hand-off; S >= 1: S K slices per tile
  int balanced;            // 1: contiguous ranges, every piece of a tile to its own output matrix (no hand-off)
  long long slice_stride;  // floats between the C matrices of consecutive K slices
  GemmEpilogue epi;
  float* sk_scratch;       // [grid][halves][NB][128] partial accumulators of split tiles
  unsigned int* sk_flags;
  int* err;
  unsigned long long wait_ns;  // limit of every bounded wait in the kernel
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

// One piece of work: K blocks [kb0, kb1) of `tile`; `slice` selects the output matrix in sliced mode.
struct Segment {
  int tile, kb0, kb1, slice;
};
// Contiguous mode (splits == 0): the flattened (tile, K block) list is cut into one range per CTA and
// a segment is the part of a tile inside that range.  Sliced mode: work item w = (tile, K slice), taken
// round-robin by the CTAs.  All of it in 32-bit arithmetic without a 64-bit division (the launcher checks
// the ranges): this runs in single threads at the head of the kernel, before the first load can go out.
// First unit of CTA c in contiguous mode.
__device__ __forceinline__ int range_begin(const GemmArgs& p, int c) { return c * p.unit_q + min(c, p.unit_r); }
struct SegmentWalk {
  int u, u_end;
  int n_kb, splits, w, n_items;
  int first_q, first_r;  // balanced mode: for the number of a piece within its tile
  __device__ SegmentWalk(const GemmArgs& p) : n_kb(p.n_kb), splits(p.balanced ? 0 : p.splits) {
    first_q = p.balanced ? p.unit_q : 0;
    first_r = p.unit_r;
    u = range_begin(p, blockIdx.x);
    u_end = range_begin(p, blockIdx.x + 1);
    w = blockIdx.x;
    n_items = p.n_tiles * p.splits;
  }
  __device__ bool next(Segment& s) {
    if (splits > 0) {
      if (w >= n_items) return false;
      s.tile = w / splits;
      s.slice = w - s.tile * splits;
      s.kb0 = s.slice * n_kb / splits;
      s.kb1 = (s.slice + 1) * n_kb / splits;
      w += gridDim.x;
      return true;
    }
    if (u >= u_end) return false;
    s.tile = u / n_kb;
    s.slice = 0;
    if (first_q > 0) {  // this CTA's index minus the index of the CTA that holds the tile's first K block
      const int u0 = s.tile * n_kb, big = first_r * (first_q + 1);
      s.slice = (int)blockIdx.x - (u0 < big ? u0 / (first_q + 1) : first_r + (u0 - big) / first_q);
    }
    s.kb0 = u - s.tile * n_kb;
    const int left = u_end - u;
    s.kb1 = left < n_kb - s.kb0 ? s.kb0 + left : n_kb;
    u += s.kb1 - s.kb0;
    return true;
  }
};

// kHalves: accumulators (128 weight rows each) per work tile.  kSpans: 64-wide K spans per stage.
// kLean: the plain-store epilogue of the sliced projections, run by EIGHT warps (two per TMEM lane quadrant, each
// group of four taking every other 32-column block of the tile).  What a CTA does after its last UMMA is not hidden
// behind anything, and all CTAs get there together: four warps drain a 128 KB tile at about 30 GB/s per SM (their
// instruction stream, not the memory system, sets that rate), eight in half the time.  The general epilogue
// (softmax partials, candidate gather, split-tile hand-off) needs more registers than 320 threads leave and keeps
// its four warps.
template <int kHalves, int kSpans, bool kLean>
__global__ void __launch_bounds__(kLean ? kLeanThreads : kThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tm_w, const GemmArgs p) {
  constexpr int kWSpanBytes = kHalves * kTileWBytes;  // weights of one span
  constexpr int kWBytes = kSpans * kWSpanBytes;       // weights of one stage: span after span
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tmem_full[2], tmem_empty[2];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const int a_span_bytes = 2 * p.NB * kSpan * 2;  // one span of the activations: hi block, lo block
  const int stage_bytes = kWBytes + kSpans * a_span_bytes;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      ptx::mbar_init(&full_bar[i], 1);
      ptx::mbar_init(&empty_bar[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&tmem_full[i], 1);
      ptx::mbar_init(&tmem_empty[i], kLean ? kLeanThreads - 64 : 128);
    }
    s_abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_w);
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
      const uint64_t pol_w = ptx::l2_evict_first(), pol_a = ptx::l2_evict_last();  // weights pass through once
      SegmentWalk walk(p);
      Segment sg;
      bool ok = true;
      while (ok && walk.next(sg)) {
        const int n0 = (sg.tile / n_mchunks) * (kHalves * kTileN);
        const __nv_bfloat16* a_chunk = p.A + (size_t)(sg.tile % n_mchunks) * p.a_chunk_elems;
        for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
          if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1u, abort_flag, p.err, p.wait_ns)) {
            ok = false;
            break;
          }
          uint8_t* stage = smem + s * stage_bytes;
          ptx::mbar_arrive_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
#pragma unroll
          for (int q = 0; q < kSpans; ++q)
            ptx::tma_load_2d_hint(stage + q * kWSpanBytes, &tm_w, (kb * kSpans + q) * kSpan, n0, &full_bar[s], pol_w);
          // the activations of these K blocks are contiguous in the staged layout: one bulk copy
          ptx::bulk_load_hint(stage + kWBytes, a_chunk + (size_t)kb * (kSpans * 2 * NB * kSpan),
                              (uint32_t)(kSpans * a_span_bytes), &full_bar[s], pol_a);
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
      // combine: the high parts and the remainders of the activation rows are one 2 NB-row operand (the two
      // blocks are adjacent in a stage), their products land in separate column ranges and meet in the
      // epilogue: half as many UMMAs, and the weight tile is read from shared memory once per K step
      const uint32_t idesc = ptx::umma_idesc_bf16(kTileN, p.combine ? 2 * p.NB : p.NB);
      const bool combine = p.combine != 0;
      const int stages = p.stages;
      const uint32_t lo_off = (uint32_t)(p.NB * kSpan * 2) >> 4;  // descriptor units of 16 bytes
      int s = 0;
      uint32_t ph = 0, seg_i = 0;
      SegmentWalk walk(p);
      Segment sg;
      bool ok = true;
      // The first trip through the issue loop runs with every tensor-core instruction predicated off and
      // waits for nothing: it only pulls the loop into the instruction cache (cold at every launch, the
      // weights having streamed through the L2 since) while the first stage is still on its way.  The
      // flag comes out of an asm statement so that the compiler keeps one copy of the loop.
      uint32_t live;
      asm volatile("mov.u32 %0, 0;" : "=r"(live));
      while (ok && walk.next(sg)) {
        const uint32_t acc = seg_i & 1u, aph = (seg_i >> 1) & 1u;
        ++seg_i;
        if (!ptx::mbar_wait(&tmem_empty[acc], aph ^ 1u, abort_flag, p.err, p.wait_ns)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * (uint32_t)p.acc_cols;
        uint32_t accumulate = 0;
        for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
          if (live != 0u) {
            if (!ptx::mbar_wait(&full_bar[s], ph, abort_flag, p.err, p.wait_ns)) {
              ok = false;
              break;
            }
            ptx::tc_fence_after();
          }
          const uint32_t w_addr = smem_base + (uint32_t)(s * stage_bytes);
#pragma unroll
          for (int q = 0; q < kSpans; ++q) {
            const uint64_t ad0 = ptx::umma_desc_sw128(w_addr + kWBytes + q * a_span_bytes);
#pragma unroll
            for (int t = 0; t < kHalves; ++t) {
              const uint64_t wd0 = ptx::umma_desc_sw128(w_addr + q * kWSpanBytes + t * kTileWBytes);
              const uint32_t d = d_tmem + t * (uint32_t)p.NB;
#pragma unroll
              for (int ks = 0; ks < kSpan / 16; ++ks) {
                // advancing 16 K elements = 32 bytes = 2 descriptor units inside the swizzle span
                ptx::umma_bf16_if(live, d, wd0 + 2 * ks, ad0 + 2 * ks, idesc, (q | ks) == 0 ? accumulate : 1u);
                if (!combine) ptx::umma_bf16_if(live, d, wd0 + 2 * ks, ad0 + lo_off + 2 * ks, idesc, 1u);
              }
            }
          }
          ptx::umma_commit_if(live, &empty_bar[s]);  // stage reusable once these UMMAs have read it
          if (live == 0u) {
            asm volatile("mov.u32 %0, 1;" : "=r"(live));
            --kb;  // now for real
            continue;
          }
          accumulate = 1u;
          if (++s == stages) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (!ok) break;
        ptx::umma_commit(&tmem_full[acc]);
      }
    }
  } else if constexpr (kLean) {
    // ---------------- plain-store epilogue (256 threads: two groups of four warps) ----------------
    __shared__ __align__(16) float st2[2][32 * kTileN];   // per group: 32 activation rows x 128 weight rows
    const int quad = warp & 3;                  // TMEM lane quadrant this warp may read
    const int vl = quad * 32 + lane;            // weight row within the tile
    const int group = (warp - 2) >> 2, gwarp = (warp - 2) & 3;
    float* const stg = st2[group];
    const GemmEpilogue& e = p.epi;
    const int NB = p.NB;
    const int blocks_per_half = (NB + 31) / 32;
    uint32_t seg_i = 0;
    SegmentWalk walk(p);
    Segment sg;
    while (walk.next(sg)) {
      const uint32_t acc = seg_i & 1u, aph = (seg_i >> 1) & 1u;
      ++seg_i;
      const int macro = sg.tile / p.n_mchunks, m0 = (sg.tile % p.n_mchunks) * NB;
      float* const c_out = e.C + (size_t)sg.slice * p.slice_stride;
      if (!ptx::mbar_wait(&tmem_full[acc], aph, abort_flag, p.err, p.wait_ns)) break;
      ptx::tc_fence_after();
#pragma unroll 1  // run-once code at the end of the kernel: one copy of the block's instructions
      for (int blk = group; blk < kHalves * blocks_per_half; blk += 2) {
        const int half = blk / blocks_per_half, c0 = (blk - half * blocks_per_half) * 32;
        const int n_tile = macro * kHalves + half;
        if (n_tile * kTileN >= p.N) break;      // second half of the last work tile lies beyond N
        const int n_cols = min(32, NB - c0);
        const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * (uint32_t)p.acc_cols +
                                half * (uint32_t)NB + (uint32_t)c0;
        float v[32];
        if (n_cols == 32) {
          ptx::tmem_ld32(t_addr, v);
        } else {
          ptx::tmem_ld16(t_addr, v);            // NB is a multiple of 16: the last block of a half may hold 16 columns
        }
        ptx::named_bar_sync(1 + group, 128);    // the previous block has been read out of the staging buffer
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i < n_cols) stg[i * kTileN + vl] = v[i];
        ptx::named_bar_sync(1 + group, 128);
        // output rows are contiguous over the weight rows: a warp writes the 128 weight rows of an activation row
        // with one 16-byte store per lane
        const int row0 = m0 + c0, n0 = n_tile * kTileN + 4 * lane;
        const bool wide = (e.ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(c_out) & 15u) == 0 && n0 + 4 <= p.N;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int i = gwarp + 4 * k;
          if (i >= n_cols || row0 + i >= p.M) continue;
          const float4 x = *reinterpret_cast<const float4*>(stg + i * kTileN + 4 * lane);
          float* dst = c_out + (size_t)(row0 + i) * e.ldc + n0;
          if (wide) {
            *reinterpret_cast<float4*>(dst) = x;
          } else {
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (n0 + q < p.N) dst[q] = xs[q];
          }
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tmem_empty[acc]);
    }
  } else {
    // ---------------- epilogue (128 threads) ----------------
    __shared__ __align__(16) float st[kStCols * kStRow];
    __shared__ int s_gather_n;
    __shared__ int4 s_gather[kGatherCap];  // {weight row in tile, parent column, grandparent column, idx}
    const int quad = warp & 3;                  // TMEM lane quadrant this warp may read
    const int vl = quad * 32 + lane;            // weight row within the tile
    const int eid = (warp - 2) * 32 + lane;     // 0..127
    const int st_col = eid >> 2, st_part = eid & 3;  // softmax round: 4 threads per staged activation row
    const int st_wr = (vl >> 5) * 33 + (vl & 31);    // where this thread's weight row goes in a staged row
    const GemmEpilogue& e = p.epi;
    const int NB = p.NB;
    uint32_t seg_i = 0;
    SegmentWalk walk(p);
    Segment sg;
    while (walk.next(sg)) {
      const uint32_t acc = seg_i & 1u, aph = (seg_i >> 1) & 1u;
      ++seg_i;
      const int macro = sg.tile / p.n_mchunks, m0 = (sg.tile % p.n_mchunks) * NB;
      const bool contributor = p.splits == 0 && sg.kb0 > 0;
      const bool owner_of_split = p.splits == 0 && sg.kb0 == 0 && sg.kb1 < p.n_kb;
      float* const c_out = e.C != nullptr ? e.C + (size_t)sg.slice * p.slice_stride : nullptr;
      int n_contrib = 0;
      bool presummed = false;
      // spare TMEM columns behind the two accumulator sets hold the sum of the other CTAs' partials
      const uint32_t stash_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(2 * p.acc_cols);
      if (owner_of_split) {
        // the CTAs after this one whose range starts inside this tile each hold one partial of it
        const int tile_end = (sg.tile + 1) * p.n_kb;
        for (int c = blockIdx.x + 1; c < (int)gridDim.x && range_begin(p, c) < tile_end; ++c) ++n_contrib;
        if (eid == 0) {
          for (int i = 1; i <= n_contrib && !*abort_flag; ++i) {
            const unsigned int* f = p.sk_flags + blockIdx.x + i;
            if (ld_acquire(f) != 0u) continue;
            const uint64_t t0 = ptx::global_timer_ns();
            uint32_t polls = 0;
            while (ld_acquire(f) == 0u) {
              if ((++polls & 63u) == 0 && ptx::global_timer_ns() - t0 > p.wait_ns) {
                *abort_flag = 1;
                atomicOr(p.err, 1);
                break;
              }
            }
          }
        }
        ptx::named_bar_sync(1, 128);
        if (*abort_flag) break;
        if (p.stash) {
          // they finished their piece earlier: add them up now, while this CTA's own UMMAs are running
          presummed = true;
          for (int c = 0; c < kHalves * NB; c += 16) {  // column c of the [half][NB] slot layout
            float acc16[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) acc16[i] = 0.f;
            for (int k = 1; k <= n_contrib; ++k) {
              const float* slot = p.sk_scratch + ((size_t)(blockIdx.x + k) * (kHalves * NB) + c) * kTileN + vl;
              float t[16];
#pragma unroll
              for (int i = 0; i < 16; ++i) t[i] = __ldcg(slot + (size_t)i * kTileN);
#pragma unroll
              for (int i = 0; i < 16; ++i) acc16[i] += t[i];
            }
            ptx::tmem_st16(stash_addr + c, acc16);
          }
        }
      }
      if (!ptx::mbar_wait(&tmem_full[acc], aph, abort_flag, p.err, p.wait_ns)) break;
      ptx::tc_fence_after();
#pragma unroll 1  // run-once code: the second half re-uses the instruction lines of the first
      for (int half = 0; half < kHalves; ++half) {
        const int n_tile = macro * kHalves + half;
        if (n_tile * kTileN >= p.N) break;  // second half of the last work tile lies beyond N
        const int n = n_tile * kTileN + vl;
        const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * (uint32_t)p.acc_cols + half * (uint32_t)NB;
        // plain result tiles that lie fully inside C with 16-byte aligned rows take the staged store
        const bool wide_store = c_out != nullptr && !contributor && !e.accumulate && e.part == nullptr &&
                                (e.ldc & 3) == 0 && (n_tile + 1) * kTileN <= p.N &&
                                (reinterpret_cast<uintptr_t>(c_out) & 15u) == 0;
        int n_gather = 0;
        if (e.tok != nullptr && !contributor) {
          // which of the logits the acceptance rule reads (tok[idx] under its parent's and grandparent's
          // rows) fall into this 128-row tile: found once here, served from the staging buffer below
          ptx::named_bar_sync(1, 128);
          if (eid == 0) s_gather_n = 0;
          ptx::named_bar_sync(1, 128);
          for (int idx = eid; idx < e.n_rows; idx += 128) {
            const int ln = e.tok[idx] - n_tile * kTileN;
            if ((unsigned)ln >= (unsigned)kTileN) continue;
            const int b = idx / e.T, j = idx - b * e.T;
            const int pi = e.parent[j];
            if (pi < 0) continue;
            const int gp = e.parent[pi];
            // columns are activation rows relative to this row chunk; rows of other chunks are served by
            // the CTAs that hold those chunks (-1: not here)
            const int n_valid = min(NB, p.M - m0);
            int cp = b * e.T + pi - m0, cg = gp >= 0 ? b * e.T + gp - m0 : -1;
            if ((unsigned)cp >= (unsigned)n_valid) cp = -1;
            if ((unsigned)cg >= (unsigned)n_valid) cg = -1;
            if (cp < 0 && cg < 0) continue;
            const int pos = atomicAdd(&s_gather_n, 1);
            if (pos < kGatherCap) s_gather[pos] = make_int4((ln >> 5) * 33 + (ln & 31), cp, cg, idx);
          }
          ptx::named_bar_sync(1, 128);
          n_gather = s_gather_n;
        }
        // 64 accumulator columns at a time (NB is a multiple of 16, so the last group may be narrower)
        for (int c0 = 0; c0 < NB; c0 += 64) {
          const int n_cols = min(64, NB - c0);
          float v[64];
          if (n_cols == 64) {
            ptx::tmem_ld64(t_addr + c0, v);  // four loads in flight, one wait
          } else {
#pragma unroll
            for (int sub = 0; sub < 4; ++sub)
              if (16 * sub < n_cols) ptx::tmem_ld16(t_addr + c0 + 16 * sub, v + 16 * sub);
          }
          if (p.combine) {  // the remainders' products: NB columns further on
#pragma unroll
            for (int sub = 0; sub < 4; ++sub)
              if (16 * sub < n_cols) {
                float t[16];
                ptx::tmem_ld16(t_addr + NB + c0 + 16 * sub, t);
#pragma unroll
                for (int i = 0; i < 16; ++i) v[16 * sub + i] += t[i];
              }
          }
          if (contributor) {
            // partial of a split tile, [column][weight row]: coalesced over the lanes
            float* slot = p.sk_scratch + (((size_t)blockIdx.x * kHalves + half) * NB + c0) * kTileN + vl;
#pragma unroll
            for (int i = 0; i < 64; ++i)
              if (i < n_cols) slot[(size_t)i * kTileN] = v[i];
            continue;
          }
          if (presummed) {
#pragma unroll
            for (int sub = 0; sub < 4; ++sub)
              if (16 * sub < n_cols) {
                float t[16];
                ptx::tmem_ld16(stash_addr + half * NB + c0 + 16 * sub, t);
#pragma unroll
                for (int i = 0; i < 16; ++i) v[16 * sub + i] += t[i];
              }
          } else {
            for (int k = 1; k <= n_contrib; ++k) {
              const float* slot = p.sk_scratch + (((size_t)(blockIdx.x + k) * kHalves + half) * NB + c0) * kTileN + vl;
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                float t[32];
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (32 * q + i < n_cols) t[i] = __ldcg(slot + (size_t)(32 * q + i) * kTileN);
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (32 * q + i < n_cols) v[32 * q + i] += t[i];
              }
            }
          }
          if (wide_store) {
            // Output rows are contiguous over the weight rows (n), a thread holds one n: staged through shared
            // memory, a warp writes the 128 weight rows of an activation row with one 16-byte store per lane
            // (a quarter of the store instructions of the direct path, each a full 512 bytes).
#pragma unroll
            for (int r = 0; r < 2; ++r) {
              if (r * kStCols >= n_cols) break;
              ptx::named_bar_sync(1, 128);  // the previous round has been read
#pragma unroll
              for (int i = 0; i < kStCols; ++i)
                if (r * kStCols + i < n_cols) st[i * kTileN + vl] = v[r * kStCols + i];
              ptx::named_bar_sync(1, 128);
              const int row0 = m0 + c0 + r * kStCols;
              float* dst = c_out + (size_t)row0 * e.ldc + n_tile * kTileN + 4 * lane;
#pragma unroll
              for (int k = 0; k < kStCols / 4; ++k) {
                const int i = (warp - 2) + 4 * k;
                if (r * kStCols + i < n_cols && row0 + i < p.M)
                  *reinterpret_cast<float4*>(dst + (size_t)i * e.ldc) = *reinterpret_cast<const float4*>(st + i * kTileN + 4 * lane);
              }
            }
          } else if (c_out != nullptr && n < p.N) {
            float* dst = c_out + (size_t)(m0 + c0) * e.ldc + n;
            const int rows = min(n_cols, p.M - (m0 + c0));  // rows of this group that exist
            if (e.accumulate) {
#pragma unroll
              for (int i = 0; i < 64; ++i)
                if (i < rows) dst[(size_t)i * e.ldc] += v[i];
            } else {
#pragma unroll
              for (int i = 0; i < 64; ++i)
                if (i < rows) dst[(size_t)i * e.ldc] = v[i];
            }
          }
          if (e.part != nullptr) {
            // per-(activation row, tile) softmax partials: 32 activation rows per round go through shared
            // memory so that 4 threads see the 128 weight rows of one activation row
#pragma unroll
            for (int r = 0; r < 2; ++r) {
              if (r * kStCols >= n_cols) break;
              const int cs = c0 + r * kStCols;  // first activation row (column) of this round
              ptx::named_bar_sync(1, 128);      // the previous round has been read
#pragma unroll
              for (int i = 0; i < kStCols; ++i)
                if (r * kStCols + i < n_cols) st[i * kStRow + st_wr] = (n < p.N) ? v[r * kStCols + i] : -INFINITY;
              ptx::named_bar_sync(1, 128);
              const float* row = st + st_col * kStRow + st_part * 33;
              float mx = row[0];
#pragma unroll
              for (int i = 1; i < 32; ++i) mx = fmaxf(mx, row[i]);
              float sum = 0.f;
              if (mx != -INFINITY) {
#pragma unroll
                for (int i = 0; i < 32; ++i) sum += __expf(row[i] - mx);
              }
#pragma unroll
              for (int o = 1; o < 4; o <<= 1) {
                const float mo = __shfl_xor_sync(0xffffffffu, mx, o), so = __shfl_xor_sync(0xffffffffu, sum, o);
                combine_ms(mx, sum, mo, so);
              }
              const int m = m0 + cs + st_col;
              if (st_part == 0 && r * kStCols + st_col < n_cols && m < p.M)
                e.part[(size_t)m * e.part_ld + n_tile] = make_float2(mx, sum);
              if (n_gather <= kGatherCap) {
                for (int i = eid; i < n_gather; i += 128) {
                  const int4 g = s_gather[i];
                  int col = g.y - cs;
                  if (g.y >= 0 && (unsigned)col < (unsigned)kStCols) e.cand_parent[g.w] = st[col * kStRow + g.x];
                  col = g.z - cs;
                  if (g.z >= 0 && (unsigned)col < (unsigned)kStCols) e.cand_gparent[g.w] = st[col * kStRow + g.x];
                }
              } else {
                // more hits in one tile than the list holds: scan the tokens again in every round
                for (int idx = eid; idx < e.n_rows; idx += 128) {
                  const int ln = e.tok[idx] - n_tile * kTileN;
                  if ((unsigned)ln >= (unsigned)kTileN) continue;
                  const int b = idx / e.T, j = idx - b * e.T;
                  const int pi = e.parent[j];
                  if (pi < 0) continue;
                  const int at = (ln >> 5) * 33 + (ln & 31);
                  const int n_valid = min(NB, p.M - m0);
                  int row = b * e.T + pi - m0, col = row - cs;
                  if ((unsigned)row < (unsigned)n_valid && (unsigned)col < (unsigned)kStCols)
                    e.cand_parent[idx] = st[col * kStRow + at];
                  const int gp = e.parent[pi];
                  if (gp < 0) continue;
                  row = b * e.T + gp - m0;
                  col = row - cs;
                  if ((unsigned)row < (unsigned)n_valid && (unsigned)col < (unsigned)kStCols)
                    e.cand_gparent[idx] = st[col * kStRow + at];
                }
              }
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

int64_t gemm_tc_scratch_floats(int sm_count) { return (int64_t)sm_count * 2 * 128 * kTileN; }

// Accumulators (128 weight rows each) per work tile.  With more than 64 activation rows a stage holds
// more activation bytes (high part and remainder, re-read from the L2 for every tile) than weight bytes,
// and what an SM can take in per second, not HBM, bounds the weight stream: a 256-row tile feeds two
// accumulators from one activation stage and halves that overhead.  Only the sliced mode does this (no
// hand-off between CTAs, so TMEM need not hold a third accumulator set, and its matrices have many tiles).
static int pick_halves(int NB, bool sliced) { return (sliced && NB > 64 && 4 * NB <= 512) ? 2 : 1; }

SliceMap gemm_tc_balanced_map(const cascade_ctx* ctx, int M, int N, int K) {
  SliceMap map;
  const OperandLayout lay = operand_layout(M, K);
  if (lay.n_chunks != 1 || K % kSpan != 0) return map;
  const int halves = pick_halves(lay.NB, true);
  const int n_tiles = cascade_detail::ceil_div(N, halves * kTileN);
  const int n_kb = K / kSpan;  // sliced launches with more than 64 rows carry one span per stage
  if (halves != 2) return map;
  const long long units = (long long)n_tiles * n_kb;
  const int grid = units < ctx->sm_count ? (int)units : ctx->sm_count;
  map.q = (int)(units / grid);
  map.r = (int)(units % grid);
  map.n_kb = n_kb;
  map.tile_cols = halves * kTileN;
  int most = 1;
  for (int t = 0; t < n_tiles; ++t) {
    auto cta_of = [&](long long u) {
      const long long big = (long long)map.r * (map.q + 1);
      return (int)(u < big ? u / (map.q + 1) : map.r + (u - big) / map.q);
    };
    const int pieces = cta_of((long long)(t + 1) * n_kb - 1) - cta_of((long long)t * n_kb) + 1;
    if (pieces > most) most = pieces;
  }
  map.n_slices = most;
  map.balanced = 1;
  return map;
}

int gemm_tc_pick_splits(int sm_count, int M, int N, int K, int max_splits) {
  const OperandLayout lay = operand_layout(M, K);
  const int halves = pick_halves(lay.NB, true);
  const int n_tiles = cascade_detail::ceil_div(N, halves * kTileN) * lay.n_chunks;
  const int n_kb = cascade_detail::ceil_div(K, kSpan);
  const long long kb_cost = halves * 16 + lay.NB / 4;  // KB an SM takes in per K block: weights + activation pair
  int best = 1;
  long long best_cost = -1;
  // a stage may carry two 64-wide K spans, and every slice needs at least one stage
  for (int s = 1; s <= max_splits && s <= cascade_detail::ceil_div(K, 2 * kSpan); ++s) {
    // time ~ rounds x K blocks per item, plus writing and re-reading one output matrix per slice at about
    // the same rate
    const long long rounds = cascade_detail::ceil_div(n_tiles * s, sm_count);
    const long long cost = rounds * cascade_detail::ceil_div(n_kb, s) * kb_cost + (long long)s * M * N / 6250;
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

int launch_gemm_tc(cascade_ctx* ctx, const __nv_bfloat16* W, int N, int K, const __nv_bfloat16* A, int M,
                   const GemmEpilogue& epi, int kernel_id, cudaStream_t s) {
  if (K % kSpan != 0 || M < 1 || N < 1) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  if (epi.part != nullptr && epi.part_ld < cascade_detail::ceil_div(N, kTileN)) return CASCADE_ERR_INVALID_ARG;
  if (epi.splits < 0 || (epi.splits > 1 && (epi.part != nullptr || epi.accumulate || epi.C == nullptr)))
    return CASCADE_ERR_INVALID_ARG;
  if (epi.tok != nullptr && (epi.part == nullptr || epi.parent == nullptr || epi.cand_parent == nullptr ||
                             epi.cand_gparent == nullptr || epi.T < 1))
    return CASCADE_ERR_INVALID_ARG;
  GemmArgs a;
  a.M = M;
  a.N = N;
  const OperandLayout lay = operand_layout(M, K);
  a.n_mchunks = lay.n_chunks;
  a.NB = lay.NB;
  a.A = A;
  a.a_chunk_elems = (long long)lay.n_kb * 2 * lay.NB * kSpan;
  a.epi = epi;
  a.sk_scratch = ctx->gemm_scratch;
  a.sk_flags = ctx->gemm_flags;
  a.err = ctx->dev_error;
  a.wait_ns = ctx->wait_limit_ns;
  // A stage carries 32 KB of weights where three such stages fit (two K spans of a 128-row tile): the
  // round trip of the single producer / issue threads per stage limits the stream below that.  With
  // many activation rows the activation part of a stage is too large for that: one span per stage.
  // (With at most 64 activation rows, 256-row tiles measured no faster on the stream and split the LM
  // head of a 16384-token vocabulary over too few tiles.)
  const int halves = pick_halves(a.NB, epi.splits > 0);
  // static shared memory (general epilogue: 19 KB; eight-warp epilogue: two 16 KB staging buffers) + alignment slack
  const bool lean_cfg = epi.splits >= 1 && epi.part == nullptr && !epi.accumulate && epi.C != nullptr && epi.tok == nullptr;
  const int budget = 227 * 1024 - (lean_cfg ? 33 : 20) * 1024 - 1024;
  const int span_bytes = halves * kTileWBytes + 2 * a.NB * kSpan * 2;
  const int spans = (K % (2 * kSpan) == 0 && budget / (2 * span_bytes) >= 3) ? 2 : 1;
  const int stage_bytes = spans * span_bytes;
  a.stages = budget / stage_bytes;
  if (a.stages > kMaxStages) a.stages = kMaxStages;
  if (a.stages < 2) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  a.n_kb = cascade_detail::ceil_div(K, kSpan * spans);
  if (epi.splits > a.n_kb) return CASCADE_ERR_INVALID_ARG;  // a slice without a K block would have no result
  const int n_tiles = cascade_detail::ceil_div(N, halves * kTileN) * a.n_mchunks;
  a.units = (long long)n_tiles * a.n_kb;
  a.n_tiles = n_tiles;
  a.splits = epi.splits;
  a.balanced = epi.balanced;
  if (epi.balanced && (epi.splits < 1 || a.n_mchunks != 1 || epi.part != nullptr || epi.accumulate || epi.C == nullptr))
    return CASCADE_ERR_INVALID_ARG;
  a.slice_stride = epi.slice_stride;
  // one UMMA over both operand parts where 64 or fewer activation rows leave the room in TMEM
  a.combine = (halves == 1 && a.NB <= 64) ? 1 : 0;
  a.acc_cols = a.combine ? 2 * a.NB : halves * a.NB;
  a.stash = epi.splits == 0 && 2 * a.acc_cols + halves * a.NB <= 512;
  a.tmem_cols = 32;
  while (a.tmem_cols < 2 * a.acc_cols + (a.stash ? halves * a.NB : 0)) a.tmem_cols *= 2;
  const CUtensorMap* tw =
      get_tmap_2d_bf16(ctx, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, (uint32_t)(halves * kTileN), kSpan);
  if (tw == nullptr) return CASCADE_ERR_CUDA;
  const int smem = a.stages * stage_bytes + 1024;
  if (halves == 2 && spans == 2) return CASCADE_ERR_UNSUPPORTED_SHAPE;  // cannot happen: such stages do not fit
  // the sliced projections (plain store of every piece into its own matrix) take the eight-warp epilogue
  const bool lean = epi.splits >= 1 && epi.part == nullptr && !epi.accumulate && epi.C != nullptr && epi.tok == nullptr;
  auto kern = lean ? (halves == 2 ? k_gemm_tc<2, 1, true> : (spans == 2 ? k_gemm_tc<1, 2, true> : k_gemm_tc<1, 1, true>))
                   : (halves == 2 ? k_gemm_tc<2, 1, false> : (spans == 2 ? k_gemm_tc<1, 2, false> : k_gemm_tc<1, 1, false>));
  int* configured_smem = ctx->gemm_smem_configured;
  const int kern_i = (halves == 2 ? 2 : spans - 1) + (lean ? 3 : 0);
  if (smem > configured_smem[kern_i]) {
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured_smem[kern_i] = smem;
  }
  long long grid = (epi.splits > 0 && !epi.balanced) ? (long long)n_tiles * epi.splits : a.units;
  if (grid > ctx->sm_count) grid = ctx->sm_count;
  // the kernel's work assignment is 32-bit
  if (a.units >= (1ll << 30) || (long long)a.n_kb * (epi.splits + 1) >= (1ll << 30) || (long long)n_tiles * (epi.splits + 1) >= (1ll << 30))
    return CASCADE_ERR_UNSUPPORTED_SHAPE;
  a.unit_q = (int)(a.units / grid);
  a.unit_r = (int)(a.units % grid);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(lean ? kLeanThreads : kThreads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: the split-tile hand-off waits on peers
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = epi.splits == 0 ? 1 : 0;
  {
    KernelScope ks(ctx, kernel_id, s);
    CASCADE_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, *tw, a));
  }
  return CASCADE_OK;
}

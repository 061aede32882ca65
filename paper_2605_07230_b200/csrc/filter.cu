// Top-k / nucleus truncation of the target distribution, in place on the logits (the sampling settings of the
// paper's experiments, Appendix D.1: temperature 1, top-p 1.0, top-k 2000).  A dropped token's logit becomes
// -inf, so every later consumer (row statistics, the acceptance rule, the bonus-token draw) sees probability
// zero for it and the kept tokens renormalised.
//
//   top-k : keep the tokens whose logit is >= the k-th largest logit of the row (ties stay together);
//   top-p : on the distribution renormalised over what top-k kept, keep a token iff the probability of the
//           tokens with a strictly larger logit is < p.
//
// One CTA per row.  Both thresholds are found exactly by a radix descent over an order-preserving 32-bit
// image of the logits, 8 bits per pass from the top: a histogram of the current digit over the elements that
// match the digits fixed so far, then the bucket where the running total (from the largest digit down)
// reaches the target.  For top-k the histogram counts elements; for top-p it adds exp(l - max) as 40-bit
// fixed point, so the sums do not depend on the order of the additions and the result is reproducible.
// The digits of a row crowd into a few buckets, so the histograms are built without atomics: one per warp,
// the lanes that hit the same bucket found with match.any and served by one of them.
#include "cascade_internal.h"

namespace {

constexpr int kFilterThreads = 1024;
constexpr int kWarps = kFilterThreads / 32;
constexpr int kRegItems = 16;                 // rows of up to 16384 logits stay in registers between the passes
constexpr float kFixedOne = 1099511627776.f;  // 2^40

__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // larger float <=> larger key; -inf is the smallest
}
__device__ __forceinline__ float key_value(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Shared memory: a histogram per warp (no two warps touch the same counter; inside a warp the lanes that hit the
// same bucket are found with match.any and one of them adds for all), then the totals and the scan's result.
struct FilterShared {
  unsigned long long total[256];
  unsigned long long red[kWarps];
  float redf[kWarps];
  uint32_t digit;
  unsigned long long above;
};

// The row's keys: in registers (kReg) or re-read from memory every pass.
template <bool kReg>
struct RowKeys {
  const float* row;
  int V;
  uint32_t reg[kReg ? kRegItems : 1];
  __device__ __forceinline__ void load() {
    if constexpr (kReg) {
#pragma unroll
      for (int t = 0; t < kRegItems; ++t) {
        const int i = t * kFilterThreads + threadIdx.x;
        reg[t] = i < V ? order_key(__ldcg(row + i)) : 0u;  // 0 is below every real key (even -inf's)
      }
    }
  }
  // f(key, valid) for every element slot of this thread; all lanes of a warp make the same number of calls
  template <typename F>
  __device__ __forceinline__ void each(F f) const {
    if constexpr (kReg) {
#pragma unroll
      for (int t = 0; t < kRegItems; ++t) f(reg[t], t * kFilterThreads + (int)threadIdx.x < V);
    } else if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(row) & 15u) == 0) {
      // 16 bytes per lane, two loads in flight
      const float4* row4 = reinterpret_cast<const float4*>(row);
      const int n4 = V / 4, n = (n4 + kFilterThreads - 1) / kFilterThreads;
      for (int t = 0; t < n; t += 2) {
        const int i0 = t * kFilterThreads + threadIdx.x, i1 = i0 + kFilterThreads;
        const bool v0 = i0 < n4, v1 = t + 1 < n && i1 < n4;
        const float4 a = v0 ? __ldcg(row4 + i0) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 b = v1 ? __ldcg(row4 + i1) : make_float4(0.f, 0.f, 0.f, 0.f);
        f(v0 ? order_key(a.x) : 0u, v0);
        f(v0 ? order_key(a.y) : 0u, v0);
        f(v0 ? order_key(a.z) : 0u, v0);
        f(v0 ? order_key(a.w) : 0u, v0);
        if (t + 1 < n) {
          f(v1 ? order_key(b.x) : 0u, v1);
          f(v1 ? order_key(b.y) : 0u, v1);
          f(v1 ? order_key(b.z) : 0u, v1);
          f(v1 ? order_key(b.w) : 0u, v1);
        }
      }
    } else {
      const int n = (V + kFilterThreads - 1) / kFilterThreads;
      for (int t = 0; t < n; ++t) {
        const int i = t * kFilterThreads + threadIdx.x;
        const bool valid = i < V;
        f(valid ? order_key(__ldcg(row + i)) : 0u, valid);
      }
    }
  }
};

template <bool kMass>
__device__ __forceinline__ unsigned long long weight_of(uint32_t key, float m) {
  return kMass ? __float2ull_rz(expf(key_value(key) - m) * kFixedOne) : 1ull;
}

__device__ __forceinline__ unsigned long long block_total(unsigned long long acc, FilterShared& sh) {
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = acc;
  __syncthreads();
  unsigned long long t = 0;
  for (int i = 0; i < kWarps; ++i) t += sh.red[i];
  return t;
}

// The key x with W(> x) < target <= W(>= x), W = weight of the elements with key >= floor_key (1 each, or
// exp(l - m) in fixed point).  hist: [kWarps][256] in dynamic shared memory.
template <bool kMass, bool kReg>
__device__ uint32_t descend(const RowKeys<kReg>& keys, float m, uint32_t floor_key, unsigned long long target,
                            FilterShared& sh, unsigned long long* hist) {
  uint32_t prefix = 0;
  unsigned long long above = 0;  // weight of the keys above the digits fixed so far
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long* my_hist = hist + warp * 256;
  unsigned int* my_count = reinterpret_cast<unsigned int*>(hist) + warp * 256;  // counts: 32-bit, same memory
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = lane; i < 256; i += 32) {
      if constexpr (kMass)
        my_hist[i] = 0ull;
      else
        my_count[i] = 0u;
    }
    __syncwarp();
    keys.each([&](uint32_t key, bool valid) {
      const bool in = valid && key >= floor_key && (shift == 24 || (key >> (shift + 8)) == (prefix >> (shift + 8)));
      if constexpr (!kMass) {
        // counts: the shared-memory atomic unit resolves lanes on one counter quickly enough
        if (in) atomicAdd(&my_count[(key >> shift) & 255u], 1u);
        return;
      }
      const uint32_t d = in ? ((key >> shift) & 255u) : 0xffffffffu;
      const uint32_t peers = __match_any_sync(0xffffffffu, d);
      unsigned long long w;
      if constexpr (kMass) {
        // integer sums (the order does not matter); weights are below 2^40, added in two 20-bit pieces
        w = 0;
        if (in) {
          const unsigned long long mine = weight_of<true>(key, m);
          const unsigned int lo = __reduce_add_sync(peers, (unsigned int)(mine & 0xfffffull));
          const unsigned int hi = __reduce_add_sync(peers, (unsigned int)(mine >> 20));
          w = ((unsigned long long)hi << 20) + lo;
        }
      } else {
        w = (unsigned long long)__popc(peers);
      }
      if (in && lane == __ffs(peers) - 1) my_hist[d] += w;
      __syncwarp();
    });
    __syncthreads();
    if (threadIdx.x < 256) {
      unsigned long long t = 0;
      if constexpr (kMass) {
        for (int c = 0; c < kWarps; ++c) t += hist[c * 256 + threadIdx.x];
      } else {
        for (int c = 0; c < kWarps; ++c) t += reinterpret_cast<const unsigned int*>(hist)[c * 256 + threadIdx.x];
      }
      sh.total[threadIdx.x] = t;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      // lane L owns the buckets 255 - 8L ... 248 - 8L, largest digit first
      unsigned long long loc[8], sum = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        loc[i] = sh.total[255 - 8 * lane - i];
        sum += loc[i];
      }
      unsigned long long inc = sum;
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const unsigned long long exc = inc - sum;
      const bool mine = above + exc < target && target <= above + inc;
      const uint32_t who = __ballot_sync(0xffffffffu, mine);
      if (who == 0u) {
        if (lane == 0) {  // the target lies beyond everything left: the lowest digit keeps it all
          sh.digit = 0u;
          sh.above = above;
        }
      } else if (mine) {
        unsigned long long run = above + exc;
        uint32_t d = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run + loc[i] >= target) {
            d = 255u - 8u * lane - i;
            break;
          }
          run += loc[i];
        }
        sh.digit = d;
        sh.above = run;
      }
    }
    __syncthreads();
    prefix |= sh.digit << shift;
    above = sh.above;
  }
  return prefix;
}

template <bool kReg>
__global__ void __launch_bounds__(kFilterThreads) k_filter_logits(float* __restrict__ logits, int V, int top_k,
                                                                  float top_p, int32_t* __restrict__ kept_count) {
  extern __shared__ unsigned long long hist[];  // [kWarps][256]
  __shared__ FilterShared sh;
  float* row = logits + (size_t)blockIdx.x * V;
  RowKeys<kReg> keys;
  keys.row = row;
  keys.V = V;
  keys.load();
  // row maximum: only the nucleus needs it (its weights are exp(l - max))
  float m = 0.f;
  if (top_p < 1.f) {
    uint32_t mk = 0;
    keys.each([&](uint32_t key, bool valid) { mk = valid ? max(mk, key) : mk; });
    for (int o = 16; o > 0; o >>= 1) mk = max(mk, __shfl_xor_sync(0xffffffffu, mk, o));
    if ((threadIdx.x & 31) == 0) sh.redf[threadIdx.x >> 5] = __uint_as_float(mk);
    __syncthreads();
    for (int i = 0; i < kWarps; ++i) mk = max(mk, __float_as_uint(sh.redf[i]));
    m = key_value(mk);
  }

  uint32_t floor_key = 1u;  // every real key (0 marks an empty slot)
  if (top_k > 0 && top_k < V) floor_key = descend<false, kReg>(keys, m, floor_key, (unsigned long long)top_k, sh, hist);
  if (top_p < 1.f) {
    unsigned long long acc = 0;
    keys.each([&](uint32_t key, bool valid) {
      if (valid && key >= floor_key) acc += weight_of<true>(key, m);
    });
    const unsigned long long Z = block_total(acc, sh);
    unsigned long long target = (unsigned long long)((double)top_p * (double)Z);
    if (target < 1ull) target = 1ull;
    const uint32_t nucleus_key = descend<true, kReg>(keys, m, floor_key, target, sh, hist);
    floor_key = max(floor_key, nucleus_key);
  }
  unsigned long long kept = 0;
  if constexpr (kReg) {
#pragma unroll
    for (int t = 0; t < kRegItems; ++t) {
      const int i = t * kFilterThreads + threadIdx.x;
      if (i < V) {
        if (keys.reg[t] >= floor_key)
          ++kept;
        else
          row[i] = -INFINITY;
      }
    }
  } else {
    for (int i = threadIdx.x; i < V; i += kFilterThreads) {
      if (order_key(__ldcg(row + i)) >= floor_key)
        ++kept;
      else
        row[i] = -INFINITY;
    }
  }
  if (kept_count != nullptr) {
    const unsigned long long t = block_total(kept, sh);
    if (threadIdx.x == 0) kept_count[blockIdx.x] = (int32_t)t;
  }
}

}  // namespace

int launch_filter_logits(cascade_ctx* ctx, float* logits, int n_rows, int top_k, float top_p, int32_t* kept_count,
                         cudaStream_t s) {
  const size_t smem = (size_t)kWarps * 256 * sizeof(unsigned long long);  // 64 KB of per-warp histograms
  const bool in_regs = ctx->shape.V <= kRegItems * kFilterThreads;
  bool& configured = ctx->filter_configured;
  if (!configured) {
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(k_filter_logits<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(k_filter_logits<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = true;
  }
  {
    KernelScope ks(ctx, K_FILTER_LOGITS, s);
    if (in_regs)
      k_filter_logits<true><<<n_rows, kFilterThreads, smem, s>>>(logits, ctx->shape.V, top_k, top_p, kept_count);
    else
      k_filter_logits<false><<<n_rows, kFilterThreads, smem, s>>>(logits, ctx->shape.V, top_k, top_p, kept_count);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

extern "C" int cascade_filter_logits(cascade_ctx* ctx, float* logits, int32_t n_rows, int32_t top_k, float top_p,
                                     int32_t* kept_count, void* stream) {
  if (ctx == nullptr || logits == nullptr) return CASCADE_ERR_INVALID_ARG;
  if (n_rows < 1 || top_k < 0 || !(top_p > 0.f) || top_p > 1.f) return CASCADE_ERR_INVALID_ARG;  // also rejects NaN
  ctx->launches = 0;
  if ((top_k == 0 || top_k >= ctx->shape.V) && top_p >= 1.f && kept_count == nullptr) return CASCADE_OK;  // nothing to do
  return launch_filter_logits(ctx, logits, n_rows, top_k, top_p, kept_count, static_cast<cudaStream_t>(stream));
}

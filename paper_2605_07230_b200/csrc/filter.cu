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
#include "cascade_internal.h"

namespace {

constexpr int kFilterThreads = 1024;
constexpr int kCopies = 8;  // histogram copies (lane mod 8): the digits of a row crowd into few buckets
constexpr float kFixedOne = 1099511627776.f;  // 2^40

__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // larger float <=> larger key; -inf is the smallest
}

struct FilterShared {
  unsigned long long hist[kCopies][256];
  unsigned long long red[kFilterThreads / 32];
  float redf[kFilterThreads / 32];
  uint32_t digit;
  unsigned long long above;
};

// Weight of the row's elements with key >= floor_key, summed over the whole row.
template <bool kMass>
__device__ unsigned long long total_weight(const float* row, int V, float m, uint32_t floor_key, FilterShared& sh) {
  unsigned long long acc = 0;
  for (int i = threadIdx.x; i < V; i += kFilterThreads) {
    const float x = __ldcg(row + i);
    if (order_key(x) >= floor_key) acc += kMass ? __float2ull_rz(expf(x - m) * kFixedOne) : 1ull;
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = acc;
  __syncthreads();
  unsigned long long t = 0;
  for (int i = 0; i < kFilterThreads / 32; ++i) t += sh.red[i];
  return t;
}

// The key x with W(> x) < target <= W(>= x), W = weight of the elements with key >= floor_key.
template <bool kMass>
__device__ uint32_t descend(const float* row, int V, float m, uint32_t floor_key, unsigned long long target,
                            FilterShared& sh) {
  uint32_t prefix = 0;
  unsigned long long above = 0;  // weight of the keys above the digits fixed so far
  const int lane = threadIdx.x & 31;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < kCopies * 256; i += kFilterThreads) (&sh.hist[0][0])[i] = 0ull;
    __syncthreads();
    for (int i = threadIdx.x; i < V; i += kFilterThreads) {
      const float x = __ldcg(row + i);
      const uint32_t key = order_key(x);
      if (key < floor_key) continue;
      if (shift < 24 && (key >> (shift + 8)) != (prefix >> (shift + 8))) continue;
      const unsigned long long w = kMass ? __float2ull_rz(expf(x - m) * kFixedOne) : 1ull;
      atomicAdd(&sh.hist[lane & (kCopies - 1)][(key >> shift) & 255u], w);
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      // lane L owns the buckets 255 - 8L ... 248 - 8L, largest digit first
      unsigned long long loc[8], sum = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        unsigned long long v = 0;
        for (int c = 0; c < kCopies; ++c) v += sh.hist[c][255 - 8 * lane - i];
        loc[i] = v;
        sum += v;
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
    __syncthreads();
  }
  return prefix;
}

__global__ void __launch_bounds__(kFilterThreads) k_filter_logits(float* __restrict__ logits, int V, int top_k,
                                                                  float top_p, int32_t* __restrict__ kept_count) {
  __shared__ FilterShared sh;
  float* row = logits + (size_t)blockIdx.x * V;
  // row maximum (the nucleus weights are exp(l - max))
  float m = -INFINITY;
  for (int i = threadIdx.x; i < V; i += kFilterThreads) m = fmaxf(m, __ldcg(row + i));
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) sh.redf[threadIdx.x >> 5] = m;
  __syncthreads();
  for (int i = 0; i < kFilterThreads / 32; ++i) m = fmaxf(m, sh.redf[i]);
  __syncthreads();

  uint32_t floor_key = 0;
  if (top_k > 0 && top_k < V) floor_key = descend<false>(row, V, m, 0u, (unsigned long long)top_k, sh);
  if (top_p < 1.f) {
    const unsigned long long Z = total_weight<true>(row, V, m, floor_key, sh);
    unsigned long long target = (unsigned long long)((double)top_p * (double)Z);
    if (target < 1ull) target = 1ull;
    const uint32_t nucleus_key = descend<true>(row, V, m, floor_key, target, sh);
    floor_key = max(floor_key, nucleus_key);
  }
  int kept = 0;
  for (int i = threadIdx.x; i < V; i += kFilterThreads) {
    const float x = __ldcg(row + i);
    if (order_key(x) >= floor_key)
      ++kept;
    else
      row[i] = -INFINITY;
  }
  if (kept_count != nullptr) {
    __syncthreads();  // the reduction buffer is free
    unsigned long long acc = (unsigned long long)kept;
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned long long t = 0;
      for (int i = 0; i < kFilterThreads / 32; ++i) t += sh.red[i];
      kept_count[blockIdx.x] = (int32_t)t;
    }
  }
}

}  // namespace

extern "C" int cascade_filter_logits(cascade_ctx* ctx, float* logits, int32_t n_rows, int32_t top_k, float top_p,
                                     int32_t* kept_count, void* stream) {
  if (ctx == nullptr || logits == nullptr) return CASCADE_ERR_INVALID_ARG;
  if (n_rows < 1 || top_k < 0 || !(top_p > 0.f) || top_p > 1.f) return CASCADE_ERR_INVALID_ARG;  // also rejects NaN
  ctx->launches = 0;
  if ((top_k == 0 || top_k >= ctx->shape.V) && top_p >= 1.f && kept_count == nullptr) return CASCADE_OK;  // nothing to do
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    KernelScope ks(ctx, K_FILTER_LOGITS, s);
    k_filter_logits<<<n_rows, kFilterThreads, 0, s>>>(logits, ctx->shape.V, top_k, top_p, kept_count);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

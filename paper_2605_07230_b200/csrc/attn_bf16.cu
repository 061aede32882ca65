// Tree-masked attention of the draft-tree rows over the prefix KV cache plus their tree ancestors
// (Section 3 of the paper: the whole draft tree is verified by the target in one parallel pass), bf16,
// for sm_100a.  Memory-bound decode-style kernel: every key/value row is streamed from HBM once per
// (CFG row, head) and shared by all tree rows.
//
// One CTA per (KV split, query head x row block, CFG row); the splits of one unit form a thread-block cluster.  What
// follows describes row blocks of 64 tree rows (trees of up to 64 rows); larger trees take the wide form, row blocks
// of 128 (see the kernel's template parameter).
//   * two producer threads stream 128-key K tiles and V tiles (bf16, 128-byte swizzle) through their own
//     rings (2 and 3 slots) and ask the L2 for the tiles after those;
//   * one thread issues the tensor-core work: S = Q K^T (UMMA 128x128x128) into one of two TMEM score
//     buffers, and O += P V into the TMEM output accumulator;
//   * eight softmax warps own the 128 TMEM lanes twice over.  A row block holds at most 64 tree rows and the Q
//     tile is loaded twice (UMMA rows r and r+64 are the same tree row), so that lanes 0-63 can take keys 0-63 of
//     every tile and lanes 64-127 keys 64-127; the two warps that share a lane quadrant split those 64 keys again.
//     Four threads therefore work on one tree row, 32 keys each;
//   * the probabilities go to the tensor core as a bf16 pair: the value rounded to bf16 in P rows 0-63 and what the
//     rounding dropped (again bf16) in P rows 64-127, so that one UMMA over the 128-row P tile accumulates
//     sum(p_hi v) in output rows 0-63 and sum(p_lo v) in rows 64-127.  Their sum carries 16 significant bits of
//     every weight instead of 8; a bf16-rounded P alone limits the output to about 2e-3, which one decoder layer
//     turns into 2e-2 on the logits;
//   * online softmax in the exp2 domain with ONE reference per tree row, shared by its four threads and raised
//     lazily: weights are 2^(s - ref), and ref only has to stay within a few dozen binary orders of the true
//     maximum for fp32 accumulators (the final division removes it).  The first tile fixes ref by an exchange
//     through shared memory behind one barrier; later a thread that meets a score more than 2^8 above ref posts
//     it, and all four threads of the row adopt it at the start of the NEXT tile, behind the wait for the
//     previous output product, where everybody is known to have seen the post.  The rows already accumulated in
//     TMEM are then rescaled in place (tcgen05.ld/st); this is rare;
//   * keys of the prefix are visible to every row up to prefix_len; keys of the tree are visible to
//     row j iff bit i of the packed ancestor-or-self mask of j is set.
// With several KV splits every CTA leaves its un-normalised partial (output rows, reference, sum) in its own shared
// memory; the rank-0 CTA of the cluster reads the others' through distributed shared memory, merges in split
// order and writes the rows.  No global scratch, no counters.
// Every mbarrier wait is bounded (error word + normal teardown on expiry); the cluster barriers at the start and
// the end are reached by every thread on every path.
#include "cascade_internal.h"
#include "operand.cuh"
#include "ptx.cuh"
#include "tmap.h"

namespace {

constexpr int kD = 128;
constexpr int kTileKeys = 128;
constexpr int kRowsNarrow = 64;   // rows per block with the duplicated Q tile (trees of up to 64 rows)
constexpr int kRowsWide = 128;    // rows per block without duplication (larger trees)
constexpr int kSoftmaxThreads = 256;  // warps 0-7
constexpr int kThreads = 320;         // + warp 8: TMA, warp 9: UMMA issue + TMEM alloc
constexpr int kQBytes = 128 * kD * 2;        // 32 KB: two 64-wide halves of [128 rows][64] bf16
constexpr int kPBytes = 128 * kTileKeys * 2;  // 32 KB
constexpr int kKVTileBytes = kTileKeys * kD * 2;  // 32 KB for K, same for V
constexpr int kKSlots = 2;     // K tiles in shared memory (a slot is free again once S = Q K^T has read it)
constexpr int kVSlotsNarrow = 3, kVSlotsWide = 2;  // V tiles in shared memory (free once O += P V has read it); the
                               // wide form holds two P tiles (values and remainders) and has room for two
constexpr int kPrefetch = 0;   // with a ring of n slots, tile i + n - 1 + kPrefetch is requested into the L2 when tile i is
                               // loaded (measured 0..3 on 20-tile rows: deeper requests delay the loads that are waited for)
constexpr int kSmemBytes = kQBytes + kPBytes + (kKSlots + kVSlotsNarrow) * kKVTileBytes + 1024;
static_assert(kQBytes + 2 * kPBytes + (kKSlots + kVSlotsWide) * kKVTileBytes + 1024 == kSmemBytes, "both forms use the same shared memory");
constexpr int kXRow = 132;     // floats per row of the partial-result buffer: 128 outputs, reference, sum, 2 pad
constexpr int kMaxSplits = 4;
constexpr float kLazy = 8.f;   // the reference is raised when a score exceeds it by more than this (log2 units)

// 8 consecutive outputs of (row m of R*T, column col of Hq*D): bf16 row-major, or -- for the output
// projection that follows inside a decoder layer -- the bf16 pair (value, what the rounding dropped) in the
// GEMM's staged operand layout
template <typename Args>
__device__ __forceinline__ void store8(const Args& p, int m, int col, int row_len, const float* v) {
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    hi[k] = ptx::pack_bf16x2(v[2 * k], v[2 * k + 1]);
    lo[k] = ptx::pack_bf16x2(v[2 * k] - __uint_as_float(hi[k] << 16), v[2 * k + 1] - __uint_as_float(hi[k] & 0xffff0000u));
  }
  if (p.out_as_operand) {
    *reinterpret_cast<uint4*>(p.out + operand_index(p.out_lay, m, col, 0)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(p.out + operand_index(p.out_lay, m, col, 1)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  } else {
    *reinterpret_cast<uint4*>(p.out + (size_t)m * row_len + col) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
  }
}

struct AttnArgs {
  int T, Hq, Hkv, splits, n_rb, prefix_cap;
  const int32_t* prefix_len;
  const uint64_t* anc;
  __nv_bfloat16* out;
  int out_as_operand;     // 1: `out` receives the (R*T x Hq*D) matrix as a GEMM operand (bf16 pair, staged layout)
  OperandLayout out_lay;
  float c;  // softmax_scale * log2(e)
  int* err;
  unsigned long long wait_ns;  // limit of every bounded wait in the kernel
};

// order-preserving image of a float in a signed int (for atomicMax on shared memory)
__device__ __forceinline__ int float_key(float f) {
  const int b = __float_as_int(f);
  return b >= 0 ? b : b ^ 0x7fffffff;
}
__device__ __forceinline__ float key_float(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7fffffff); }

// kWide = false: row blocks of 64 tree rows, Q tile loaded twice, four threads per row, one P tile whose rows 0-63 /
// 64-127 hold the values / the remainders (one output product per key tile).  kWide = true (trees of more than 64
// rows): row blocks of 128, two threads per row with 64 keys each, two P tiles and two output products per key tile
// into the same accumulator -- one pass over the keys for up to 128 rows instead of one per 64.
template <bool kWide>
__global__ void __launch_bounds__(kThreads, 1)
k_tree_attn_bf16(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kp,
                 const __grid_constant__ CUtensorMap tm_vp, const __grid_constant__ CUtensorMap tm_kt,
                 const __grid_constant__ CUtensorMap tm_vt, const AttnArgs p) {
  constexpr int kRowsPerBlock = kWide ? kRowsWide : kRowsNarrow;
  constexpr int kVSlots = kWide ? kVSlotsWide : kVSlotsNarrow;
  constexpr int kKeysPerThread = kWide ? 64 : 32;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t q_full, k_full[kKSlots], k_empty[kKSlots], v_full[kVSlots], v_empty[kVSlots],
      s_full[2], s_empty[2], p_full, o_full, ref_ready, peers_ready;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  __shared__ int s_rowmax[3][kRowsPerBlock];   // posted row maxima, one buffer per tile index mod 3

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t q_addr = smem_base, p_addr = smem_base + kQBytes, k_ring = p_addr + (kWide ? 2 : 1) * kPBytes,
                 v_ring = k_ring + kKSlots * kKVTileBytes;

  if (threadIdx.x == kSoftmaxThreads) {  // the TMA warp's first loads should not wait for their descriptors
    ptx::prefetch_tmap(&tm_q);
    ptx::prefetch_tmap(&tm_kp);
    ptx::prefetch_tmap(&tm_vp);
    ptx::prefetch_tmap(&tm_kt);
    ptx::prefetch_tmap(&tm_vt);
  }
  const int split = blockIdx.x, head = blockIdx.y / p.n_rb, rb = blockIdx.y % p.n_rb, r = blockIdx.z;
  const int hk = head / (p.Hq / p.Hkv);
  const int P = p.prefix_len[r];
  const int n_ptiles = (P + kTileKeys - 1) / kTileKeys;
  const int n_ttiles = (p.T + kTileKeys - 1) / kTileKeys;
  const int total = n_ptiles + n_ttiles;
  // the tiles of the tree's own keys stay in one split (they count as one item of the division), so that in every
  // CTA a row either sees a key in the CTA's first tile or in none of its tiles
  const int items = n_ptiles + 1;
  const int per = (items + p.splits - 1) / p.splits;
  const int tile_begin = min(split * per, items);
  const int item_end = min(items, tile_begin + per);
  const int tile_end = item_end == items ? total : item_end;
  const int n = max(0, tile_end - tile_begin);

  if (threadIdx.x == 0) {
    ptx::mbar_init(&q_full, 1);
    for (int i = 0; i < kKSlots; ++i) {
      ptx::mbar_init(&k_full[i], 1);
      ptx::mbar_init(&k_empty[i], 1);
    }
    for (int i = 0; i < kVSlots; ++i) {
      ptx::mbar_init(&v_full[i], 1);
      ptx::mbar_init(&v_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&s_full[i], 1);
      ptx::mbar_init(&s_empty[i], kSoftmaxThreads);
    }
    ptx::mbar_init(&p_full, kSoftmaxThreads);
    ptx::mbar_init(&o_full, 1);
    ptx::mbar_init(&ref_ready, kSoftmaxThreads);
    ptx::mbar_init(&peers_ready, max(1, p.splits - 1));
    s_abort = 0;
    ptx::fence_mbar_init();
  }
  for (int i = threadIdx.x; i < 3 * kRowsPerBlock; i += kThreads) (&s_rowmax[0][0])[i] = float_key(-INFINITY);
  __syncthreads();  // barriers are initialised: the producers start streaming at once
  ptx::cluster_arrive();  // ... and the other CTAs of the cluster may signal this one once they have seen this
  volatile int* abort_flag = &s_abort;
  if (warp != 8) {
    if (warp == 9) {
      ptx::tmem_alloc(&s_tmem_base, 512);
      ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    ptx::named_bar_sync(2, kThreads - 32);
    ptx::tc_fence_after();
  }
  const uint32_t tmem_base = warp != 8 ? s_tmem_base : 0u;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 256;
  // partial result [rows][kXRow], in the K (and V) ring once the loop is over
  float* xbuf = reinterpret_cast<float*>(smem + kQBytes + (kWide ? 2 : 1) * kPBytes);
  // small arrays of the end phase, in the Q tile's place (idle once the last scores have been issued)
  float (*s_lsum)[kRowsPerBlock] = reinterpret_cast<float (*)[kRowsPerBlock]>(smem);          // a row's four (two) partial sums: 1 KB
  float (*s_w)[kRowsPerBlock] = reinterpret_cast<float (*)[kRowsPerBlock]>(smem + 1024);      // [kMaxSplits]: merge weights
  float* s_inv = reinterpret_cast<float*>(smem + 1024 + kMaxSplits * kRowsPerBlock * 4);

  if (warp == 8) {
    // ---------------- TMA producers: lane 0 streams Q and the K tiles, lane 1 the V tiles ----------------
    // The rings hold less than HBM latency x this SM's share of the bandwidth, so tiles further ahead
    // are also requested into the L2.
    if (lane < 2 && n > 0) {
      const bool is_v = lane == 1;
      const int slots = is_v ? kVSlots : kKSlots;
      uint64_t* full = is_v ? v_full : k_full;
      uint64_t* empty = is_v ? v_empty : k_empty;
      const uint32_t ring_off = (is_v ? v_ring : k_ring) - smem_base;
      if (!is_v) {
        ptx::mbar_arrive_expect_tx(&q_full, kQBytes);
        for (int half = 0; half < 2; ++half)
          for (int copy = 0; copy < 2; ++copy)
            ptx::tma_load_4d(smem + half * (kQBytes / 2) + copy * (64 * 128), &tm_q, half * 64, head,
                             rb * kRowsPerBlock + (kWide ? copy * 64 : 0), r, &q_full);
      }
      int slot = 0;
      uint32_t ph = 0;
      const uint64_t pol_kv = ptx::l2_evict_first();  // the cache is read once per step
      auto load_tile = [&](int i) {
        const int tile = tile_begin + i;
        const bool in_prefix = tile < n_ptiles;
        const CUtensorMap* m = is_v ? (in_prefix ? &tm_vp : &tm_vt) : (in_prefix ? &tm_kp : &tm_kt);
        const int key0 = (in_prefix ? tile : tile - n_ptiles) * kTileKeys;
        uint8_t* dst = smem + ring_off + slot * kKVTileBytes;
        ptx::mbar_arrive_expect_tx(&full[slot], kKVTileBytes);
        ptx::tma_load_4d_hint(dst, m, 0, hk, key0, r, &full[slot], pol_kv);
        ptx::tma_load_4d_hint(dst + kKVTileBytes / 2, m, 64, hk, key0, r, &full[slot], pol_kv);
        if (++slot == slots) {
          slot = 0;
          ph ^= 1u;
        }
      };
      auto prefetch_tile = [&](int t) {
        const int tile = tile_begin + t;
        const bool in_prefix = tile < n_ptiles;
        const CUtensorMap* m = is_v ? (in_prefix ? &tm_vp : &tm_vt) : (in_prefix ? &tm_kp : &tm_kt);
        const int key0 = (in_prefix ? tile : tile - n_ptiles) * kTileKeys;
        ptx::tma_prefetch_4d(m, 0, hk, key0, r);
        ptx::tma_prefetch_4d(m, 64, hk, key0, r);
      };
      // The TMA unit works in order and a request queues in front of whatever is issued after it, so
      // requests go out in the order the tiles are needed: the rings' first loads, then the tiles beyond
      // the rings into the L2 (keys and values alternating: the two lanes run these loops in step), then
      // with every tile loaded into a freed slot one more tile further ahead.
      const int n_fill = min(slots, n);
      for (int i = 0; i < n_fill; ++i) load_tile(i);  // the slots start empty
      __syncwarp(3u);
      for (int d = 0; d < kVSlots + kPrefetch - 1; ++d) {
        const int t = slots + d;
        if (d < slots + kPrefetch - 1 && t < n) prefetch_tile(t);
      }
      for (int i = n_fill; i < n; ++i) {
        if (!ptx::mbar_wait(&empty[slot], ph ^ 1u, abort_flag, p.err, p.wait_ns)) break;
        load_tile(i);
        const int t = i + slots + kPrefetch - 1;
        if (t < n) prefetch_tile(t);
      }
    }
  } else if (warp == 9) {
    // ---------------- UMMA issue ----------------
    // S(i) = Q K_i^T needs K tile i and a free score buffer; O += P_i V_i needs the softmax of tile i and
    // V tile i.  Whichever is ready is issued, so scores run ahead of the softmax while the output product
    // never waits for the next tile's keys.
    if (lane == 0 && n > 0) {
      const uint32_t idesc_s = ptx::umma_idesc_bf16(128, kTileKeys);
      const uint32_t idesc_o = ptx::umma_idesc_bf16_b_mn(128, kD);
      bool ok = ptx::mbar_wait(&q_full, 0, abort_flag, p.err, p.wait_ns);
      int is = 0, ip = 0;             // next S, next PV
      int ks_slot = 0, vs_slot = 0;   // ring positions
      uint32_t k_ph = 0, v_ph = 0;
      uint64_t t_idle = 0;
      uint32_t polls = 0;
      while (ok && ip < n) {
        bool did = false;
        if (is < n && ptx::mbar_test_wait(&k_full[ks_slot], k_ph) &&
            ptx::mbar_test_wait(&s_empty[is & 1], ((is >> 1) & 1u) ^ 1u)) {
          ptx::tc_fence_after();
          const uint32_t k_addr = k_ring + ks_slot * kKVTileBytes;
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks) {
            const uint32_t off = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
            ptx::umma_bf16(tmem_s + (is & 1) * 128, ptx::umma_desc_sw128(q_addr + off),
                           ptx::umma_desc_sw128(k_addr + off), idesc_s, ks != 0);
          }
          ptx::umma_commit(&s_full[is & 1]);
          ptx::umma_commit(&k_empty[ks_slot]);
          if (++ks_slot == kKSlots) {
            ks_slot = 0;
            k_ph ^= 1u;
          }
          ++is;
          did = true;
        }
        if (ip < is && ptx::mbar_test_wait(&p_full, ip & 1u) && ptx::mbar_test_wait(&v_full[vs_slot], v_ph)) {
          ptx::tc_fence_after();
          const uint32_t v_addr = v_ring + vs_slot * kKVTileBytes;
#pragma unroll
          for (int ks = 0; ks < kTileKeys / 16; ++ks) {
            // A = P: K-major, two 64-key column blocks of [128 rows][128 B]
            const uint64_t pd = ptx::umma_desc_sw128(p_addr + (ks >> 2) * (128 * 128) + (ks & 3) * 32);
            // B = V: [key][d] with d contiguous (MN-major); 16 keys = two 8-row groups of 1 KB;
            // the two 64-wide halves of d are 16 KB apart
            const uint64_t vd = ptx::umma_desc_sw128_strides(v_addr + ks * 2048, kKVTileBytes / 2, 1024);
            ptx::umma_bf16(tmem_o, pd, vd, idesc_o, (ip | ks) != 0);  // O accumulates across tiles
          }
          if constexpr (kWide) {   // the remainders' tile into the same accumulator
#pragma unroll
            for (int ks = 0; ks < kTileKeys / 16; ++ks) {
              const uint64_t pd = ptx::umma_desc_sw128(p_addr + kPBytes + (ks >> 2) * (128 * 128) + (ks & 3) * 32);
              const uint64_t vd = ptx::umma_desc_sw128_strides(v_addr + ks * 2048, kKVTileBytes / 2, 1024);
              ptx::umma_bf16(tmem_o, pd, vd, idesc_o, 1u);
            }
          }
          ptx::umma_commit(&o_full);
          ptx::umma_commit(&v_empty[vs_slot]);
          if (++vs_slot == kVSlots) {
            vs_slot = 0;
            v_ph ^= 1u;
          }
          ++ip;
          did = true;
        }
        if (did) {
          polls = 0;
        } else if ((++polls & 255u) == 0) {  // bounded: give up after the wait limit without progress
          if (*abort_flag) break;
          const uint64_t now = ptx::global_timer_ns();
          if (polls == 256u) t_idle = now;
          if (now - t_idle > p.wait_ns) {
            *abort_flag = 1;
            atomicOr(p.err, 1);
            break;
          }
        }
      }
    }
  } else {
    // ---------------- softmax warps ----------------
    const int quad = warp & 3, sub = warp >> 2;   // TMEM lane quadrant; which half of the quadrant's keys
    // narrow: tree row = lane within half the quadrants, TMEM lanes row and row + 64 belong to it, 32 keys per thread;
    // wide: tree row = TMEM lane, 64 keys per thread
    const int row = kWide ? quad * 32 + lane : (quad & 1) * 32 + lane;
    const int kofs = kWide ? sub * 64 : (quad >> 1) * 64 + sub * 32;  // first key (within a tile) of this thread's share
    const int j = rb * kRowsPerBlock + row;       // tree row
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint64_t anc_w[4] = {0, 0, 0, 0};
    if (j < p.T) {
#pragma unroll
      for (int w = 0; w < 4; ++w) anc_w[w] = p.anc[(size_t)j * 4 + w];
    }
    // P rows `row` (bf16 value) and `row + 64` (remainder); this thread's 32 keys are 4 pieces of 16 bytes in the
    // 64-key column block (quad >> 1), at piece positions 4 sub .. 4 sub + 3 before the swizzle
    // (wide: rows `row` of the value tile and of the remainder tile, all 8 pieces of column block `sub`)
    const uint32_t p_hi_row = p_addr + (kWide ? sub : (quad >> 1)) * (128 * 128) + row * 128;
    const uint32_t p_lo_row = p_hi_row + (kWide ? kPBytes : 64 * 128);
    const uint32_t o_cols = tmem_o + lane_addr + sub * 64;  // the 64 output columns this thread rescales / reads
    float m_ref = -INFINITY;   // the row's reference (same value in the row's four threads)
    float l_run = 0.f;         // sum of this thread's weights
    bool ok = n > 0;
    for (int i = 0; ok && i < n; ++i) {
      if (!ptx::mbar_wait(&s_full[i & 1], (i >> 1) & 1u, abort_flag, p.err, p.wait_ns)) { ok = false; break; }
      ptx::tc_fence_after();
      const int tile = tile_begin + i;
      const bool in_prefix = tile < n_ptiles;
      const int key0 = (in_prefix ? tile : tile - n_ptiles) * kTileKeys + kofs;
      // visibility of this thread's 32 keys (rows beyond T see the prefix like any other: their query is the
      // zero fill of the tensor map and nothing of theirs is ever stored; that keeps the test below uniform)
      constexpr uint64_t kAll = kWide ? ~0ull : 0xffffffffull;
      uint64_t vis;
      if (in_prefix) {
        const int nvis = P - key0;
        vis = nvis <= 0 ? 0ull : (nvis >= kKeysPerThread ? kAll : ((1ull << nvis) - 1ull));
      } else {
        vis = (anc_w[(key0 >> 6) & 3] >> (key0 & 63)) & kAll;
      }
      float sc[kKeysPerThread];
      if constexpr (kWide) {
        ptx::tmem_ld64(tmem_s + lane_addr + (i & 1) * 128 + kofs, sc);
      } else {
        ptx::tmem_ld32(tmem_s + lane_addr + (i & 1) * 128 + kofs, sc);
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&s_empty[i & 1]);
      // A tile every row of the warp sees whole (all but the last prefix tile) needs no masking, and with a
      // positive scale the maximum can be taken before scaling: weight = 2^(s * c - ref) in one multiply-add.
      const bool whole = p.c > 0.f && __all_sync(0xffffffffu, vis == kAll);
      float m_tile = -INFINITY;
      if (whole) {
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int k = 0; k < kKeysPerThread; ++k) m4[k & 3] = fmaxf(m4[k & 3], sc[k]);
        m_tile = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * p.c;
      } else {
#pragma unroll
        for (int k = 0; k < kKeysPerThread; ++k) {
          sc[k] = ((vis >> k) & 1ull) ? sc[k] * p.c : -INFINITY;
          m_tile = fmaxf(m_tile, sc[k]);
        }
      }
      const float mul = whole ? p.c : 1.f;  // the masked path has scaled its scores already
      if (i == 0) {
        // the first tile fixes the row's reference: the maximum over its four threads
        if (m_tile != -INFINITY) atomicMax(&s_rowmax[0][row], float_key(m_tile));
        ptx::mbar_arrive(&ref_ready);
        if (!ptx::mbar_wait(&ref_ready, 0, abort_flag, p.err, p.wait_ns)) { ok = false; break; }
        m_ref = key_float(s_rowmax[0][row]);
      } else if (m_tile > m_ref + kLazy) {
        atomicMax(&s_rowmax[i % 3][row], float_key(m_tile));  // adopted by the whole row at the next tile
      }
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      float rowsum = 0.f;
#pragma unroll
      for (int k = 0; k < kKeysPerThread; ++k) {
        sc[k] = ptx::ex2(fmaf(sc[k], mul, -m_use));
        rowsum += sc[k];
      }
      if (!(rowsum < 1e37f)) {
        // a score more than 2^120 above everything the row met in earlier tiles (the reference follows with one
        // tile's delay): weights are capped at 2^120 instead of overflowing.  What came before is then below
        // 2^-96 of the result either way.
        rowsum = 0.f;
#pragma unroll
        for (int k = 0; k < kKeysPerThread; ++k) {
          sc[k] = fminf(sc[k], 1.329228e36f);
          rowsum += sc[k];
        }
      }
      if (i >= 1) {
        // PV(i-1) complete: P may be overwritten, O holds tiles 0..i-1, and every post of tile i-1 is visible
        if (!ptx::mbar_wait(&o_full, (i - 1) & 1u, abort_flag, p.err, p.wait_ns)) { ok = false; break; }
        const float posted = key_float(s_rowmax[(i - 1) % 3][row]);
        float alpha = 1.f;
        if (posted > m_ref + kLazy) {   // the same decision in all four threads of the row
          alpha = m_ref == -INFINITY ? 0.f : ptx::ex2(m_ref - posted);
          m_ref = posted;
        }
        if (__any_sync(0xffffffffu, alpha != 1.f)) {
          // rare: this tile's weights and what has been accumulated so far move to the new reference
#pragma unroll
          for (int k = 0; k < kKeysPerThread; ++k) sc[k] *= alpha;
          rowsum *= alpha;
          l_run *= alpha;
          ptx::tc_fence_after();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            float t[16];
            ptx::tmem_ld16(o_cols + c * 16, t);
#pragma unroll
            for (int k = 0; k < 16; ++k) t[k] *= alpha;
            ptx::tmem_st16(o_cols + c * 16, t);
          }
          ptx::tc_fence_before();
        }
      }
      // the bf16 value and what its rounding dropped, four (eight) 16-byte pieces each
#pragma unroll
      for (int c = 0; c < kKeysPerThread / 8; ++c) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float a = sc[8 * c + 2 * k], b = sc[8 * c + 2 * k + 1];
          hi[k] = ptx::pack_bf16x2(a, b);
          lo[k] = ptx::pack_bf16x2(a - __uint_as_float(hi[k] << 16), b - __uint_as_float(hi[k] & 0xffff0000u));
        }
        const uint32_t piece = (uint32_t)(((kWide ? 0 : 4 * sub) + c) ^ (row & 7)) << 4;
        ptx::st_shared_v4(p_hi_row + piece, hi[0], hi[1], hi[2], hi[3]);
        ptx::st_shared_v4(p_lo_row + piece, lo[0], lo[1], lo[2], lo[3]);
      }
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(&p_full);
      l_run += rowsum;
    }
    // The code from here to the end of the kernel runs once per CTA from a cold instruction cache, where
    // every instruction line costs a fetch of its own: loops are rolled and the accumulator is taken from
    // TMEM 16 columns at a time.
    bool have_o = false;
    if (ok && n > 0) have_o = ptx::mbar_wait(&o_full, (n - 1) & 1u, abort_flag, p.err, p.wait_ns);
    have_o = __all_sync(0xffffffffu, have_o);  // the TMEM loads below are warp-wide
    ptx::tc_fence_after();
    // All UMMAs and TMA copies of this CTA have completed: the rings are free to hold the partial result.
    ptx::named_bar_sync(1, kSoftmaxThreads);
    float* x = xbuf + row * kXRow + sub * 64;
    if constexpr (kWide) {
      // every TMEM lane is a tree row of its own: its 64 columns go straight to the buffer
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float v[16];
        if (have_o) {
          ptx::tmem_ld16(o_cols + 16 * c, v);
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) v[k] = 0.f;
        }
        float4* dst = reinterpret_cast<float4*>(x + 16 * c);
#pragma unroll
        for (int k = 0; k < 4; ++k) dst[k] = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
      }
      s_lsum[sub][row] = l_run;
      ptx::named_bar_sync(1, kSoftmaxThreads);
      if (sub == 0) {   // the row's reference and the sum of its weights ride behind its 128 outputs
        xbuf[row * kXRow + kD] = m_ref;
        xbuf[row * kXRow + kD + 1] = s_lsum[0][row] + s_lsum[1][row];
      }
    } else {
      // Rows 64-127 of the accumulator (the remainders' share) go to the buffer first, rows 0-63 are added to them.
      if (quad >= 2) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float v[16];
          if (have_o) {
            ptx::tmem_ld16(o_cols + 16 * c, v);
          } else {
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = 0.f;
          }
          float4* dst = reinterpret_cast<float4*>(x + 16 * c);
#pragma unroll
          for (int k = 0; k < 4; ++k) dst[k] = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
        }
      }
      s_lsum[(quad >> 1) * 2 + sub][row] = l_run;
      ptx::named_bar_sync(1, kSoftmaxThreads);
      if (quad < 2) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float v[16];
          if (have_o) {
            ptx::tmem_ld16(o_cols + 16 * c, v);
          } else {
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = 0.f;
          }
          float4* dst = reinterpret_cast<float4*>(x + 16 * c);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float4 lo = dst[k];
            dst[k] = make_float4(v[4 * k] + lo.x, v[4 * k + 1] + lo.y, v[4 * k + 2] + lo.z, v[4 * k + 3] + lo.w);
          }
        }
        if (sub == 0) {   // the row's reference and the sum of its weights ride behind its 128 outputs
          xbuf[row * kXRow + kD] = m_ref;
          xbuf[row * kXRow + kD + 1] = s_lsum[0][row] + s_lsum[1][row] + s_lsum[2][row] + s_lsum[3][row];
        }
      }
    }
    ptx::tc_fence_before();
  }
  // ---- splits: rank 0 of the cluster collects the partial results of the others ----
  // (measured against sharing the rows between the CTAs, each reading its rows of every partial: loads from
  // another CTA's shared memory are slow enough that one reader of all rows finishes a microsecond sooner)
  const uint32_t rank = ptx::cluster_ctarank();
  __syncwarp();
  ptx::cluster_wait();   // every CTA of the cluster has initialised its barriers (arrived right after doing so)
  __syncthreads();       // ... and this CTA's partial result is complete for every thread to see
  if (p.splits > 1 && rank != 0 && threadIdx.x == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&peers_ready), 0));
  if (warp < 8 && (p.splits == 1 || rank == 0)) {
    bool merged_ok = true;
    if (p.splits > 1) merged_ok = ptx::mbar_wait_cluster(&peers_ready, 0, abort_flag, p.err, p.wait_ns);
    merged_ok = __all_sync(0xffffffffu, merged_ok);
    // weights of the splits per row: out = sum_s w_s O_s / sum_s w_s l_s, w_s = 2^(ref_s - max ref), in split order
    const uint32_t x_addr = ptx::smem_u32(xbuf);
    if (threadIdx.x < kRowsPerBlock) {
      const int rw = threadIdx.x;
      float ms[kMaxSplits], ls[kMaxSplits], m = -INFINITY;
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s) {
        ms[s] = -INFINITY;
        ls[s] = 0.f;
        if (s == 0) {
          ms[s] = xbuf[rw * kXRow + kD];
          ls[s] = xbuf[rw * kXRow + kD + 1];
        } else if (s < p.splits && merged_ok) {
          const uint32_t a = ptx::map_to_cta(x_addr + (uint32_t)(rw * kXRow + kD) * 4u, (uint32_t)s);
          ms[s] = ptx::ld_cluster_f32(a);
          ls[s] = ptx::ld_cluster_f32(a + 4u);
        }
        m = fmaxf(m, ms[s]);
      }
      float l = 0.f;
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s) {
        const float w = ms[s] == -INFINITY ? 0.f : ptx::ex2(ms[s] - m);
        s_w[s][rw] = w;
        l += w * ls[s];
      }
      s_inv[rw] = 1.f / l;
    }
    ptx::named_bar_sync(1, kSoftmaxThreads);
    // 16 pieces of 8 outputs per row; consecutive threads take consecutive pieces (rolled: run-once code)
#pragma unroll 1
    for (int i = 0; i < kRowsPerBlock / 16; ++i) {
      const int idx = i * kSoftmaxThreads + (int)threadIdx.x, rw = idx >> 4, piece = idx & 15;
      const int jj = rb * kRowsPerBlock + rw;
      if (jj >= p.T) continue;
      const uint32_t off = (uint32_t)(rw * kXRow + piece * 8) * 4u;
      float4 a = *reinterpret_cast<const float4*>(xbuf + rw * kXRow + piece * 8);
      float4 b = *reinterpret_cast<const float4*>(xbuf + rw * kXRow + piece * 8 + 4);
      const float w0 = s_w[0][rw];
      float acc[8] = {a.x * w0, a.y * w0, a.z * w0, a.w * w0, b.x * w0, b.y * w0, b.z * w0, b.w * w0};
      if (merged_ok) {
        for (int s = 1; s < p.splits; ++s) {
          const uint32_t ra = ptx::map_to_cta(x_addr + off, (uint32_t)s);
          a = ptx::ld_cluster_v4(ra);
          b = ptx::ld_cluster_v4(ra + 16u);
          const float w = s_w[s][rw];
          acc[0] += w * a.x;
          acc[1] += w * a.y;
          acc[2] += w * a.z;
          acc[3] += w * a.w;
          acc[4] += w * b.x;
          acc[5] += w * b.y;
          acc[6] += w * b.z;
          acc[7] += w * b.w;
        }
      }
      const float inv = s_inv[rw];
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] *= inv;
      store8(p, r * p.T + jj, head * kD + piece * 8, p.Hq * kD, acc);
    }
  }
  __syncwarp();
  __syncthreads();
  if (*abort_flag) __nanosleep(500000);
  if (warp == 9) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
  // nobody leaves while a CTA of the cluster may still read its shared memory
  ptx::cluster_arrive();
  ptx::cluster_wait();
}

}  // namespace

int launch_tree_attn_bf16(cascade_ctx* ctx, const cascade_tree* tree, const __nv_bfloat16* q,
                          const __nv_bfloat16* kp, const __nv_bfloat16* vp, int prefix_cap,
                          const int32_t* prefix_len, const __nv_bfloat16* kt, const __nv_bfloat16* vt,
                          __nv_bfloat16* out, bool out_as_operand, float scale, cudaStream_t s) {
  const cascade_shape& sh = ctx->shape;
  if (sh.D != kD) return CASCADE_ERR_UNSUPPORTED_SHAPE;
  const int T = tree->T, R = 2 * sh.B;
  AttnArgs a;
  a.T = T;
  a.Hq = sh.Hq;
  a.Hkv = sh.Hkv;
  const bool wide = T > kRowsNarrow;
  const int rows_per_block = wide ? kRowsWide : kRowsNarrow;
  a.n_rb = cascade_detail::ceil_div(T, rows_per_block);
  a.prefix_cap = prefix_cap;
  a.prefix_len = prefix_len;
  a.anc = tree->d_anc;
  a.out = out;
  a.out_as_operand = out_as_operand ? 1 : 0;
  a.out_lay = operand_layout(R * T, sh.Hq * kD);
  a.c = scale * 1.4426950408889634f;
  a.err = ctx->dev_error;
  a.wait_ns = ctx->wait_limit_ns;
  // KV splits (1, 2 or 4 CTAs in a cluster per unit): as many as fit on the SMs at once, each keeping a minimum of
  // tiles of the longest possible row
  const int items = cascade_detail::ceil_div(prefix_cap, kTileKeys) + 1;  // prefix tiles + the tree's own tiles as one
  const int units = R * sh.Hq * a.n_rb;
  int splits = 1;
  for (int cand = kMaxSplits; cand > 1; cand /= 2) {
    if (units * cand <= ctx->sm_count && cascade_detail::ceil_div(items, cand) >= ctx->attn_min_tiles_per_split) {
      splits = cand;
      break;
    }
  }
  a.splits = splits;

  const uint64_t dq[4] = {(uint64_t)kD, (uint64_t)sh.Hq, (uint64_t)T, (uint64_t)R};
  const uint64_t sq[3] = {(uint64_t)kD, (uint64_t)sh.Hq * kD, (uint64_t)T * sh.Hq * kD};
  const uint32_t bq[4] = {64, 1, 64, 1};  // 64 rows per load: the wide form fetches its 128 rows in two
  const uint64_t dt[4] = {(uint64_t)kD, (uint64_t)sh.Hkv, (uint64_t)T, (uint64_t)R};
  const uint64_t stt[3] = {(uint64_t)kD, (uint64_t)sh.Hkv * kD, (uint64_t)T * sh.Hkv * kD};
  const uint32_t bkv[4] = {64, 1, kTileKeys, 1};
  const CUtensorMap* mq = get_tmap_4d_bf16(ctx, q, dq, sq, bq);
  const CUtensorMap* mkt = get_tmap_4d_bf16(ctx, kt, dt, stt, bkv);
  const CUtensorMap* mvt = get_tmap_4d_bf16(ctx, vt, dt, stt, bkv);
  const CUtensorMap* mkp = mkt;
  const CUtensorMap* mvp = mvt;
  if (prefix_cap > 0) {
    const uint64_t dp[4] = {(uint64_t)kD, (uint64_t)sh.Hkv, (uint64_t)prefix_cap, (uint64_t)R};
    const uint64_t sp[3] = {(uint64_t)kD, (uint64_t)sh.Hkv * kD, (uint64_t)prefix_cap * sh.Hkv * kD};
    mkp = get_tmap_4d_bf16(ctx, kp, dp, sp, bkv);
    mvp = get_tmap_4d_bf16(ctx, vp, dp, sp, bkv);
  }
  if (!mq || !mkt || !mvt || !mkp || !mvp) return CASCADE_ERR_CUDA;
  bool& configured = ctx->attn_configured;
  if (!configured) {
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(k_tree_attn_bf16<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(k_tree_attn_bf16<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    configured = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, sh.Hq * a.n_rb, R);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;  // the splits of one (row, head, row block) are one cluster
  attr[0].val.clusterDim.x = splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  {
    KernelScope ks(ctx, K_TREE_ATTN, s);
    if (wide)
      CASCADE_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_tree_attn_bf16<true>, *mq, *mkp, *mvp, *mkt, *mvt, a));
    else
      CASCADE_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_tree_attn_bf16<false>, *mq, *mkp, *mvp, *mkt, *mvt, a));
  }
  return CASCADE_OK;
}

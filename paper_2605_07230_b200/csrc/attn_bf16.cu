// Tree-masked attention of the draft-tree rows over the prefix KV cache plus their tree ancestors
// (Section 3 of the paper: the whole draft tree is verified by the target in one parallel pass), bf16,
// for sm_100a.  Memory-bound decode-style kernel: every key/value row is streamed from HBM once per
// (CFG row, head) and shared by all tree rows.
//
// One CTA per (KV split, query head x row block, CFG row):
//   * two producer threads stream 128-key K tiles and V tiles (bf16, 128-byte swizzle) through their own
//     rings (2 and 3 slots) and ask the L2 for the tiles after those;
//   * one thread issues the tensor-core work: S = Q K^T (UMMA 128x128x128) into one of two TMEM score
//     buffers, and O_tile = P V into one of two TMEM output buffers;
//   * four softmax warps own the 128 TMEM lanes.  A row block holds at most 64 tree rows, and the
//     Q tile is loaded twice (UMMA rows r and r+64 are the same tree row): lanes 0-63 take keys 0-63
//     of every tile and lanes 64-127 take keys 64-127, so all four warps work although there are only
//     64 rows.  Each lane keeps its own running (max, sum, output[128]) in registers (online softmax in
//     the exp2 domain); P goes to shared memory as bf16 in the swizzled K-major layout the UMMA reads,
//     with the other half of each row held at zero.  The two halves of a row are merged once at the end;
//   * keys of the prefix are visible to every row up to prefix_len; keys of the tree are visible to
//     row j iff bit i of the packed ancestor-or-self mask of j is set (one 64-bit word per lane and
//     tile half).
// With several KV splits each CTA writes an un-normalised partial (output, max, sum); the CTA of a
// (CFG row, head, row block) that finishes last merges them in split order (a counter per unit, no
// waiting) and writes the bf16 rows.  With one split the CTA writes the final rows itself.
// Every mbarrier wait is bounded (error word + normal teardown on expiry).
#include "cascade_internal.h"
#include "operand.cuh"
#include "ptx.cuh"
#include "tmap.h"

namespace {

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

constexpr int kD = 128;
constexpr int kTileKeys = 128;
constexpr int kRowsPerBlock = 64;
constexpr int kThreads = 192;  // warps 0-3 softmax, warp 4 TMA, warp 5 UMMA issue + TMEM alloc
constexpr int kQBytes = 128 * kD * 2;        // 32 KB: two 64-wide halves of [128 rows][64] bf16
constexpr int kPBytes = 128 * kTileKeys * 2;  // 32 KB
constexpr int kKVTileBytes = kTileKeys * kD * 2;  // 32 KB for K, same for V
constexpr int kKSlots = 2;     // K tiles in shared memory (a slot is free again once S = Q K^T has read it)
constexpr int kVSlots = 3;     // V tiles in shared memory (free once O += P V has read it)
constexpr int kPrefetch = 0;   // with a ring of n slots, tile i + n - 1 + kPrefetch is requested into the L2 when tile i is
                               // loaded (measured 0..3 on 20-tile rows: deeper requests delay the loads that are waited for)
constexpr int kSmemBytes = kQBytes + kPBytes + (kKSlots + kVSlots) * kKVTileBytes + 1024;
constexpr int kXRow = 132;  // row stride (floats) of the half-merge exchange buffer (16-byte aligned rows)
constexpr int kORow = 132;  // row stride (floats) of the output staging buffer (16-byte aligned rows)

struct AttnArgs {
  int T, Hq, Hkv, splits, n_rb, t_pad, prefix_cap;
  const int32_t* prefix_len;
  const uint64_t* anc;
  __nv_bfloat16* out;
  int out_as_operand;     // 1: `out` receives the (R*T x Hq*D) matrix as a GEMM operand (bf16 pair, staged layout)
  OperandLayout out_lay;
  float* part_o;
  float2* part_ml;
  float c;  // softmax_scale * log2(e)
  int* err;
  unsigned long long wait_ns;  // limit of every bounded wait in the kernel
  unsigned int* unit_done;  // [R * Hq * n_rb] finished-split counters, zero between launches
};

__global__ void __launch_bounds__(kThreads, 1)
k_tree_attn_bf16(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kp,
                 const __grid_constant__ CUtensorMap tm_vp, const __grid_constant__ CUtensorMap tm_kt,
                 const __grid_constant__ CUtensorMap tm_vt, const AttnArgs p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t q_full, k_full[kKSlots], k_empty[kKSlots], v_full[kVSlots], v_empty[kVSlots],
      s_full[2], s_empty[2], p_full, o_full;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort, s_last;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t q_addr = smem_base, p_addr = smem_base + kQBytes, k_ring = p_addr + kPBytes,
                 v_ring = k_ring + kKSlots * kKVTileBytes;

  if (threadIdx.x == 128) {  // the TMA warp's first loads should not wait for their descriptors
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
  const int per = (total + p.splits - 1) / p.splits;
  const int tile_begin = split * per;
  const int tile_end = min(total, tile_begin + per);
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
      ptx::mbar_init(&s_empty[i], 128);
    }
    ptx::mbar_init(&p_full, 128);
    ptx::mbar_init(&o_full, 1);
    s_abort = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();  // barriers are initialised: the producers start streaming at once
  volatile int* abort_flag = &s_abort;
  if (warp != 4) {
    // meanwhile the other warps zero P (each UMMA row only ever writes its own key half) and get TMEM
    for (int i = warp == 5 ? 128 + lane : threadIdx.x; i < kPBytes / 16; i += 160)
      reinterpret_cast<uint4*>(smem + kQBytes)[i] = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async_smem();
    if (warp == 5) {
      ptx::tmem_alloc(&s_tmem_base, 512);
      ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    ptx::named_bar_sync(2, 160);
    ptx::tc_fence_after();
  }
  const uint32_t tmem_base = warp != 4 ? s_tmem_base : 0u;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 256;

  // softmax state (warps 0-3)
  float m_run = -INFINITY, l_run = 0.f;

  if (warp == 4) {
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
                             rb * kRowsPerBlock, r, &q_full);
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
  } else if (warp == 5) {
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
    const int urow = warp * 32 + lane;        // UMMA row == TMEM lane
    const int row_in_block = urow & 63;
    const int khalf = urow >> 6;              // which 64 keys of each tile this lane owns
    const int j = rb * kRowsPerBlock + row_in_block;  // tree row
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    uint64_t anc_w[4] = {0, 0, 0, 0};
    if (j < p.T) {
#pragma unroll
      for (int w = 0; w < 4; ++w) anc_w[w] = p.anc[(size_t)j * 4 + w];
    }
    const uint32_t p_row_addr = p_addr + khalf * (128 * 128) + urow * 128;
    const uint32_t o_addr = tmem_o + lane_addr;
    // Online softmax with a lazily updated reference: weights are 2^(s - m_run) where m_run is only
    // raised when a tile's maximum exceeds it by more than kLazy (so weights stay below 2^kLazy).
    // The outputs then accumulate across tiles inside TMEM (the UMMA adds into O); this lane's O and
    // sum are rescaled only on the rare tile that raises m_run.
    constexpr float kLazy = 8.f;
    bool ok = n > 0;
    for (int i = 0; ok && i < n; ++i) {
      if (!ptx::mbar_wait(&s_full[i & 1], (i >> 1) & 1u, abort_flag, p.err, p.wait_ns)) { ok = false; break; }
      ptx::tc_fence_after();
      const int tile = tile_begin + i;
      const bool in_prefix = tile < n_ptiles;
      const int key0 = (in_prefix ? tile : tile - n_ptiles) * kTileKeys + khalf * 64;
      // visibility of this lane's 64 keys as one 64-bit word (rows beyond T see the prefix like any other:
      // their query is the zero fill of the tensor map and nothing of theirs is ever stored; that keeps the
      // test below uniform over a warp)
      uint64_t vis;
      if (in_prefix) {
        const int nvis = P - key0;
        vis = nvis <= 0 ? 0ull : (nvis >= 64 ? ~0ull : ((1ull << nvis) - 1ull));
      } else {
        vis = anc_w[(key0 >> 6) & 3];
      }
      float sc[64];
      ptx::tmem_ld64(tmem_s + lane_addr + (i & 1) * 128 + khalf * 64, sc);
      ptx::tc_fence_before();
      ptx::mbar_arrive(&s_empty[i & 1]);
      // A tile every row of the warp sees whole (all but the last prefix tile) needs no masking, and with a
      // positive scale the maximum can be taken before scaling: weight = 2^(s * c - m) in one multiply-add.
      const bool whole = p.c > 0.f && __all_sync(0xffffffffu, vis == ~0ull);
      float m_tile = -INFINITY;
      if (whole) {
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int k = 0; k < 64; ++k) m4[k & 3] = fmaxf(m4[k & 3], sc[k]);
        m_tile = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * p.c;
      } else {
#pragma unroll
        for (int k = 0; k < 64; ++k) {
          sc[k] = ((vis >> k) & 1ull) ? sc[k] * p.c : -INFINITY;
          m_tile = fmaxf(m_tile, sc[k]);
        }
      }
      const float mul = whole ? p.c : 1.f;  // the masked path has scaled its scores already
      float alpha = 1.f;  // factor for what this lane has accumulated so far
      if (m_run == -INFINITY) {
        m_run = m_tile;   // nothing accumulated yet (all weights so far were zero)
      } else if (m_tile > m_run + kLazy) {
        alpha = ptx::ex2(m_run - m_tile);
        m_run = m_tile;
      }
      const float m_use = m_run == -INFINITY ? 0.f : m_run;
      float rowsum = 0.f;
      uint32_t packed[32];
#pragma unroll
      for (int k = 0; k < 64; k += 2) {
        const float p0 = ptx::ex2(fmaf(sc[k], mul, -m_use)), p1 = ptx::ex2(fmaf(sc[k + 1], mul, -m_use));
        packed[k >> 1] = ptx::pack_bf16x2(p0, p1);
        // sum what the tensor core will actually see (bf16-rounded) so that weights add up to one
        rowsum += __uint_as_float(packed[k >> 1] << 16) + __uint_as_float(packed[k >> 1] & 0xffff0000u);
      }
      if (i >= 1) {
        // PV(i-1) complete: P may be overwritten and O holds tiles 0..i-1
        if (!ptx::mbar_wait(&o_full, (i - 1) & 1u, abort_flag, p.err, p.wait_ns)) { ok = false; break; }
        if (__any_sync(0xffffffffu, alpha != 1.f)) {
          ptx::tc_fence_after();
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float t[16];
            ptx::tmem_ld16(o_addr + c * 16, t);
#pragma unroll
            for (int k = 0; k < 16; ++k) t[k] *= alpha;
            ptx::tmem_st16(o_addr + c * 16, t);
          }
          ptx::tc_fence_before();
        }
      }
#pragma unroll
      for (int c = 0; c < 8; ++c)
        ptx::st_shared_v4(p_row_addr + ((c ^ (urow & 7)) << 4), packed[4 * c], packed[4 * c + 1], packed[4 * c + 2],
                          packed[4 * c + 3]);
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(&p_full);
      l_run = l_run * alpha + rowsum;
    }
    // The code from here to the end of the kernel runs once per CTA from a cold instruction cache, where
    // every instruction line costs a fetch of its own: loops are rolled and the accumulator is taken from
    // TMEM 16 columns at a time instead of as 128 registers.
    bool have_o = false;
    if (ok && n > 0) have_o = ptx::mbar_wait(&o_full, (n - 1) & 1u, abort_flag, p.err, p.wait_ns);
    have_o = __all_sync(0xffffffffu, have_o);  // the TMEM loads below are warp-wide
    ptx::tc_fence_after();
    // ---- merge the two key halves of each row (lanes r and r+64), then write ----
    // all UMMAs and TMA copies of this CTA have completed: the KV ring is free to reuse
    float* xbuf = reinterpret_cast<float*>(smem + kQBytes + kPBytes);  // the K ring: 64 rows x kXRow floats fit
    ptx::named_bar_sync(1, 128);
    if (khalf == 1) {
      float* x = xbuf + row_in_block * kXRow;
#pragma unroll 1
      for (int c = 0; c < kD / 16; ++c) {
        float v[16];
        if (have_o) {
          ptx::tmem_ld16(o_addr + 16 * c, v);
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) v[k] = 0.f;
        }
        float4* dst = reinterpret_cast<float4*>(x + 16 * c);
#pragma unroll
        for (int k = 0; k < 4; ++k) dst[k] = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
      }
      x[kD] = m_run;
      x[kD + 1] = l_run;
    }
    ptx::named_bar_sync(1, 128);
    // Rows leave through shared memory: a thread holds a whole row here, and writing it directly would put
    // 16 bytes per lane 512 bytes apart (measured: 5 us for 32 KB).  The Q / P area is idle by now.
    float* obuf = reinterpret_cast<float*>(smem);  // [64 rows][kORow floats]
    if (khalf == 0) {
      const float* x = xbuf + row_in_block * kXRow;
      const float m1 = x[kD], l1 = x[kD + 1];
      const float m = fmaxf(m_run, m1);
      float w0 = m_run == -INFINITY ? 0.f : ptx::ex2(m_run - m);
      float w1 = m1 == -INFINITY ? 0.f : ptx::ex2(m1 - m);
      const float l = l_run * w0 + l1 * w1;
      if (p.splits == 1) {  // final values
        const float inv = 1.f / l;
        w0 *= inv;
        w1 *= inv;
      } else if (j < p.T) {
        const size_t unit = ((size_t)r * p.Hq + head) * p.splits + split;
        p.part_ml[unit * p.t_pad + j] = make_float2(m, l);
      }
      float* orow = obuf + row_in_block * kORow;
#pragma unroll 1
      for (int c = 0; c < kD / 16; ++c) {
        float v[16];
        if (have_o) {
          ptx::tmem_ld16(o_addr + 16 * c, v);
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) v[k] = 0.f;
        }
        if (j < p.T) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float4 xv = *reinterpret_cast<const float4*>(x + 16 * c + 4 * k);
            *reinterpret_cast<float4*>(orow + 16 * c + 4 * k) =
                make_float4(v[4 * k] * w0 + xv.x * w1, v[4 * k + 1] * w0 + xv.y * w1, v[4 * k + 2] * w0 + xv.z * w1,
                            v[4 * k + 3] * w0 + xv.w * w1);
          }
        }
      }
    }
    ptx::tc_fence_before();
    ptx::named_bar_sync(1, 128);
    if (p.splits == 1) {
      // 16 pieces of 8 outputs per row; consecutive lanes take consecutive pieces (rolled: run-once code)
#pragma unroll 1
      for (int i = 0; i < 8; ++i) {
        const int idx = i * 128 + (int)threadIdx.x, row = idx >> 4, piece = idx & 15;
        const int jj = rb * kRowsPerBlock + row;
        if (jj < p.T) {
          const float4 a = *reinterpret_cast<const float4*>(obuf + row * kORow + piece * 8);
          const float4 b = *reinterpret_cast<const float4*>(obuf + row * kORow + piece * 8 + 4);
          const float v8[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
          store8(p, r * p.T + jj, head * kD + piece * 8, p.Hq * kD, v8);
        }
      }
    } else {
      const size_t unit = ((size_t)r * p.Hq + head) * p.splits + split;
#pragma unroll 2
      for (int i = 0; i < 16; ++i) {
        const int idx = i * 128 + (int)threadIdx.x, row = idx >> 5, c4 = idx & 31;
        const int jj = rb * kRowsPerBlock + row;
        if (jj < p.T)
          *reinterpret_cast<float4*>(p.part_o + (unit * p.t_pad + jj) * kD + 4 * c4) =
              *reinterpret_cast<const float4*>(obuf + row * kORow + 4 * c4);
      }
    }
  }
  __syncwarp();
  __syncthreads();
  if (*abort_flag) __nanosleep(500000);
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
  if (p.splits == 1) return;
  // ---- the last split of this (CFG row, head, row block) to finish merges all of them ----
  const unsigned int unit_id = ((unsigned)r * p.Hq + head) * p.n_rb + rb;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int ticket = atomicAdd(p.unit_done + unit_id, 1u);
    s_last = ticket == (unsigned)p.splits - 1;
    if (s_last) p.unit_done[unit_id] = 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (threadIdx.x >= 128) return;
  // out = sum_s w_s O_s / sum_s w_s l_s, w_s = 2^(m_s - max m), splits taken in index order.  The weights of a
  // row go through shared memory, so that consecutive lanes can take consecutive 32-byte pieces of the
  // partial outputs (a row per lane would read 16 bytes every 512).
  const size_t unit0 = ((size_t)r * p.Hq + head) * p.splits;
  float* s_w = reinterpret_cast<float*>(smem);  // [splits][64] weights, then [64] 1 / sum
  float* s_inv = s_w + p.splits * kRowsPerBlock;
  if (threadIdx.x < kRowsPerBlock) {
    const int row = threadIdx.x, jj = rb * kRowsPerBlock + row;
    if (jj < p.T) {
      float m = -INFINITY;
      for (int s = 0; s < p.splits; ++s) m = fmaxf(m, __ldcg(&p.part_ml[(unit0 + s) * p.t_pad + jj]).x);
      float l = 0.f;
      for (int s = 0; s < p.splits; ++s) {
        const float2 ml = __ldcg(&p.part_ml[(unit0 + s) * p.t_pad + jj]);
        const float w = ml.x == -INFINITY ? 0.f : ptx::ex2(ml.x - m);
        s_w[s * kRowsPerBlock + row] = w;
        l += w * ml.y;
      }
      s_inv[row] = 1.f / l;
    }
  }
  ptx::named_bar_sync(1, 128);
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[i][k] = 0.f;
  for (int s = 0; s < p.splits; ++s) {
    float4 t[8][2];
#pragma unroll
    for (int i = 0; i < 8; ++i) {  // every load of this split issued before the first use
      const int idx = i * 128 + (int)threadIdx.x, row = idx >> 4, piece = idx & 15;
      const int jj = min(rb * kRowsPerBlock + row, p.T - 1);
      const float4* src = reinterpret_cast<const float4*>(p.part_o + ((unit0 + s) * p.t_pad + jj) * kD + piece * 8);
      t[i][0] = __ldcg(src);
      t[i][1] = __ldcg(src + 1);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float w = s_w[s * kRowsPerBlock + ((i * 128 + (int)threadIdx.x) >> 4)];
      acc[i][0] += w * t[i][0].x;
      acc[i][1] += w * t[i][0].y;
      acc[i][2] += w * t[i][0].z;
      acc[i][3] += w * t[i][0].w;
      acc[i][4] += w * t[i][1].x;
      acc[i][5] += w * t[i][1].y;
      acc[i][6] += w * t[i][1].z;
      acc[i][7] += w * t[i][1].w;
    }
  }
  // The sums go back to shared memory and leave through a short rolled loop: this code runs once per CTA
  // from a cold instruction cache, and every instruction line of an unrolled version costs a fetch.
  float* obuf = s_inv + kRowsPerBlock;  // [64 rows][kORow floats]
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int idx = i * 128 + (int)threadIdx.x, row = idx >> 4, piece = idx & 15;
    float4* dst = reinterpret_cast<float4*>(obuf + row * kORow + piece * 8);
    dst[0] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    dst[1] = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
  }
  __syncwarp();  // a thread reads back only what it wrote
#pragma unroll 1
  for (int i = 0; i < 8; ++i) {
    const int idx = i * 128 + (int)threadIdx.x, row = idx >> 4, piece = idx & 15;
    const int jj = rb * kRowsPerBlock + row;
    if (jj >= p.T) continue;
    const float inv = s_inv[row];
    const float4 a = *reinterpret_cast<const float4*>(obuf + row * kORow + piece * 8);
    const float4 b = *reinterpret_cast<const float4*>(obuf + row * kORow + piece * 8 + 4);
    const float v8[8] = {a.x * inv, a.y * inv, a.z * inv, a.w * inv, b.x * inv, b.y * inv, b.z * inv, b.w * inv};
    store8(p, r * p.T + jj, head * kD + piece * 8, p.Hq * kD, v8);
  }
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
  a.n_rb = cascade_detail::ceil_div(T, kRowsPerBlock);
  a.t_pad = (int)cascade_detail::align_up(sh.T_max, 64);
  a.prefix_cap = prefix_cap;
  a.prefix_len = prefix_len;
  a.anc = tree->d_anc;
  a.out = out;
  a.out_as_operand = out_as_operand ? 1 : 0;
  a.out_lay = operand_layout(R * T, sh.Hq * kD);
  a.part_o = ctx->attn_part_o;
  a.part_ml = ctx->attn_part_ml;
  a.c = scale * 1.4426950408889634f;
  a.err = ctx->dev_error;
  a.wait_ns = ctx->wait_limit_ns;
  a.unit_done = ctx->attn_unit_done;
  // KV splits: as many as fit on the SMs at once, never more splits than tiles or than the scratch holds
  const int n_tiles = cascade_detail::ceil_div(prefix_cap, kTileKeys) + cascade_detail::ceil_div(T, kTileKeys);
  const int units = R * sh.Hq * a.n_rb;
  int splits = ctx->sm_count / units;
  if (splits > n_tiles) splits = n_tiles;
  if (splits > ctx->attn_max_splits) splits = ctx->attn_max_splits;
  // merging splits costs a few microseconds of its own: not worth it for a handful of tiles
  if (splits > 1 && n_tiles - cascade_detail::ceil_div(n_tiles, splits) < 4) splits = 1;
  if (splits < 1) splits = 1;
  a.splits = splits;

  const uint64_t dq[4] = {(uint64_t)kD, (uint64_t)sh.Hq, (uint64_t)T, (uint64_t)R};
  const uint64_t sq[3] = {(uint64_t)kD, (uint64_t)sh.Hq * kD, (uint64_t)T * sh.Hq * kD};
  const uint32_t bq[4] = {64, 1, kRowsPerBlock, 1};
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
    CASCADE_CUDA_TRY(cudaFuncSetAttribute(k_tree_attn_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    configured = true;
  }
  dim3 grid(splits, sh.Hq * a.n_rb, R);
  {
    KernelScope ks(ctx, K_TREE_ATTN, s);
    k_tree_attn_bf16<<<grid, kThreads, kSmemBytes, s>>>(*mq, *mkp, *mvp, *mkt, *mvt, a);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}

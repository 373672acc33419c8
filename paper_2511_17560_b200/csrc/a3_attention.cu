// Attention of the carried rows over the fused GQA cache (Eq. 4, Eq. 5) on the 5th-generation tensor cores.
//
// Row m sits at global position pos[m] and sees cache slots 0..pos[m].  The G = Hq/Hkv query heads that share one
// KV head are packed into the row dimension (flat row r -> token r / G, head r % G); one CTA owns 128 flat rows of
// one KV head and walks the keys in tiles of 128 up to the largest position among its rows.
//
//   warp 0 (one lane)   TMA producer: K and V tiles of the cache ([slots][Hkv*D] seen as a 2-D tensor, 128-byte
//                       swizzle), a ring of three stages each.
//   warp 1 (one lane)   tcgen05.mma issuer: S = Q K^T (128 x 128 x D) into one of two TMEM buffers, and, once the
//                       probabilities of a tile are back in tensor memory, O~ += P V (128 x D x 128; P is the A
//                       operand read from TMEM, V an MN-major operand in shared memory) accumulated in TMEM.
//                       S of tile t+1 is issued before P V of tile t, so the tensor core works while the
//                       softmax threads do.
//   warps 2..9          two threads per row, each owning half of the tile's key columns with an exponent
//                       reference, a row sum and a TMEM output accumulator of its own: the row of S is read into
//                       registers, P = exp2(s * scale - ref) (one FMA and one ex2.approx per element) is written
//                       as bf16 pairs over the columns S came from.  The reference is the first tile's maximum; no
//                       maximum is tracked afterwards - a logit far above the reference shows as a row sum beyond
//                       2^16, and only then is the tile's maximum taken, the reference raised, the accumulator
//                       rescaled in TMEM and the tile redone.  At the end of an item the two partial softmaxes of
//                       a row are merged, normalised and stored.
// TMEM (512 columns): S buffers at 0 and 128, the two output accumulators at 256 and 256 + D.
// Statistics are fp32 in the exp2 domain.  Every mbarrier wait is bounded (see a3_gemm.cu); there is no block-
// wide or named barrier inside the loops, so a role that gives up cannot strand another.
#include <cuda.h>

#include "a3_internal.cuh"
#include "a3_attn.cuh"

namespace a3 {

constexpr int ATC_THREADS = 320;  // TMA warp, MMA warp, 8 softmax warps (two threads per row)
template <int D>
struct AtcLayout {
  static constexpr int SUB = 128 * 64 * 2;           // one [128][64] bf16 sub-tile: 16 KiB
  static constexpr int Q_BYTES = (D / 64) * SUB;
  static constexpr int KV_STAGE = 2 * (D / 64) * SUB;  // K then V
  static constexpr int KV_STAGES = 3;
  static constexpr int Q_OFF = 0;
  static constexpr int KV_OFF = Q_BYTES;
  static constexpr int BAR_OFF = KV_OFF + KV_STAGES * KV_STAGE;
  static constexpr int XCH_OFF = BAR_OFF + 256;          // float2 exchange[2 halves][128 rows]
  static constexpr int SMEM_BYTES = XCH_OFF + 2048;      // the dynamic shared window must be 1024-byte aligned (checked)
};

// One unit of work: a 128-row tile of one KV head and one segment of its key tiles.
struct AtcItem {
  int g, r0, maxpos, minpos;
  int nkt_all;   // key tiles the row tile needs in total
  int kt0, nkt;  // this segment: first key tile and count
  int z;         // segment index
  bool valid;    // the segment exists for this row tile
  bool partial;  // the row tile has several segments: leave unnormalised partial results for the combine kernel
};

// Items are numbered longest row tile first (rows are sorted by position, so the last tile sees the most keys),
// then segment, then KV head.
__device__ __forceinline__ AtcItem atc_item(int i, const int32_t* __restrict__ pos, int M, int G, int Hkv, int kv_len,
                                            int row_tiles, int n_split, int tiles_per_split) {
  AtcItem it;
  const int per_tile = n_split * Hkv;
  const int tile = row_tiles - 1 - i / per_tile;
  const int rem = i % per_tile;
  it.z = rem / Hkv;
  it.g = rem % Hkv;
  it.r0 = tile * ATC_BM;
  const int last_tok = min(M - 1, (it.r0 + ATC_BM - 1) / G);
  it.maxpos = min(pos[last_tok], kv_len - 1);
  it.minpos = pos[it.r0 / G];
  it.nkt_all = it.maxpos < 0 ? 0 : it.maxpos / ATC_BN + 1;
  const int n_active = (it.nkt_all + tiles_per_split - 1) / tiles_per_split;
  it.valid = it.z < max(n_active, 1);
  it.kt0 = it.z * tiles_per_split;
  it.nkt = max(0, min(tiles_per_split, it.nkt_all - it.kt0));
  it.partial = n_active > 1;
  return it;
}

// Persistent kernel: one CTA per SM walks its share of the items.  Item i of round r goes to CTA (i mod C) on even
// rounds and to CTA C-1-(i mod C) on odd ones, so every CTA gets a mix of long and short items without any atomic.
// Barrier phases and buffer indices follow counters that run across items (`it`: key tiles, `qn`: items with work),
// so the TMA producer keeps prefetching the next item's K/V while the current one drains.
template <int D>
__global__ void __launch_bounds__(ATC_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const bf16* __restrict__ q, const int32_t* __restrict__ pos, int M, int kv_len, bf16* __restrict__ o,
                    float* __restrict__ lse, int Hq, int Hkv, float scale_log2, uint32_t* status,
                    int n_split, int tiles_per_split, float* __restrict__ part_o, float2* __restrict__ part_ml) {
  using L = AtcLayout<D>;
  using namespace atc;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* base_ptr = smem_raw;
  if (base & 1023u) {  // the swizzled tiles need a 1024-byte aligned window; uniform for the CTA, nothing is set up yet
    if (threadIdx.x == 0) atomicOr(status, A3_DEV_WAIT_EXHAUSTED);
    return;
  }
  // barriers: k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], p_ready[2], q_ready, p_free[2].
  // K and V have separate rings: a K stage is free as soon as its S = Q K^T has run, so the next K tile is on its
  // way long before the P V of the same tile releases the V stage; with one barrier for both, every tile would
  // wait for a full copy latency.
  const uint32_t bars = base + L::BAR_OFF;
  auto k_full = [&](int s) { return bars + 8u * s; };
  auto k_empty = [&](int s) { return bars + 8u * (3 + s); };
  auto v_full = [&](int s) { return bars + 8u * (6 + s); };
  auto v_empty = [&](int s) { return bars + 8u * (9 + s); };
  auto s_full = [&](int b) { return bars + 8u * (12 + b); };
  // p_ready alternates between two barriers: a fast warp may finish tile t+1 before a slow warp has arrived for
  // tile t, and on a single barrier its second arrival would be counted towards tile t
  auto p_ready = [&](int b) { return bars + 8u * (14 + b); };
  const uint32_t q_ready = bars + 8u * 16;
  auto p_free = [&](int b) { return bars + 8u * (17 + b); };
  // pair[q][parity]: the two warps that share TMEM lane quarter q (64 threads) meet here to exchange row statistics
  auto pair_bar = [&](int qd, int par) { return bars + 8u * (19 + qd * 2 + par); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::BAR_OFF + 8 * 27);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::BAR_OFF + 8 * 27 + 8);
  float2* xch = reinterpret_cast<float2*>(base_ptr + L::XCH_OFF);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = Hq / Hkv;
  const int rows_total = M * G;
  const int row_tiles = (rows_total + ATC_BM - 1) / ATC_BM;
  const int rows_pad = row_tiles * ATC_BM;
  const int n_items = row_tiles * n_split * Hkv;
  const int C = gridDim.x, cta = blockIdx.x;
  const bool want_o = o != nullptr;
  // item of round r for this CTA, or -1
  auto item_index = [&](int r) {
    const int i = r * C + ((r & 1) ? C - 1 - cta : cta);
    return i < n_items ? i : -1;
  };
  const int rounds = (n_items + C - 1) / C;

  if (threadIdx.x == 0) {
    for (int i = 0; i < L::KV_STAGES; ++i) {
      mbar_init(k_full(i), 1);
      mbar_init(k_empty(i), 1);
      mbar_init(v_full(i), 1);
      mbar_init(v_empty(i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(s_full(i), 1);
      mbar_init(p_free(i), 1);
    }
    mbar_init(p_ready(0), 256);
    mbar_init(p_ready(1), 256);
    mbar_init(q_ready, 256);
    for (int i = 0; i < 8; ++i) mbar_init(pair_bar(i >> 1, i & 1), 64);
    abort_flag[0] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();  // the set-up above overlapped the previous kernel's tail; positions, Q and the cache are read below
  pdl_launch_dependents();
  const uint32_t tmem_s0 = tmem_base, tmem_o = tmem_base + 256;

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmV) : "memory");
      uint32_t it = 0;
      bool ok = true;
      for (int r = 0; r < rounds && ok; ++r) {
        const int i = item_index(r);
        if (i < 0) continue;
        const AtcItem w = atc_item(i, pos, M, G, Hkv, kv_len, row_tiles, n_split, tiles_per_split);
        if (!w.valid) continue;
        for (int kt = 0; kt < w.nkt; ++kt, ++it) {
          const int s = it % L::KV_STAGES;
          const uint32_t ph = (it / L::KV_STAGES) & 1;
          const uint32_t sk = base + L::KV_OFF + s * L::KV_STAGE, sv = sk + (D / 64) * L::SUB;
          ok = mbar_wait(k_empty(s), ph ^ 1, abort_flag, status);
          if (!ok) break;
          mbar_expect_tx(k_full(s), L::KV_STAGE / 2);
#pragma unroll
          for (int j = 0; j < D / 64; ++j) tma_load_2d(sk + j * L::SUB, &tmK, w.g * D + 64 * j, (w.kt0 + kt) * ATC_BN, k_full(s));
          if (want_o) {  // the statistics-only pass never reads V
            ok = mbar_wait(v_empty(s), ph ^ 1, abort_flag, status);
            if (!ok) break;
            mbar_expect_tx(v_full(s), L::KV_STAGE / 2);
#pragma unroll
            for (int j = 0; j < D / 64; ++j) tma_load_2d(sv + j * L::SUB, &tmV, w.g * D + 64 * j, (w.kt0 + kt) * ATC_BN, v_full(s));
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc(ATC_BN, 0);
      constexpr uint32_t idesc_o = idesc(D, 1);
      const uint32_t sq = base + L::Q_OFF;
      auto issue_s = [&](uint32_t t) {  // S of running key tile t into S buffer t & 1, from K stage t mod 3
        const uint32_t sk = base + L::KV_OFF + (t % L::KV_STAGES) * L::KV_STAGE;
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t sub = (k / 4) * L::SUB + (k % 4) * 32;
          mma_f16(tmem_s0 + (t & 1) * 128, desc_k_sw128(sq + sub), desc_k_sw128(sk + sub), idesc_s, k != 0);
        }
        commit(s_full(t & 1));
        commit(k_empty(t % L::KV_STAGES));  // the K stage is free once these MMAs have read it
      };
      uint32_t it = 0, qn = 0;
      bool ok = true;
      for (int r = 0; r < rounds && ok; ++r) {
        const int i = item_index(r);
        if (i < 0) continue;
        const AtcItem w = atc_item(i, pos, M, G, Hkv, kv_len, row_tiles, n_split, tiles_per_split);
        if (!w.valid || w.nkt == 0) continue;
        ok = mbar_wait(q_ready, qn & 1, abort_flag, status);
        ++qn;
        ok = ok && mbar_wait(k_full(it % L::KV_STAGES), (it / L::KV_STAGES) & 1, abort_flag, status);
        if (!ok) break;
        fence_after();
        issue_s(it);
        for (int kt = 0; kt < w.nkt; ++kt, ++it) {
          if (kt + 1 < w.nkt) {
            ok = mbar_wait(k_full((it + 1) % L::KV_STAGES), ((it + 1) / L::KV_STAGES) & 1, abort_flag, status);
            if (!ok) break;
            fence_after();
            issue_s(it + 1);
          }
          ok = mbar_wait(p_ready(it & 1), (it >> 1) & 1, abort_flag, status);
          if (!ok) break;
          if (want_o) {
            ok = mbar_wait(v_full(it % L::KV_STAGES), (it / L::KV_STAGES) & 1, abort_flag, status);
            if (!ok) break;
          }
          fence_after();
          if (want_o) {
            const uint32_t sv = base + L::KV_OFF + (it % L::KV_STAGES) * L::KV_STAGE + (D / 64) * L::SUB;
            // P of this tile lies over the first half of each thread's S columns (see the softmax warps): keys
            // 64 h + 16 kk .. + 15 in the eight 32-bit columns at 64 h + 8 kk of S buffer it & 1.  The next S into
            // that buffer is issued after these MMAs and the tensor pipe runs in order.
            const uint32_t tp = tmem_s0 + (it & 1) * 128;
#pragma unroll
            for (int k = 0; k < ATC_BN / 16; ++k) {
              const uint64_t db = desc_mn_sw128(sv + k * 16 * 128, L::SUB);
              // each half of the tile's keys accumulates into an output of its own (see the softmax warps)
              mma_f16_ts(tmem_o + (k / 4) * D, tp + (k / 4) * 64 + (k % 4) * 8, db, idesc_o, (kt | (k % 4)) != 0);
            }
            commit(p_free(it & 1));  // P V of this tile is complete: the outputs hold tiles 0..kt
            commit(v_empty(it % L::KV_STAGES));
          }
        }
      }
    }
  } else {
    // ---------------- softmax / epilogue: two threads per row.  Thread `half` of a row owns keys 64*half .. +63 of
    // every key tile, with an exponent reference, a row sum and an output accumulator in TMEM of its own, so the
    // two never have to agree on anything while the keys stream; they meet once per item (warps w and w+4 share a
    // TMEM lane quarter, a 64-thread mbarrier and an exchange slot in shared memory) to merge the two partial
    // softmaxes, and each then normalises and stores half of the output columns.
    const int half = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t tmem_oh = tmem_o + half * D;  // this thread's accumulator
    constexpr float OVERFLOW_GUARD = 65536.f;
    uint32_t it = 0, px = 0;  // running key tile; running count of pair exchanges (parity of the pair barrier)
    bool ok = true;
    // publish `mine`, meet the partner, return the partner's value; false if the wait was abandoned
    auto exchange = [&](float2 mine, float2& theirs) {
      // One slot per thread is enough: a thread overwrites its slot at the end of the next item, after that item's
      // first S tile, which the MMA warp issues only once all 256 threads have arrived at q_ready - and the
      // partner arrives there after it has read this slot.
      const int par = px & 1;
      xch[half * 128 + row] = mine;
      mbar_arrive(pair_bar(quarter, par));
      const bool got = __all_sync(0xffffffffu, mbar_wait(pair_bar(quarter, par), (px >> 1) & 1, abort_flag, status));
      theirs = xch[(half ^ 1) * 128 + row];
      ++px;
      return got;
    };

    for (int r = 0; r < rounds && ok; ++r) {
      const int i = item_index(r);
      if (i < 0) continue;
      const AtcItem w = atc_item(i, pos, M, G, Hkv, kv_len, row_tiles, n_split, tiles_per_split);
      if (!w.valid) continue;
      const int fr = w.r0 + row;
      const bool row_ok = fr < rows_total;
      const int tok = row_ok ? fr / G : 0;
      const int hq = w.g * G + (row_ok ? fr % G : 0);
      const int lim = row_ok ? min(pos[tok], kv_len - 1) : -1;
      const size_t prow = ((size_t)w.z * Hkv + w.g) * (size_t)rows_pad + fr;  // partial-result row

      if (w.nkt == 0) {
        // no visible key at all (only with invalid positions): defined output, no pipeline work
        if (row_ok && want_o && !w.partial) {
          uint4* dst = reinterpret_cast<uint4*>(o + ((size_t)tok * Hq + hq) * D + half * (D / 2));
#pragma unroll
          for (int c = 0; c < D / 16; ++c) dst[c] = make_uint4(0, 0, 0, 0);
        }
        if (row_ok && w.partial && half == 0) part_ml[prow] = make_float2(0.f, 0.f);
        if (row_ok && !w.partial && lse && half == 0) lse[(size_t)tok * Hq + hq] = -INFINITY;
        continue;
      }

      // Q row -> shared memory, swizzled K-major sub-tiles (each thread copies half of the row's 16-byte chunks).
      // The previous item's S MMAs have all completed (their last s_full was waited for), so the Q buffer is free.
      {
        const uint4* src = reinterpret_cast<const uint4*>(q + ((size_t)tok * Hq + hq) * D);
#pragma unroll
        for (int cc = 0; cc < D / 16; ++cc) {
          const int c = half * (D / 16) + cc;
          uint4 v = row_ok ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
          *reinterpret_cast<uint4*>(base_ptr + L::Q_OFF + (c / 8) * L::SUB + swz(row, c % 8)) = v;
        }
        fence_async_smem();
        mbar_arrive(q_ready);
      }

      // Exponent reference m_ref and row sum l_run of this thread's keys (see the file header for the protocol).
      float m_ref = 0.f, l_run = 0.f;
      uint32_t it_last = it;
      for (int kt = 0; kt < w.nkt; ++kt, ++it) {
        it_last = it;
        // the result of every wait is made warp-uniform: tcgen05.ld/st are warp-wide instructions
        ok = __all_sync(0xffffffffu, mbar_wait(s_full(it & 1), (it >> 1) & 1, abort_flag, status));
        if (!ok) break;
        fence_after();
        const uint32_t ts = tmem_s0 + (it & 1) * 128 + lane_addr + half * 64;
        const int key0 = (w.kt0 + kt) * ATC_BN + half * 64;  // first key of this thread's columns
        const bool need_mask = (w.kt0 + kt) * ATC_BN + ATC_BN - 1 > w.minpos;
        // The row's 64 logits of this thread, raw, into registers
        float x[64];
        ld32(ts, x);
        ld32(ts + 32, x + 32);
        wait_ld();
        if (want_o && it >= 2) {
          // keeps every phase of p_free[b] observed in order, so that the parity waits below cannot mistake an older
          // completion for the one they mean (P V of running tile it-2 finished long ago: this does not block)
          ok = __all_sync(0xffffffffu, mbar_wait(p_free(it & 1), ((it >> 1) & 1) ^ 1, abort_flag, status));
          if (!ok) break;
        }
        // maximum of the scaled, masked logits (first tile and the rare re-reference only)
        auto row_max = [&]() {
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int e = 0; e < 64; ++e) {
            const float t = (need_mask && key0 + e > lim) ? -INFINITY : x[e] * scale_log2;
            m4[e & 3] = fmaxf(m4[e & 3], t);
          }
          return fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        };
        // x <- exp2(x * scale - m_ref) (one FMA and one ex2.approx per element; ex2 maps -inf to +0); returns the sum
        auto to_probabilities = [&]() {
          float ls[4] = {0.f, 0.f, 0.f, 0.f};
          const float neg_ref = -m_ref;
          if (need_mask) {
#pragma unroll
            for (int e = 0; e < 64; ++e) {
              float t = fmaf(x[e], scale_log2, neg_ref);
              if (key0 + e > lim) t = -INFINITY;
              x[e] = ex2_approx(t);
              ls[e & 3] += x[e];
            }
          } else {
            // packed fp32 pairs (fma.rn.f32x2 / add.rn.f32x2): half the issue slots for the FMA and the sum
            const float2 sc2 = make_float2(scale_log2, scale_log2), nr2 = make_float2(neg_ref, neg_ref);
            float2 s2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int e = 0; e < 64; e += 2) {
              const float2 t = __ffma2_rn(make_float2(x[e], x[e + 1]), sc2, nr2);
              x[e] = ex2_approx(t.x);
              x[e + 1] = ex2_approx(t.y);
              s2[(e >> 1) & 1] = __fadd2_rn(s2[(e >> 1) & 1], make_float2(x[e], x[e + 1]));
            }
            ls[0] = s2[0].x, ls[1] = s2[0].y, ls[2] = s2[1].x, ls[3] = s2[1].y;
          }
          return (ls[0] + ls[1]) + (ls[2] + ls[3]);
        };
        if (kt == 0) {
          const float mx = row_max();
          m_ref = mx == -INFINITY ? 0.f : mx;
        }
        float lsum = to_probabilities();
        // No maximum is tracked on the way: a logit far above the reference shows in the sum (each of the 64 terms
        // is at most the largest one), and anything below 2^16 is harmless for bf16 P and the fp32 accumulators.
        // Above it - rare - the reference is raised to the tile's true maximum, the output and the sum so far are
        // rescaled, and the tile is redone from the logits still in tensor memory.
        if (kt > 0 && __any_sync(0xffffffffu, !(lsum <= OVERFLOW_GUARD))) {
          ld32(ts, x);
          ld32(ts + 32, x + 32);
          wait_ld();
          const float mx = row_max();
          const float raise = fmaxf(mx - m_ref, 0.f);  // lanes that triggered nothing keep their reference (raise 0)
          const float f = exp2f(-raise);
          m_ref += raise;
          l_run *= f;
          if (want_o) {
            // the output so far must be complete (P V of the previous tile) before it is rescaled in place
            ok = __all_sync(0xffffffffu, mbar_wait(p_free((it - 1) & 1), ((it - 1) >> 1) & 1, abort_flag, status));
            if (!ok) break;
            fence_after();
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              float t[32];
              const uint32_t to = tmem_oh + lane_addr + c * 32;
              ld32(to, t);
              wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) t[e] *= f;
              st32(to, t);
            }
            wait_st();
          }
          lsum = to_probabilities();
        }
        l_run += lsum;
        if (want_o) {
          // P as bf16 pairs over the first 32 of this thread's 64 S columns (all of them are in registers by now):
          // the A operand of the P V MMA is read from tensor memory
          uint32_t pk[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 v = pack8(x + 8 * j);
            pk[4 * j] = v.x, pk[4 * j + 1] = v.y, pk[4 * j + 2] = v.z, pk[4 * j + 3] = v.w;
          }
          st32(ts, reinterpret_cast<const float*>(pk));
          wait_st();
          if (w.kt0 + kt == w.nkt_all - 1 && half == 0) {
            // slots beyond the row tile's last visible key may hold anything: they get probability zero, and zero
            // times a non-finite value would still poison the product, so clear those V rows of the last tile
            // (thread `row` of the first half clears key `row`)
            const int first_bad = w.maxpos - (w.kt0 + kt) * ATC_BN + 1;
            const int vs = it % L::KV_STAGES;
            const bool landed = mbar_wait(v_full(vs), (it / L::KV_STAGES) & 1, abort_flag, status);  // the V tile must have landed before rows of it are cleared
            if (landed && row >= first_bad) {
              unsigned char* sv = base_ptr + L::KV_OFF + vs * L::KV_STAGE + (D / 64) * L::SUB;
#pragma unroll
              for (int j = 0; j < D / 64; ++j)
#pragma unroll
                for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(sv + j * L::SUB + row * 128 + c * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_async_smem();
          }
        }
        fence_before();
        mbar_arrive(p_ready(it & 1));
      }
      if (!ok) break;
      // merge the two partial softmaxes of the row: common reference m, weights f_mine / f_other for the two
      // accumulators, row sum l (a half that saw no visible key has l == 0 and no say in the reference)
      float f_mine, f_other;
      {
        float2 other;
        ok = exchange(make_float2(m_ref, l_run), other);
        if (!ok) break;
        const float m_a = l_run > 0.f ? m_ref : -INFINITY, m_b = other.y > 0.f ? other.x : -INFINITY;
        const float m = fmaxf(m_a, m_b);
        f_mine = l_run > 0.f ? exp2f(m_a - m) : 0.f;
        f_other = other.y > 0.f ? exp2f(m_b - m) : 0.f;
        const float l0 = half == 0 ? l_run * f_mine : other.y * f_other, l1 = half == 0 ? other.y * f_other : l_run * f_mine;
        l_run = l0 + l1;  // same order in both threads
        m_ref = m == -INFINITY ? 0.f : m;
      }
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      if (want_o) {
        ok = __all_sync(0xffffffffu, mbar_wait(p_free(it_last & 1), (it_last >> 1) & 1, abort_flag, status));
        if (!ok) break;
        fence_after();
        bf16* dst = o + ((size_t)tok * Hq + hq) * D + half * (D / 2);
        const float fa = (half == 0 ? f_mine : f_other) * (w.partial ? 1.f : inv), fb = (half == 0 ? f_other : f_mine) * (w.partial ? 1.f : inv);
#pragma unroll 1
        for (int c = 0; c < D / 64; ++c) {  // this thread's half of the output columns, from both accumulators
          float t[32], u[32];
          ld32(tmem_o + lane_addr + half * (D / 2) + c * 32, t);
          ld32(tmem_o + D + lane_addr + half * (D / 2) + c * 32, u);
          wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) t[e] = fmaf(t[e], fa, u[e] * fb);
          if (row_ok && w.partial) {
            float4* pd = reinterpret_cast<float4*>(part_o + prow * D + half * (D / 2) + c * 32);
#pragma unroll
            for (int j = 0; j < 8; ++j) pd[j] = make_float4(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3]);
          } else if (row_ok) {
#pragma unroll
            for (int j = 0; j < 4; ++j) reinterpret_cast<uint4*>(dst + c * 32)[j] = pack8(t + 8 * j);
          }
          __syncwarp();
        }
        // the next item's first P V overwrites O: it is issued only after this item's p_ready arrivals of all 256
        // threads for that tile, which each thread makes after the loads above
        fence_before();
      }
      if (half == 0) {
        if (row_ok && w.partial) part_ml[prow] = make_float2(m_ref, l_run);
        if (row_ok && !w.partial && lse) lse[(size_t)tok * Hq + hq] = l_run > 0.f ? (m_ref + log2f(l_run)) * ATC_LN2 : -INFINITY;
      }
    }
  }
  atc::fence_before();
  __syncthreads();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

// One warp per (flat row, KV head) of a row tile that was split over the keys: merges the segments' partial results
// in segment order (fixed, so the result is reproducible): O = sum_z O_z 2^(m_z - m) / sum_z l_z 2^(m_z - m).
template <int D>
__global__ void __launch_bounds__(128)
attention_combine_kernel(const int32_t* __restrict__ pos, int M, int kv_len, int Hq, int Hkv, int tiles_per_split, int rows_pad,
                         const float* __restrict__ part_o, const float2* __restrict__ part_ml, bf16* __restrict__ o,
                         float* __restrict__ lse) {
  const int G = Hq / Hkv;
  const int rows_total = M * G;
  const int fr = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int g = blockIdx.y, lane = threadIdx.x & 31;
  if (fr >= rows_total) return;
  const int r0 = (fr / ATC_BM) * ATC_BM;
  const int last_tok = min(M - 1, (r0 + ATC_BM - 1) / G);
  const int maxpos = min(pos[last_tok], kv_len - 1);
  const int nkt_all = maxpos < 0 ? 0 : maxpos / ATC_BN + 1;
  const int n_active = (nkt_all + tiles_per_split - 1) / tiles_per_split;
  if (n_active <= 1) return;  // written directly by the attention kernel
  float m = -INFINITY;
  for (int z = 0; z < n_active; ++z) {
    const float2 ml = part_ml[((size_t)z * Hkv + g) * rows_pad + fr];
    if (ml.y > 0.f) m = fmaxf(m, ml.x);
  }
  constexpr int PER = D / 32;
  float acc[PER];
#pragma unroll
  for (int e = 0; e < PER; ++e) acc[e] = 0.f;
  float l = 0.f;
  for (int z = 0; z < n_active; ++z) {
    const size_t prow = ((size_t)z * Hkv + g) * rows_pad + fr;
    const float2 ml = part_ml[prow];
    if (!(ml.y > 0.f)) continue;
    const float w = exp2f(ml.x - m);
    l += ml.y * w;
    if (o) {
      const float* src = part_o + prow * D + lane * PER;
#pragma unroll
      for (int e = 0; e < PER; ++e) acc[e] += src[e] * w;
    }
  }
  const int tok = fr / G, hq = g * G + fr % G;
  const float inv = l > 0.f ? 1.f / l : 0.f;
  if (o) {
    bf16* dst = o + ((size_t)tok * Hq + hq) * D + lane * PER;
#pragma unroll
    for (int e = 0; e < PER; e += 2) *reinterpret_cast<uint32_t*>(dst + e) = pack2(acc[e] * inv, acc[e + 1] * inv);
  }
  if (lse && lane == 0) lse[(size_t)tok * Hq + hq] = l > 0.f ? (m + log2f(l)) * ATC_LN2 : -INFINITY;
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn2)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static int make_cache_tmap(CUtensorMap* map, const void* ptr, long long rows, long long cols) {
  static EncodeTiledFn2 fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess || qres != cudaDriverEntryPointSuccess)
      return A3_ECUDA;
    fn = (EncodeTiledFn2)p;
  }
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)ATC_BN};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda_error = (int)r;
    return A3_ECUDA;
  }
  return A3_OK;
}

// Key segments of a statistics-only call on nq rows: as many as leave every SM at most one item, within the cap.
static int stats_max_splits(const a3_handle* h, int nq) {
  const int Hkv = h->m.n_kv_heads, G = h->m.n_q_heads / Hkv;
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
  const long long row_tiles = cdiv((long long)(nq > 0 ? nq : 1) * G, ATC_BM);
  const long long per_split = row_tiles * ATC_BM * Hkv * (long long)sizeof(float2);
  long long s = sms / (row_tiles * Hkv);
  if (s > (long long)(STATS_PART_CAP / per_split)) s = (long long)(STATS_PART_CAP / per_split);
  return s < 2 ? 1 : (int)s;
}
size_t stats_part_bytes(const a3_handle* h, int nq) {
  const int Hkv = h->m.n_kv_heads, G = h->m.n_q_heads / Hkv;
  const int s = stats_max_splits(h, nq);
  if (s < 2) return 0;
  return (size_t)s * cdiv((long long)(nq > 0 ? nq : 1) * G, ATC_BM) * ATC_BM * Hkv * sizeof(float2);
}

size_t attention_part_bytes(const a3_handle* h) {
  // split only happens when the unsplit grid has fewer than two CTAs per SM; up to 4 segments
  const size_t rows = (size_t)2 * (h->sm_count > 0 ? h->sm_count : 148) * ATC_BM;
  return 4 * rows * ((size_t)h->m.head_dim + 2) * sizeof(float);
}

int attention_rows(const a3_handle* h, const bf16* q, const int32_t* pos, int M, const bf16* k, const bf16* v,
                      int kv_len, bf16* o, float* lse, void* part, size_t part_bytes, cudaStream_t st) {
  if (M <= 0) return A3_OK;
  const int Hq = h->m.n_q_heads, Hkv = h->m.n_kv_heads, D = h->m.head_dim;
  const int G = Hq / Hkv;
  CUtensorMap tK, tV;
  A3_TRY(make_cache_tmap(&tK, k, kv_len, (long long)Hkv * D));
  A3_TRY(make_cache_tmap(&tV, v, kv_len, (long long)Hkv * D));
  dim3 grid(cdiv((long long)M * G, ATC_BM), Hkv);
  const float scale_log2 = ATC_LOG2E / sqrtf((float)D);
  {
    // many row tiles: two per CTA (a3_attention_pair.cu); few: one per CTA, where the longest item sets the time
    const int sms_ = h->sm_count > 0 ? h->sm_count : 148;
    const int pair_items = (((int)grid.x + 1) / 2) * Hkv;
    const bool use_pair = h->opt[A3_OPT_ATTN_PAIR] < 0 ? pair_items >= 2 * sms_ : h->opt[A3_OPT_ATTN_PAIR] > 0;
    if (use_pair && o && D == 128) {
      const int s = attention_rows_pair(h, tK, tV, q, pos, M, kv_len, o, lse, st);
      if (s != A3_EUNSUPPORTED) return s;
    }
  }
  // split over the keys when the grid would leave SMs idle behind a few long row tiles
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
  const int base_ctas = (int)grid.x * Hkv, all_tiles = cdiv(kv_len, ATC_BN);
  int n_split = 1;
  if (o && part && base_ctas < 2 * sms && all_tiles >= 8) {
    n_split = h->opt[A3_OPT_ATTN_SPLIT] > 0 ? h->opt[A3_OPT_ATTN_SPLIT] : 1;  // measured: with the persistent schedule no split beats 2..4 segments (7 us per item)
    const size_t need = (size_t)n_split * base_ctas * ATC_BM * ((size_t)D + 2) * sizeof(float);
    if (need > part_bytes) n_split = 1;
  }
  if (!o && part && all_tiles >= 2) {
    // statistics only (the question rows' log-sum-exps before the score pass): a handful of row tiles, so the keys are
    // split over the SMs; partial (reference, sum) pairs only, merged in segment order by the combine kernel
    n_split = stats_max_splits(h, M);
    if (n_split > all_tiles) n_split = all_tiles;
    if ((size_t)n_split * base_ctas * ATC_BM * sizeof(float2) > part_bytes) n_split = 1;
  }
  const int tiles_per_split = cdiv(all_tiles, n_split);
  n_split = cdiv(all_tiles, tiles_per_split);
  const int rows_pad = (int)grid.x * ATC_BM;
  const int n_items = (int)grid.x * Hkv * n_split;
  int n_ctas = n_items < sms ? n_items : sms;  // persistent: at most one CTA per SM
  if (h->opt[A3_OPT_ATTN_MAX_CTAS] > 0 && n_ctas > h->opt[A3_OPT_ATTN_MAX_CTAS]) n_ctas = h->opt[A3_OPT_ATTN_MAX_CTAS];
  float* part_o = (float*)part;
  float2* part_ml = !part ? nullptr : !o ? (float2*)part : (float2*)(part_o + (size_t)n_split * Hkv * rows_pad * D);
  static SmemAttrOnce attr128, attr64;
  if (D == 128) A3_TRY(smem_attr_once(attr128, h->device, attention_tc_kernel<128>, AtcLayout<128>::SMEM_BYTES));
  else A3_TRY(smem_attr_once(attr64, h->device, attention_tc_kernel<64>, AtcLayout<64>::SMEM_BYTES));
  ProfScope prof(h, A3_K_ATTENTION, st);
  if (D == 128)
    A3_CUDA(launch_pdl(attention_tc_kernel<128>, dim3(n_ctas), dim3(ATC_THREADS), (size_t)AtcLayout<128>::SMEM_BYTES, st, tK, tV, q, pos, M, kv_len, o,
                       lse, Hq, Hkv, scale_log2, h->dev_status, n_split, tiles_per_split, part_o, part_ml));
  else
    A3_CUDA(launch_pdl(attention_tc_kernel<64>, dim3(n_ctas), dim3(ATC_THREADS), (size_t)AtcLayout<64>::SMEM_BYTES, st, tK, tV, q, pos, M, kv_len, o,
                       lse, Hq, Hkv, scale_log2, h->dev_status, n_split, tiles_per_split, part_o, part_ml));
  A3_LAUNCHED();
  if (n_split > 1) {
    dim3 cgrid(cdiv((long long)M * G, 4), Hkv);
    if (D == 128) attention_combine_kernel<128><<<cgrid, 128, 0, st>>>(pos, M, kv_len, Hq, Hkv, tiles_per_split, rows_pad, part_o, part_ml, o, lse);
    else attention_combine_kernel<64><<<cgrid, 128, 0, st>>>(pos, M, kv_len, Hq, Hkv, tiles_per_split, rows_pad, part_o, part_ml, o, lse);
    A3_LAUNCHED();
  }
  return A3_OK;
}

}  // namespace a3


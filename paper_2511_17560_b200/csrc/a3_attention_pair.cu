// Attention of the carried rows (Eq. 4, Eq. 5) for launches with many row tiles: TWO row tiles per CTA.
//
// The kernel in a3_attention.cu walks one 128-row tile per CTA and is paced by its softmax warps: while they work
// the tensor core waits, and the other way round.  Here a CTA takes two adjacent row tiles A and B of one KV head.
// Every K/V tile is loaded once for both, and the tensor pipe alternates between them, so one tile's softmax runs
// under the other's MMAs:
//
//   warp 0 (one lane)   TMA producer: K and V tiles, two stages each
//   warps 1 and 10      (one lane each; warp 1 row tile A, warp 10 row tile B: one thread cannot issue the 24
//                       instructions per key tile and row tile fast enough for both) tcgen05.mma: S_A = Q_A K^T, S_B = Q_B K^T, O_A += P_A V, O_B += P_B V, everything in halves
//                       of 64 keys.  P of a half is read from tensor memory, where it lies over the first 32 columns
//                       of that half's own logits; a half's P V is issued as soon as its P is stored, and right
//                       behind it the same half of S_X for the NEXT key tile (those columns are free from then on),
//                       so the softmax warps find their next logits waiting: the first half of tile t+1 is computed
//                       under the softmax of the second half of tile t, the second half under that of the first
//   warps 2..5          softmax of row tile A, one thread per row (exponent reference, row sum, rescale as in
//                       a3_attention.cu; the 128 logits of a row are taken in two halves of 64)
//   warps 6..9          the same for row tile B
// Tensor memory (512 columns): S_A at 0 (keys 0..63 in columns 0..63, keys 64..127 in 64..127), S_B at 128, O_A at 256,
// O_B at 384.  Head dimension 128 only; rows sorted
// by position, so B (the later rows) sees at least as many key tiles as A.  Every wait is bounded.
#include <cuda.h>

#include "a3_internal.cuh"
#include "a3_attn.cuh"

namespace a3 {

constexpr int AT2_THREADS = 352;  // warp 0 TMA, warp 1 MMA of row tile A, warps 2..9 softmax, warp 10 MMA of row tile B
constexpr int AT2_D = 128;

struct At2Layout {
  static constexpr int SUB = 128 * 64 * 2;  // one [128][64] bf16 sub-tile: 16 KiB
  static constexpr int TILE = 2 * SUB;      // a [128][128] bf16 tile
  static constexpr int Q_OFF = 0;           // Q_A, Q_B
  static constexpr int K_OFF = 2 * TILE;    // two stages
  static constexpr int V_OFF = 4 * TILE;    // two stages
  static constexpr int BAR_OFF = 6 * TILE;
  static constexpr int SMEM_BYTES = BAR_OFF + 256;
};

struct At2Item {
  int g;
  int r0[2], maxpos[2], minpos[2], nkt[2];
  int T;  // key tiles to walk: max of the two
};

// Items: row-tile pairs from the last (longest) to the first, KV heads innermost.
__device__ __forceinline__ At2Item at2_item(int i, const int32_t* __restrict__ pos, int M, int G, int Hkv, int kv_len, int row_tiles,
                                            int n_pairs) {
  At2Item w;
  const int pair = n_pairs - 1 - i / Hkv;
  w.g = i % Hkv;
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    const int tile = 2 * pair + x;
    w.r0[x] = tile * ATC_BM;
    if (tile < row_tiles) {
      const int last_tok = min(M - 1, (w.r0[x] + ATC_BM - 1) / G);
      w.maxpos[x] = min(pos[last_tok], kv_len - 1);
      w.minpos[x] = pos[w.r0[x] / G];
      w.nkt[x] = w.maxpos[x] < 0 ? 0 : w.maxpos[x] / ATC_BN + 1;
    } else {
      w.maxpos[x] = -1;
      w.minpos[x] = 0;
      w.nkt[x] = 0;
    }
  }
  w.T = max(w.nkt[0], w.nkt[1]);
  return w;
}

__global__ void __launch_bounds__(AT2_THREADS, 1)
attention_pair_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                      const bf16* __restrict__ q, const int32_t* __restrict__ pos, int M, int kv_len, bf16* __restrict__ o,
                      float* __restrict__ lse, int Hq, int Hkv, float scale_log2, uint32_t* status) {
  using L = At2Layout;
  using namespace atc;
  constexpr int D = AT2_D;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* base_ptr = smem_raw;
  if (base & 1023u) {  // the swizzled tiles need a 1024-byte aligned window; uniform for the CTA, nothing is set up yet
    if (threadIdx.x == 0) atomicOr(status, A3_DEV_WAIT_EXHAUSTED);
    return;
  }
  const uint32_t bars = base + L::BAR_OFF;
  auto k_full = [&](int s) { return bars + 8u * s; };
  auto k_empty = [&](int s) { return bars + 8u * (2 + s); };
  auto v_full = [&](int s) { return bars + 8u * (4 + s); };
  auto v_empty = [&](int s) { return bars + 8u * (6 + s); };
  auto s_full = [&](int x, int hh) { return bars + 8u * (hh == 0 ? 8 + x : 19 + x); };  // logits of half hh of S_X are in tensor memory
  auto p_ready = [&](int x) { return bars + 8u * (10 + x); };
  auto pv_done = [&](int x) { return bars + 8u * (12 + x); };
  const uint32_t q_ready = bars + 8u * 14;
  auto p0_ready = [&](int x) { return bars + 8u * (15 + x); };  // P of the first 64 keys is in tensor memory
  auto pv0_done = [&](int x) { return bars + 8u * (17 + x); };  // ... and its P V has completed
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::BAR_OFF + 8 * 21);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::BAR_OFF + 8 * 21 + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = Hq / Hkv;
  const int rows_total = M * G;
  const int row_tiles = (rows_total + ATC_BM - 1) / ATC_BM;
  const int n_pairs = (row_tiles + 1) / 2;
  const int n_items = n_pairs * Hkv;
  const int C = gridDim.x, cta = blockIdx.x;
  auto item_index = [&](int r) {
    const int i = r * C + ((r & 1) ? C - 1 - cta : cta);
    return i < n_items ? i : -1;
  };
  const int rounds = (n_items + C - 1) / C;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(k_full(i), 1);
      mbar_init(k_empty(i), 2);  // one arrival per MMA thread
      mbar_init(v_full(i), 1);
      mbar_init(v_empty(i), 2);
      mbar_init(s_full(i, 0), 1);
      mbar_init(s_full(i, 1), 1);
      mbar_init(p_ready(i), 128);
      mbar_init(pv_done(i), 1);
      mbar_init(p0_ready(i), 128);
      mbar_init(pv0_done(i), 1);
    }
    mbar_init(q_ready, 256);
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
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    // ---------------- TMA producer: K(t) then V(t) of every key tile the item walks
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmV) : "memory");
      uint32_t it = 0;
      bool ok = true;
      for (int r = 0; r < rounds && ok; ++r) {
        const int i = item_index(r);
        if (i < 0) continue;
        const At2Item w = at2_item(i, pos, M, G, Hkv, kv_len, row_tiles, n_pairs);
        for (int t = 0; t < w.T; ++t, ++it) {
          const int s = it & 1;
          const uint32_t ph = (it >> 1) & 1;
          ok = mbar_wait(k_empty(s), ph ^ 1, abort_flag, status);
          if (!ok) break;
          mbar_expect_tx(k_full(s), L::TILE);
          tma_load_2d(base + L::K_OFF + s * L::TILE, &tmK, w.g * D, t * ATC_BN, k_full(s));
          tma_load_2d(base + L::K_OFF + s * L::TILE + L::SUB, &tmK, w.g * D + 64, t * ATC_BN, k_full(s));
          ok = mbar_wait(v_empty(s), ph ^ 1, abort_flag, status);
          if (!ok) break;
          mbar_expect_tx(v_full(s), L::TILE);
          tma_load_2d(base + L::V_OFF + s * L::TILE, &tmV, w.g * D, t * ATC_BN, v_full(s));
          tma_load_2d(base + L::V_OFF + s * L::TILE + L::SUB, &tmV, w.g * D + 64, t * ATC_BN, v_full(s));
        }
      }
    }
  } else if (warp == 1 || warp == 10) {
    // ---------------- MMA issuers: this thread owns row tile x; K and V stages are released by both threads
    if (lane == 0) {
      const int x = warp == 1 ? 0 : 1;
      constexpr uint32_t idesc_s = idesc(ATC_BN / 2, 0);
      constexpr uint32_t idesc_o = idesc(D, 1);
      uint32_t it = 0, qn = 0, cx = 0;  // running key tile; items; tiles this row tile has done (barrier phases)
      // logits of 64 keys (half hh of the key tile in K stage `kstage`)
      auto issue_s = [&](int hh, uint32_t kstage) {
        const uint32_t sq = base + L::Q_OFF + x * L::TILE, sk = base + L::K_OFF + kstage * L::TILE + hh * (64 * 128);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t sub = (k / 4) * L::SUB + (k % 4) * 32;
          mma_f16(tmem_base + x * 128 + hh * 64, desc_k_sw128(sq + sub), desc_k_sw128(sk + sub), idesc_s, k != 0);
        }
        commit(s_full(x, hh));
      };
      // P V of 64 keys: P of half hh lies over the first 32 columns of that half of S_X
      auto issue_pv_half = [&](int hh, uint32_t vstage, bool first) {
        const uint32_t sv = base + L::V_OFF + vstage * L::TILE;
#pragma unroll
        for (int k = 4 * hh; k < 4 * hh + 4; ++k) {
          const uint64_t db = desc_mn_sw128(sv + k * 16 * 128, L::SUB);
          mma_f16_ts(tmem_base + 256 + x * 128, tmem_base + x * 128 + hh * 64 + (k - 4 * hh) * 8, db, idesc_o, !(first && k == 0));
        }
        commit(hh == 0 ? pv0_done(x) : pv_done(x));
      };
      bool ok = true;
      for (int r = 0; r < rounds && ok; ++r) {
        const int i = item_index(r);
        if (i < 0) continue;
        const At2Item w = at2_item(i, pos, M, G, Hkv, kv_len, row_tiles, n_pairs);
        const int nkt = w.nkt[x];
        ok = mbar_wait(q_ready, qn & 1, abort_flag, status);
        ++qn;
        if (!ok) break;
        if (w.T == 0) continue;
        ok = mbar_wait(k_full(it & 1), (it >> 1) & 1, abort_flag, status);
        if (!ok) break;
        fence_after();
        if (nkt > 0) {
          issue_s(0, it & 1);
          issue_s(1, it & 1);
          commit(k_empty(it & 1));
        } else {
          mbar_arrive(k_empty(it & 1));
        }
        for (int t = 0; t < w.T && ok; ++t, ++it) {
          const bool more = t + 1 < w.T;
          const uint32_t vs = it & 1, vph = (it >> 1) & 1, kn = (it + 1) & 1, kph = ((it + 1) >> 1) & 1;
          if (t < nkt) {
            const bool next = t + 1 < nkt;
            // halves in key order.  Each P V is followed by the same half of the next key tile's logits: P V has read
            // the columns they go to, and the pipe runs this thread's instructions in order.
            ok = mbar_wait(p0_ready(x), cx & 1, abort_flag, status) && mbar_wait(v_full(vs), vph, abort_flag, status);
            if (!ok) break;
            fence_after();
            issue_pv_half(0, vs, t == 0);
            if (next) {
              ok = mbar_wait(k_full(kn), kph, abort_flag, status);
              if (!ok) break;
              fence_after();
              issue_s(0, kn);
            }
            ok = mbar_wait(p_ready(x), cx & 1, abort_flag, status);
            if (!ok) break;
            fence_after();
            issue_pv_half(1, vs, t == 0);
            if (next) issue_s(1, kn);
            ++cx;
            commit(v_empty(vs));
            if (more) {
              if (next) {
                commit(k_empty(kn));
              } else {
                // this row tile is done, the other walks on: its stages still need this thread's arrival, and an
                // arrival must not run ahead of the stage's use (it would be counted in the wrong phase): wait
                // until the tile has landed
                ok = mbar_wait(k_full(kn), kph, abort_flag, status);
                if (!ok) break;
                mbar_arrive(k_empty(kn));
              }
            }
          } else {
            ok = mbar_wait(v_full(vs), vph, abort_flag, status);
            if (!ok) break;
            mbar_arrive(v_empty(vs));
            if (more) {
              ok = mbar_wait(k_full(kn), kph, abort_flag, status);
              if (!ok) break;
              mbar_arrive(k_empty(kn));
            }
          }
        }
      }
    }
  } else {
    // ---------------- softmax / epilogue: warps 2..5 row tile A, warps 6..9 row tile B, one thread per row
    const int x = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t ts = tmem_base + x * 128 + lane_addr;        // this row of S_X (P_X over its first 64 columns)
    const uint32_t to = tmem_base + 256 + x * 128 + lane_addr;  // this row of O_X
    constexpr float OVERFLOW_GUARD = 65536.f;
    uint32_t it = 0, cxx = 0;  // running key tile of the CTA; tiles this row tile has done (barrier phases)
    bool ok = true;

    for (int r = 0; r < rounds && ok; ++r) {
      const int i = item_index(r);
      if (i < 0) continue;
      const At2Item w = at2_item(i, pos, M, G, Hkv, kv_len, row_tiles, n_pairs);
      const int fr = w.r0[x] + row;
      const bool row_ok = fr < rows_total;
      const int tok = row_ok ? fr / G : 0;
      const int hq = w.g * G + (row_ok ? fr % G : 0);
      const int lim = row_ok ? min(pos[tok], kv_len - 1) : -1;
      const int nkt = w.nkt[x];

      // Q row -> shared memory, swizzled K-major sub-tiles.  The previous item's S_X MMAs have all completed (their
      // last s_full was waited for), so the buffer is free.  Every thread arrives, also when its row tile is empty.
      {
        const uint4* src = reinterpret_cast<const uint4*>(q + ((size_t)tok * Hq + hq) * D);
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
          const uint4 v = (row_ok && nkt > 0) ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
          *reinterpret_cast<uint4*>(base_ptr + L::Q_OFF + x * L::TILE + (c / 8) * L::SUB + swz(row, c % 8)) = v;
        }
        fence_async_smem();
        mbar_arrive(q_ready);
      }
      if (nkt == 0) {
        // no visible key (row tile beyond the rows, or invalid positions): defined output, no pipeline work
        if (row_ok) {
          uint4* dst = reinterpret_cast<uint4*>(o + ((size_t)tok * Hq + hq) * D);
#pragma unroll
          for (int c = 0; c < D / 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
          if (lse) lse[(size_t)tok * Hq + hq] = -INFINITY;
        }
        it += w.T;
        continue;
      }

      float m_ref = 0.f, l_run = 0.f;
      for (int t = 0; t < nkt; ++t, ++cxx) {
        // the result of every wait is made warp-uniform: tcgen05.ld/st are warp-wide instructions
        ok = __all_sync(0xffffffffu, mbar_wait(s_full(x, 0), cxx & 1, abort_flag, status));
        if (!ok) break;
        fence_after();  // the first half of the logits is there (and the first-half P V of the previous key tile is complete)
        const int key0 = t * ATC_BN;
        const bool need_mask = key0 + ATC_BN - 1 > w.minpos[x];
        float xv[64];
        auto row_max64 = [&](int kbase) {  // maximum of the scaled, masked logits in xv
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int e = 0; e < 64; ++e) {
            const float v = (need_mask && kbase + e > lim) ? -INFINITY : xv[e] * scale_log2;
            m4[e & 3] = fmaxf(m4[e & 3], v);
          }
          return fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        };
        auto to_probabilities = [&](int kbase) {  // xv <- exp2(xv * scale - m_ref); returns the sum
          float ls[4] = {0.f, 0.f, 0.f, 0.f};
          const float neg_ref = -m_ref;
          if (need_mask) {
#pragma unroll
            for (int e = 0; e < 64; ++e) {
              float v = fmaf(xv[e], scale_log2, neg_ref);
              if (kbase + e > lim) v = -INFINITY;
              xv[e] = ex2_approx(v);
              ls[e & 3] += xv[e];
            }
          } else {
            const float2 sc2 = make_float2(scale_log2, scale_log2), nr2 = make_float2(neg_ref, neg_ref);
            float2 s2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int e = 0; e < 64; e += 2) {
              const float2 v = __ffma2_rn(make_float2(xv[e], xv[e + 1]), sc2, nr2);
              if (ATC_POLY_EVERY > 0 && ((e >> 1) % ATC_POLY_EVERY) == ATC_POLY_EVERY - 1) {
                // on the FMA pipe: with both row tiles' softmax running all the time the exponential unit (16 results
                // per clock and SM = 2 048 clocks per key tile) is the bound
                const float2 p2 = exp2_poly2(v);
                xv[e] = p2.x;
                xv[e + 1] = p2.y;
              } else {
                xv[e] = ex2_approx(v.x);
                xv[e + 1] = ex2_approx(v.y);
              }
              s2[(e >> 1) & 1] = __fadd2_rn(s2[(e >> 1) & 1], make_float2(xv[e], xv[e + 1]));
            }
            ls[0] = s2[0].x, ls[1] = s2[0].y, ls[2] = s2[1].x, ls[3] = s2[1].y;
          }
          return (ls[0] + ls[1]) + (ls[2] + ls[3]);
        };
        auto load64 = [&](int h) {
          ld32(ts + h * 64, xv);
          ld32(ts + h * 64 + 32, xv + 32);
          wait_ld();
        };
        // multiplies this row of O_X by f (the caller has waited for every P V issued so far)
        auto rescale_output = [&](float f) {
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            float tv[32];
            ld32(to + c * 32, tv);
            wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) tv[e] *= f;
            st32(to + c * 32, tv);
          }
          wait_st();
        };
        if (t == 0) {
          // the reference is the true maximum of the first tile
          ok = __all_sync(0xffffffffu, mbar_wait(s_full(x, 1), cxx & 1, abort_flag, status));
          if (!ok) break;
          fence_after();
          load64(0);
          float mx = row_max64(key0);
          load64(1);
          mx = fmaxf(mx, row_max64(key0 + 64));
          m_ref = mx == -INFINITY ? 0.f : mx;
        }
        // Slots beyond the last visible key of the pair may hold anything (probability zero times a non-finite
        // value would still poison the product): clear those V rows of the last key tile before the first P V that
        // reads it - row tile A does it when it walks to the last tile (its P V is issued first), else B.
        if (t == w.T - 1 && x == (w.nkt[0] == w.T ? 0 : 1)) {
          const int first_bad = max(w.maxpos[0], w.maxpos[1]) - key0 + 1;
          const uint32_t vit = it + t;
          const bool landed = mbar_wait(v_full(vit & 1), (vit >> 1) & 1, abort_flag, status);
          if (landed && row >= first_bad) {
            unsigned char* sv = base_ptr + L::V_OFF + (vit & 1) * L::TILE;
#pragma unroll
            for (int j = 0; j < D / 64; ++j)
#pragma unroll
              for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(sv + j * L::SUB + row * 128 + c * 16) = make_uint4(0, 0, 0, 0);
          }
          fence_async_smem();
        }
        float l_tile = 0.f;
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
          if (h == 1) {
            // the second half of the logits (issued behind the second-half P V of the previous key tile)
            ok = __all_sync(0xffffffffu, mbar_wait(s_full(x, 1), cxx & 1, abort_flag, status));
            if (!ok) break;
            fence_after();
          }
          load64(h);
          float lsum = to_probabilities(key0 + 64 * h);
          // A logit far above the reference shows in the sum; anything below 2^16 is harmless.  Above it - rare -
          // the reference goes up to this half's maximum, and what was accumulated under the old one is rescaled:
          // the row sums and the output (which, in the second half, includes the first half's P V: see below).
          if (t > 0 && __any_sync(0xffffffffu, !(lsum <= OVERFLOW_GUARD))) {
            load64(h);
            const float mx = row_max64(key0 + 64 * h);
            const float raise = fmaxf(mx - m_ref, 0.f);
            const float f = exp2f(-raise);
            m_ref += raise;
            l_run *= f;
            l_tile *= f;
            // Every P V issued so far must have landed in the output before it is rescaled.  In the first half the
            // last one is the second-half P V of the previous key tile; in the second half it is this tile's
            // first-half P V, released under the old reference: once it has completed, the output holds its
            // contribution too and the factor applies to all of it.  (Older ones are complete: the pipe runs in order.)
            ok = __all_sync(0xffffffffu, h == 1 ? mbar_wait(pv0_done(x), cxx & 1, abort_flag, status)
                                                : mbar_wait(pv_done(x), (cxx - 1) & 1, abort_flag, status));
            if (!ok) break;
            fence_after();
            rescale_output(f);
            load64(h);
            lsum = to_probabilities(key0 + 64 * h);
          }
          l_tile += lsum;
          // P of this half as bf16 pairs: the first 32 columns of this half of S_X (its logits are in registers)
          uint32_t pk[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 v = pack8(xv + 8 * j);
            pk[4 * j] = v.x, pk[4 * j + 1] = v.y, pk[4 * j + 2] = v.z, pk[4 * j + 3] = v.w;
          }
          st32(ts + 64 * h, reinterpret_cast<const float*>(pk));
          if (h == 0) {
            wait_st();
            fence_before();
            mbar_arrive(p0_ready(x));
          }
        }
        if (!ok) break;
        wait_st();
        l_run += l_tile;
        fence_before();
        mbar_arrive(p_ready(x));
      }
      if (!ok) break;
      it += w.T;
      // the last P V of this row tile
      ok = __all_sync(0xffffffffu, mbar_wait(pv_done(x), (cxx - 1) & 1, abort_flag, status));
      if (!ok) break;
      fence_after();
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      bf16* dst = o + ((size_t)tok * Hq + hq) * D;
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        float tv[32];
        ld32(to + c * 32, tv);
        wait_ld();
        if (row_ok) {
#pragma unroll
          for (int e = 0; e < 32; ++e) tv[e] *= inv;
#pragma unroll
          for (int j = 0; j < 4; ++j) reinterpret_cast<uint4*>(dst + c * 32)[j] = pack8(tv + 8 * j);
        }
        __syncwarp();
      }
      fence_before();
      if (row_ok && lse) lse[(size_t)tok * Hq + hq] = l_run > 0.f ? (m_ref + log2f(l_run)) * ATC_LN2 : -INFINITY;
    }
  }
  atc::fence_before();
  __syncthreads();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

int attention_rows_pair(const a3_handle* h, const CUtensorMap& tK, const CUtensorMap& tV, const bf16* q, const int32_t* pos, int M,
                        int kv_len, bf16* o, float* lse, cudaStream_t st) {
  const int Hq = h->m.n_q_heads, Hkv = h->m.n_kv_heads, D = h->m.head_dim;
  if (D != AT2_D || !o) return A3_EUNSUPPORTED;
  const int G = Hq / Hkv;
  const int row_tiles = cdiv((long long)M * G, ATC_BM);
  const int n_items = ((row_tiles + 1) / 2) * Hkv;
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
  const int n_ctas = n_items < sms ? n_items : sms;
  const float scale_log2 = ATC_LOG2E / sqrtf((float)D);
  static SmemAttrOnce attr;
  A3_TRY(smem_attr_once(attr, h->device, attention_pair_kernel, At2Layout::SMEM_BYTES));
  ProfScope prof(h, A3_K_ATTENTION, st);
  A3_CUDA(launch_pdl(attention_pair_kernel, dim3(n_ctas), dim3(AT2_THREADS), (size_t)At2Layout::SMEM_BYTES, st, tK, tV, q, pos, M, kv_len, o, lse,
                     Hq, Hkv, scale_log2, h->dev_status));
  A3_LAUNCHED();
  return A3_OK;
}

}  // namespace a3

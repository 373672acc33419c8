// Persistent CTA-pair GEMMs of the recompute path (the feed-forward part of H(.) in Eq. 5) with the operand roles
// swapped:   SwiGLU    out[t][f] = silu(x[t] . Wg[f]) * (x[t] . Wu[f])
//            residual  C[t][f] += x[t] . W[f]            (output projection, MLP down projection)
//
// Why another kernel.  With one CTA per 128-token x 256-column tile an SM pulls 48 KiB per k-block through its L2
// port and that, not the tensor pipe, sets the pace (a wave's time follows the bytes: about 107 GB/s per SM with
// 192 KiB in flight); at 804 tokens the 128-row tiles also pad the rows to 896 and the grid to three waves.  Here
//   * the WEIGHTS are the M-side operand of tcgen05.mma.cta_group::2 (M = 256 over a CTA pair).  SwiGLU: each CTA
//     holds 64 gate rows and 64 up rows of the same 64 features (its 128 accumulator lanes), so gate and up of a
//     feature meet inside one CTA; residual: 128 rows of the one matrix;
//   * the TOKENS are the N-side operand, in tiles of N <= 256 tokens chosen to divide the row count evenly
//     (804 rows -> 4 x 208: 3 % padding instead of 11 %); each CTA loads half of the token tile, the instruction
//     reads both halves.  Per k-block an SM pulls 16 KiB of weights + N/2 token rows (13 KiB at N = 208);
//   * the kernel is persistent: CTA pair p walks units p, p + pairs, ... (unit = 128 (SwiGLU) or 256 features x one
//     token tile), accumulators are double-buffered in tensor memory (2 x N <= 512 columns), so the epilogue of a
//     unit runs under the main loop of the next one; a ring stage holds two k-blocks (one barrier hand-shake and one
//     commit per eight instructions: the single issuing thread, not the pipe, was the limit with one).
// SwiGLU epilogue: the two halves meet through shared memory (see below); a warp writes 32 consecutive features of
// one token (64 bytes) per instruction.  Measured at Llama-8B width: tensor pipe 97 % active at 5 152 rows.
// No load uses cluster multicast.  Every wait is bounded (see a3_tc.cuh): a waiter that gives up raises the CTA's
// abort flag and the device status bit, all roles leave their loops, tensor memory is released and the CTA returns.
#include <cuda.h>

#include "a3_internal.cuh"
#include "a3_tc.cuh"

namespace a3 {

constexpr int SP_THREADS = 320;  // warp 0: TMA, warp 1: MMA (leader CTA), warps 2..9: epilogue (two sets of four)
constexpr int SP_MAX_STAGES = 8;
constexpr int SP_SUB = 2;  // k-blocks of 64 per ring stage: one barrier hand-shake and one commit per 8 MMAs
constexpr int SP_FEAT = 64;                              // features per CTA (64 gate lanes + 64 up lanes)
constexpr int SP_A_BYTES = 2 * SP_FEAT * TC_BK * 2;      // 16 KiB: gate rows, then up rows
constexpr int SP_XCH_BYTES = 2 * 2 * 32 * SP_FEAT * 4;   // per warp set: two buffers of float [32 tokens][64 features]
constexpr int SP_QKV_SET_FLOATS = 4 * (32 * 32 + 4);            // QKV: per warp set, four quarters of [32 tokens][32 features] fp32, 16 bytes apart in the banks
constexpr int SP_QKV_XCH_BYTES = 2 * SP_QKV_SET_FLOATS * 4 + 128;  // + room to keep the next field 256-byte aligned
constexpr int SP_QKV_EXTRA = SP_QKV_XCH_BYTES + 256;              // ... and the checked positions of a chunk's tokens per set
constexpr int SP_SMEM_LIMIT = 227 * 1024;

struct SpParams {
  int M, K, F;
  int tok_tiles, tok_n;  // token tiles and tokens per tile (multiple of 16, at most 256)
  int n_fblocks;         // feature blocks (one per CTA pair and unit): units = n_fblocks x tok_tiles
  int group;             // feature blocks per group of the unit order (1: feature blocks outermost)
  int n_units, n_pairs;
  int stages, stage_bytes, sub_bytes;  // ring depth; bytes per stage = SP_SUB x sub_bytes (A + this CTA's half of the token tile for one k-block, 1024-byte multiple)
  bf16* C;
  int ldc;
  uint32_t* status;
  // EPI_QKV: the concatenated heads of up to three matrices (q, k, v in any subset), 128 features each
  int n_heads;
  int seg_heads_end[3];  // cumulative head counts of the segments
  int kind[3];           // 0 = q, 1 = k, 2 = v
  const bf16* bias[3];
  bf16 *q_out, *k_cache, *v_cache;
  const int32_t* pos;
  int kv_len, Hq, Hkv, layout, max_pos;
  const float2* tab;
};

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int threads) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// arrives on the barrier at the same shared-memory offset in CTA `cta` of the cluster
__device__ __forceinline__ void mbar_arrive_in_cta(uint32_t bar, uint32_t cta) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(bar), "r"(cta));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
// w (8, 16, 24 or 32; uniform for the warp) consecutive accumulator columns of this thread's lane
__device__ __forceinline__ void sp_ld_chunk(uint32_t taddr, int w, float* v) {
  if (w == 32) {
    tc_ld32(taddr, v);
  } else {  // static register indices: the array must not go to local memory
    if (w >= 8) tc_ld8(taddr, v);
    if (w >= 16) tc_ld8(taddr + 8, v + 8);
    if (w >= 24) tc_ld8(taddr + 16, v + 16);
  }
  tc_wait_ld();
}

// Unit u -> (feature block, token tile).  Units are numbered in groups of `group` feature blocks, token tiles next,
// the group's blocks innermost.  With group = 8 the 74 pairs that work side by side cover about 8 feature blocks x 9
// token tiles, and since they walk the k-blocks at the same pace, what a round pulls through L2 is 8 weight blocks +
// 9 token tiles: the order for token matrices that do not fit in L2 (with feature blocks outermost a round of the
// 32 800-row QKV launch pulled 1 weight block + 74 token tiles: 6.9 GB of DRAM reads for 0.3 GB of operands).  With
// group = 1 (feature blocks outermost) every round walks all token tiles: the order for token matrices that stay in
// L2, where the weights then stream through exactly once (SwiGLU at 5 152 rows: 418 MB of DRAM reads against 719 MB
// with groups of 8).
__device__ __forceinline__ void sp_unit(int u, int n_fblocks, int tok_tiles, int group, int& fb, int& tt) {
  const int per_group = group * tok_tiles;
  const int g = u / per_group, r = u - g * per_group;
  const int gsz = min(group, n_fblocks - g * group);
  tt = r / gsz;
  fb = g * group + (r - tt * gsz);
}

// D += A B over the CTA pair (accumulating form: no predicate to set up)
__device__ __forceinline__ void tc_mma_pair_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.eq.u32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
      : "memory");
}

// EPI_SWIGLU: tmG/tmU are the gate and up matrices (box of 64 rows each); EPI_RESIDUAL: tmG is the one weight matrix
// (box of 128 rows, tmU unused) and the epilogue adds the accumulator to C in place.
// EPI_QKV: tmG / tmU / tmW are the matrices of the segments (boxes of 128 rows: one head); a unit is two consecutive
// heads of the concatenated list, one per CTA of the pair, times one token tile; the epilogue adds the bias, rotates
// q and k at the tokens' positions (the two halves of a rotation pair sit 64 lanes apart and meet through shared
// memory, like gate and up) and writes q to its buffer and k, v into the cache rows pos[token] (the scatter of Eq. 5).
template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(SP_THREADS, 1)
pair_t_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmG,
              const __grid_constant__ CUtensorMap tmU, const __grid_constant__ CUtensorMap tmW, const SpParams p) {
  constexpr int ROWS = EPI == EPI_SWIGLU ? SP_FEAT : 2 * SP_FEAT;  // output features per CTA
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // same offset in both CTAs of the pair
  unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int S = p.stages;
  const int xch_off = S * p.stage_bytes, bar_off = xch_off + (EPI == EPI_SWIGLU ? SP_XCH_BYTES : (EPI == EPI_QKV ? SP_QKV_EXTRA : 0));
  // barriers (8 bytes each): full[8] (used in the leader), empty[8], tmem_full[2], tmem_empty[2] (used in the leader)
  const uint32_t bars = base + bar_off;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (SP_MAX_STAGES + s); };
  auto tmem_full = [&](int b) { return bars + 8u * (2 * SP_MAX_STAGES + b); };
  auto tmem_empty = [&](int b) { return bars + 8u * (2 * SP_MAX_STAGES + 2 + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + bar_off + 8 * (2 * SP_MAX_STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + bar_off + 8 * (2 * SP_MAX_STAGES + 4) + 8);
  volatile int* ep_ok = abort_flag + 2;  // the epilogue's one waiter tells the other 127 threads how its wait ended
  float* xch = reinterpret_cast<float*>(base_ptr + xch_off);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1;
  const int KT = p.K / TC_BK;  // a multiple of SP_SUB (checked by the launcher)
  const int half_n = p.tok_n >> 1;  // token rows this CTA loads per k-block (multiple of 8)
  const uint32_t b_bytes = (uint32_t)half_n * TC_BK * 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tmem_full(b), 1);
      // SwiGLU: the gate warps and the up warps of both warp sets of each CTA; residual and QKV: every epilogue warp
      mbar_init(tmem_empty(b), EPI == EPI_SWIGLU ? 8 : 16);
    }
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ep_ok[0] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // the same warp of both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();  // the peer's barriers exist before anything is signalled on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs): own gate/up rows, own half of the token tile
    if (lane == 0) {
      tmap_prefetch(&tmX);
      tmap_prefetch(&tmG);
      if (EPI == EPI_SWIGLU) tmap_prefetch(&tmU);
      int kbg = 0, issued = 0;
      int s = 0;        // ring position and phase, kept by counting: S is a run-time value and a division per
      uint32_t ph = 0;  // k-block is a long dependent chain in a one-thread role
      bool ok = true;
      if (EPI == EPI_QKV) tmap_prefetch(&tmW);
      for (int u = pair; u < p.n_units && ok; u += p.n_pairs) {
        int fb, tt;
        sp_unit(u, p.n_fblocks, p.tok_tiles, p.group, fb, tt);
        int f0 = fb * (2 * ROWS) + (int)rank * ROWS;
        const CUtensorMap* mapA = &tmG;
        if (EPI == EPI_QKV) {
          // this CTA's head of the concatenated list -> its matrix and first row there (a pair beyond the last head of
          // an odd list loads head 0 again; its epilogue stores nothing)
          int hd = 2 * fb + (int)rank;
          if (hd >= p.n_heads) hd = 0;
          const int sg = (hd >= p.seg_heads_end[0]) + (hd >= p.seg_heads_end[1]);
          f0 = (hd - (sg == 0 ? 0 : p.seg_heads_end[sg - 1])) * 128;
          mapA = sg == 0 ? &tmG : (sg == 1 ? &tmU : &tmW);
        }
        const int t0 = tt * p.tok_n + (int)rank * half_n;
        for (int kb = 0; kb < KT; kb += SP_SUB, ++kbg) {
          if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, p.status)) {
            ok = false;
            break;
          }
          const uint32_t full_leader = full_bar(s) & PAIR_LEADER_MASK;
          // the leader announces the bytes of both CTAs; a copy of the peer that completes earlier cannot end the
          // phase, because the leader's own arrival is still pending until its expect_tx
          if (leader) mbar_expect_tx(full_bar(s), 2 * SP_SUB * (SP_A_BYTES + b_bytes));
#pragma unroll
#pragma unroll
          for (int j = 0; j < SP_SUB; ++j) {
            const uint32_t sa = base + s * p.stage_bytes + j * p.sub_bytes, sb = sa + SP_A_BYTES;
            tma_load_2d_pair(sa, mapA, (kb + j) * TC_BK, f0, full_leader);
            if (EPI == EPI_SWIGLU) tma_load_2d_pair(sa + SP_A_BYTES / 2, &tmU, (kb + j) * TC_BK, f0, full_leader);
            tma_load_2d_pair(sb, &tmX, (kb + j) * TC_BK, t0, full_leader);
          }
          issued = kbg + 1;
          if (++s == S) {
            s = 0;
            ph ^= 1;
          }
        }
      }
      if (*abort_flag) {
        // let the copies already issued land before the CTA can exit (bounded)
        if (leader) {
          for (int k = max(0, issued - S); k < issued; ++k)
            mbar_wait(full_bar(k % S), (k / S) & 1, abort_flag + 1, p.status, 2000000ull);
        } else {
          const unsigned long long t0 = global_ns();
          while (global_ns() - t0 < 200000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: the leader alone, for both CTAs.
    // The tensor pipe queues only about two instructions, so everything this thread does between two of them has
    // to fit into some 200 clocks or the pipe runs dry.  The look at the next stage's barrier therefore happens in
    // the middle of a stage (after its first four instructions), the commit and the ring arithmetic at its end.
    if (lane == 0 && leader) {
      const uint32_t idesc = idesc_bf16_pair(p.tok_n);
      const uint64_t da0 = smem_desc_sw128(base), db0 = smem_desc_sw128(base + SP_A_BYTES);
      // descriptor address fields count 16-byte units: stage and k-step offsets are added to the first stage's
      const uint32_t stage16 = (uint32_t)p.stage_bytes >> 4, sub16 = (uint32_t)p.sub_bytes >> 4;
      const int per_unit = KT / SP_SUB;
      const int my_units = pair < p.n_units ? (p.n_units - pair + p.n_pairs - 1) / p.n_pairs : 0;
      const int total = my_units * per_unit;
      int s = 0, it = 0, in_unit = 0;
      uint32_t ph = 0, stage_off = 0, d = tmem_base;
      bool ok = total > 0, ready = false;
      for (int g = 0; g < total && ok; ++g) {
        if (in_unit == 0) {
          // the epilogues of both CTAs have drained this accumulator (first use: passes at once)
          const int b = it & 1;
          ok = mbar_wait(tmem_empty(b), ((it >> 1) & 1) ^ 1, abort_flag, p.status);
          if (!ok) break;
          d = tmem_base + (uint32_t)b * 256u;
        }
        if (!ready) ok = mbar_wait(full_bar(s), ph, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint64_t da_s = da0 + stage_off, db_s = db0 + stage_off;
        tc_mma_pair_f16(d, da_s, db_s, idesc, in_unit != 0);
#pragma unroll
        for (int k = 1; k < TC_BK / 16; ++k) tc_mma_pair_acc(d, da_s + (uint64_t)(2 * k), db_s + (uint64_t)(2 * k), idesc);
        // next ring position, and one look at its barrier while the pipe works on the instructions above
        int sn = s + 1;
        uint32_t phn = ph, offn = stage_off + stage16;
        if (sn == S) {
          sn = 0;
          phn ^= 1;
          offn = 0;
        }
        ready = g + 1 < total && mbar_try_wait(full_bar(sn), phn);
#pragma unroll
        for (int j = 1; j < SP_SUB; ++j) {
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k) {
            const uint64_t koff = (uint64_t)(j * sub16 + 2 * k);
            tc_mma_pair_acc(d, da_s + koff, db_s + koff, idesc);
          }
        }
        tc_commit_pair(empty_bar(s), 3);  // frees this stage in both CTAs once the instructions above have read it
        if (++in_unit == per_unit) {
          tc_commit_pair(tmem_full(it & 1), 3);  // publishes the accumulator in both CTAs
          in_unit = 0;
          ++it;
        }
        s = sn;
        ph = phn;
        stage_off = offn;
      }
    }
  } else if (EPI == EPI_SWIGLU) {
    // ---------------- epilogue: warps 2..9 of both CTAs; warp w may touch TMEM lanes 32*(w%4) .. +31.
    // Lanes 0..63 hold the gate rows of this CTA's 64 features, lanes 64..127 their up rows.  Warp set 0 (warps
    // 2..5) takes the first half of the token columns, set 1 (warps 6..9) the second.  Inside a set the two halves of
    // silu(g) * u meet through shared memory, 32 tokens at a time, in two buffers: on even chunks the up warps write
    // buffer 0 and the gate warps combine and store, on odd chunks the gate warps write buffer 1 and the up warps
    // combine and store.  Named barriers of a set: "buffer written" (writers arrive, readers wait) and "buffer read"
    // (readers arrive, writers wait before writing it again) per buffer; each is used by the same 64 + 64 threads in
    // strict alternation, so no phase can be overtaken.
    const int quarter = warp & 3;
    const int set = (warp - 2) >> 2;
    const bool up_warp = quarter >= 2;
    const int feat = (quarter & 1) * 32 + lane;  // feature within this CTA's 64
    const int ep_tid = (warp - 2) * 32 + lane;
    const int set_n = p.tok_n >> 1;              // token columns of a set (multiple of 8)
    const int n_chunks = (set_n + 31) >> 5;
    const int my_units = pair < p.n_units ? (p.n_units - pair + p.n_pairs - 1) / p.n_pairs : 0;
    const int total_chunks = my_units * n_chunks;
    const int bar_written = 2 + set * 4, bar_read = 4 + set * 4, bar_group = 10 + set * 2 + (up_warp ? 0 : 1);
    float* xset = xch + set * (2 * 32 * SP_FEAT);
    int it = 0, cc = 0;
    for (int u = pair; u < p.n_units; u += p.n_pairs, ++it) {
      const int b = it & 1;
      if (ep_tid == 0) ep_ok[0] = mbar_wait(tmem_full(b), (it >> 1) & 1, abort_flag, p.status) ? 1 : 0;
      named_bar_sync(1, 256);
      if (!ep_ok[0]) break;  // uniform for the 256 threads
      tc_fence_after();
      const uint32_t trow = tmem_base + (uint32_t)b * 256u + (uint32_t)(set * set_n) + ((uint32_t)(quarter * 32) << 16);
      int fb, tt;
      sp_unit(u, p.n_fblocks, p.tok_tiles, p.group, fb, tt);
      const int f = fb * (2 * SP_FEAT) + (int)rank * SP_FEAT + feat;
      const int t0 = tt * p.tok_n + set * set_n;
      bf16* out = p.C + f;
#pragma unroll 1
      for (int c = 0; c < n_chunks; ++c, ++cc) {
        const int buf = cc & 1;
        const int w = min(32, set_n - c * 32);
        float* xb = xset + buf * (32 * SP_FEAT);
        float v[32];
        __syncwarp();
        sp_ld_chunk(trow + c * 32, w, v);
        const bool writer = up_warp == (buf == 0);
        if (writer) {
          if (cc >= 2) named_bar_sync(bar_read + buf, 128);  // the readers are done with what this buffer held
          if (w == 32) {
#pragma unroll
            for (int e = 0; e < 32; ++e) xb[e * SP_FEAT + feat] = v[e];
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (e < w) xb[e * SP_FEAT + feat] = v[e];
          }
          named_bar_arrive(bar_written + buf, 128);
        } else {
          named_bar_sync(bar_written + buf, 128);
          bf16* orow = out + (size_t)(t0 + c * 32) * p.ldc;
          const int valid = min(w, p.M - (t0 + c * 32));  // tokens of this chunk that exist
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float o = xb[e * SP_FEAT + feat];
            const float g = up_warp ? o : v[e], uv = up_warp ? v[e] : o;
            const float r = silu_mul(g, uv);
            if (e < valid) orow[(size_t)e * p.ldc] = __float2bfloat16_rn(r);
          }
          if (cc + 2 < total_chunks) named_bar_arrive(bar_read + buf, 128);  // nobody waits for the last two
        }
      }
      // this half of the set has read its part of the accumulator (wait::ld in sp_ld_chunk): one arrival per half,
      // set and CTA on the leader's barrier hands it back to the MMA issuer
      tc_fence_before();
      named_bar_sync(bar_group, 64);
      if (lane == 0 && (quarter == 0 || quarter == 2)) mbar_arrive_in_cta(tmem_empty(b), 0);
    }
  } else if (EPI == EPI_QKV) {
    // ---------------- epilogue, q / k / v heads: warps 2..9 of both CTAs; warp w may touch TMEM lanes 32*(w%4) .. +31,
    // lane = feature of this CTA's head; warp set 0 (warps 2..5) takes the first half of the token columns, set 1 the
    // second.  32 tokens at a time, in two phases around a named barrier of the set's 128 threads:
    //   1. feature-major: every warp reads its 32 features x 32 tokens from tensor memory, adds the bias and parks the
    //      values in shared memory; the first warp also fetches and checks the tokens' positions;
    //   2. token-major: a thread takes 8 consecutive features of the head's first half and the 8 that lie 64 further of
    //      ONE token (both halves of its rotation pairs, whichever the pairing), rotates them with 16-byte loads of the
    //      token's table row and writes two 16-byte vectors: a warp stores 512 contiguous-by-row bytes per instruction
    //      where a lane-per-feature epilogue stores 64.
    const int quarter = warp & 3;
    const int set = (warp - 2) >> 2;
    const int ep_tid = (warp - 2) * 32 + lane;
    const int st = quarter * 32 + lane;  // thread within the set
    const int set_n = p.tok_n >> 1;
    const int n_chunks = (set_n + 31) >> 5;
    float* xset = xch + set * SP_QKV_SET_FLOATS;
    int* posbuf = reinterpret_cast<int*>(base_ptr + xch_off + SP_QKV_XCH_BYTES) + set * 32;
    const int bar_set = 2 + set;
    // phase 2 assignment: token e2 (+16 in the second pass), features f0 .. f0 + 7 and 64 + f0 .. 64 + f0 + 7
    const int e2 = st >> 3, f0 = (st & 7) * 8;
    const float* xlo = xset + (f0 >> 5) * (32 * 32 + 4) + (f0 & 31);
    const float* xhi = xset + (2 + (f0 >> 5)) * (32 * 32 + 4) + (f0 & 31);
    float* xmine = xset + quarter * (32 * 32 + 4) + lane;
    int it = 0;
    for (int u = pair; u < p.n_units; u += p.n_pairs, ++it) {
      const int b = it & 1;
      int fb, tt;
      sp_unit(u, p.n_fblocks, p.tok_tiles, p.group, fb, tt);
      const int hd = 2 * fb + (int)rank;
      const bool live = hd < p.n_heads;
      const int hde = live ? hd : 0;
      const int sg = (hde >= p.seg_heads_end[0]) + (hde >= p.seg_heads_end[1]);
      const int head_in_seg = hde - (sg == 0 ? 0 : p.seg_heads_end[sg - 1]);
      const int kind = p.kind[sg];
      const int t0 = tt * p.tok_n + set * set_n;
      const float bias = p.bias[sg] ? __bfloat162float(p.bias[sg][head_in_seg * 128 + quarter * 32 + lane]) : 0.f;
      const bool rotate = kind != 2;
      if (ep_tid == 0) ep_ok[0] = mbar_wait(tmem_full(b), (it >> 1) & 1, abort_flag, p.status) ? 1 : 0;
      named_bar_sync(1, 256);
      if (!ep_ok[0]) break;  // uniform for the 256 threads
      tc_fence_after();
      const uint32_t trow = tmem_base + (uint32_t)b * 256u + (uint32_t)(set * set_n) + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < n_chunks; ++c) {
        const int w = min(32, set_n - c * 32);
        const int valid = min(w, p.M - (t0 + c * 32));  // tokens of this chunk that exist (may be <= 0)
        float v[32];
        __syncwarp();
        sp_ld_chunk(trow + c * 32, w, v);
        if (quarter == 0) {  // positions of the chunk's tokens, checked: -1 where nothing is to be written
          int ps = -1;
          if (lane < valid) {
            ps = p.pos[t0 + c * 32 + lane];
            if (ps < 0 || ps >= p.kv_len || ps >= p.max_pos) {
              if (live) atomicOr(p.status, A3_DEV_BAD_POSITION);
              ps = -1;
            }
          }
          posbuf[lane] = ps;
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) xmine[e * 32] = v[e] + bias;
        named_bar_sync(bar_set, 128);
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
          const int e = e2 + 16 * pass;
          const int ps = posbuf[e];
          if (ps < 0 || !live) continue;
          float a[8], bq[8], ra[8], rb[8];
          *reinterpret_cast<float4*>(a) = *reinterpret_cast<const float4*>(xlo + e * 32);
          *reinterpret_cast<float4*>(a + 4) = *reinterpret_cast<const float4*>(xlo + e * 32 + 4);
          *reinterpret_cast<float4*>(bq) = *reinterpret_cast<const float4*>(xhi + e * 32);
          *reinterpret_cast<float4*>(bq + 4) = *reinterpret_cast<const float4*>(xhi + e * 32 + 4);
          if (!rotate) {
#pragma unroll
            for (int k = 0; k < 8; ++k) ra[k] = a[k], rb[k] = bq[k];
          } else if (p.layout == 0) {
            // pairs (i, i + 64): the thread's first 8 features rotate with the 8 that lie 64 further, frequencies f0 .. f0 + 7
            const float4* tr = reinterpret_cast<const float4*>(p.tab + (size_t)ps * 64 + f0);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float4 t = __ldg(tr + k);  // (cos, sin) of two frequencies
              ra[2 * k] = a[2 * k] * t.x - bq[2 * k] * t.y;
              rb[2 * k] = a[2 * k] * t.y + bq[2 * k] * t.x;
              ra[2 * k + 1] = a[2 * k + 1] * t.z - bq[2 * k + 1] * t.w;
              rb[2 * k + 1] = a[2 * k + 1] * t.w + bq[2 * k + 1] * t.z;
            }
          } else {
            // pairs (2i, 2i + 1): both groups of 8 hold four pairs of their own, frequencies f0/2 .. and 32 + f0/2 ..
            const float4* tl = reinterpret_cast<const float4*>(p.tab + (size_t)ps * 64 + (f0 >> 1));
            const float4* th = reinterpret_cast<const float4*>(p.tab + (size_t)ps * 64 + 32 + (f0 >> 1));
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              const float4 t = __ldg(tl + k), u4 = __ldg(th + k);
              ra[4 * k] = a[4 * k] * t.x - a[4 * k + 1] * t.y;
              ra[4 * k + 1] = a[4 * k] * t.y + a[4 * k + 1] * t.x;
              ra[4 * k + 2] = a[4 * k + 2] * t.z - a[4 * k + 3] * t.w;
              ra[4 * k + 3] = a[4 * k + 2] * t.w + a[4 * k + 3] * t.z;
              rb[4 * k] = bq[4 * k] * u4.x - bq[4 * k + 1] * u4.y;
              rb[4 * k + 1] = bq[4 * k] * u4.y + bq[4 * k + 1] * u4.x;
              rb[4 * k + 2] = bq[4 * k + 2] * u4.z - bq[4 * k + 3] * u4.w;
              rb[4 * k + 3] = bq[4 * k + 2] * u4.w + bq[4 * k + 3] * u4.z;
            }
          }
          bf16* dst = kind == 0 ? p.q_out + (size_t)(t0 + c * 32 + e) * (p.Hq * 128) + head_in_seg * 128
                    : (kind == 1 ? p.k_cache : p.v_cache) + (size_t)ps * (p.Hkv * 128) + head_in_seg * 128;
          *reinterpret_cast<uint4*>(dst + f0) = pack8(ra);
          *reinterpret_cast<uint4*>(dst + 64 + f0) = pack8(rb);
        }
        named_bar_sync(bar_set, 128);  // everybody has read this chunk's values and positions
      }
      // this warp has read its part of the accumulator (wait::ld in sp_ld_chunk): it goes back to the MMA issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_in_cta(tmem_empty(b), 0);
    }
  } else if (EPI == EPI_RESIDUAL) {
    // ---------------- epilogue, C += A B^T: warps 2..9 of both CTAs; warp w may touch TMEM lanes 32*(w%4) .. +31,
    // lane = output feature; warp set 0 (warps 2..5) takes the first half of the token columns, set 1 the second.
    // A warp reads and writes 32 consecutive features of one token (64 bytes) per instruction.
    const int quarter = warp & 3;
    const int set = (warp - 2) >> 2;
    const int ep_tid = (warp - 2) * 32 + lane;
    const int set_n = p.tok_n >> 1;
    const int n_chunks = (set_n + 31) >> 5;
    int it = 0;
    for (int u = pair; u < p.n_units; u += p.n_pairs, ++it) {
      const int b = it & 1;
      int fb, tt;
      sp_unit(u, p.n_fblocks, p.tok_tiles, p.group, fb, tt);
      const int f = fb * (2 * ROWS) + (int)rank * ROWS + quarter * 32 + lane;
      const int t0 = tt * p.tok_n + set * set_n;
      const bool f_ok = f < p.F;  // the last feature block may reach past the matrix (zero-filled loads)
      bf16* crow = p.C + (size_t)t0 * p.ldc + (f_ok ? f : 0);
      // the old values of the first chunk are on their way while the main loop still runs
      bf16 old[32];
      {
        const int valid = f_ok ? min(min(32, set_n), p.M - t0) : 0;
#pragma unroll
        for (int e = 0; e < 32; ++e) old[e] = e < valid ? crow[(size_t)e * p.ldc] : __float2bfloat16_rn(0.f);
      }
      if (ep_tid == 0) ep_ok[0] = mbar_wait(tmem_full(b), (it >> 1) & 1, abort_flag, p.status) ? 1 : 0;
      named_bar_sync(1, 256);
      if (!ep_ok[0]) break;  // uniform for the 256 threads
      tc_fence_after();
      const uint32_t trow = tmem_base + (uint32_t)b * 256u + (uint32_t)(set * set_n) + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < n_chunks; ++c) {
        const int w = min(32, set_n - c * 32);
        float v[32];
        __syncwarp();
        sp_ld_chunk(trow + c * 32, w, v);
        bf16* orow = crow + (size_t)(c * 32) * p.ldc;
        const int valid = f_ok ? min(w, p.M - (t0 + c * 32)) : 0;
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (e < valid) orow[(size_t)e * p.ldc] = __float2bfloat16_rn(v[e] + __bfloat162float(old[e]));
        if (c + 1 < n_chunks) {  // the next chunk's old values
          const int nvalid = f_ok ? min(min(32, set_n - (c + 1) * 32), p.M - (t0 + (c + 1) * 32)) : 0;
          const bf16* nrow = orow + (size_t)32 * p.ldc;
#pragma unroll
          for (int e = 0; e < 32; ++e) old[e] = e < nvalid ? nrow[(size_t)e * p.ldc] : __float2bfloat16_rn(0.f);
        }
      }
      // this warp has read its part of the accumulator (wait::ld in sp_ld_chunk): it goes back to the MMA issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_in_cta(tmem_empty(b), 0);
    }
  }
  tc_fence_before();
  cluster_sync_all();  // neither CTA releases tensor or shared memory while the other may still use it
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

// A3_OPT_SWIGLU_PAIR / A3_OPT_RESIDUAL_T: 0 never; 1 whenever the shape allows (default); cross-checks switch them off
// to compare with the other kernels
bool swiglu_pair_usable(const a3_handle* h, const GemmArgs& a) {
  return h->opt[A3_OPT_SWIGLU_PAIR] != 0 && a.M > 0 && a.K % (SP_SUB * TC_BK) == 0 && a.seg[0].n % (2 * SP_FEAT) == 0 && a.seg[0].bias == nullptr;
}
// Measured at Llama-8B width: with several units per CTA pair (5 152 rows: 336 units on 74 pairs) this kernel hides
// every epilogue but the last and wins (output projection 139 vs 165 us, down projection 522 vs 533 us); with at most
// one unit per pair (804 rows: 64 units) it has nothing to hide and the 256 x 256 CTA-pair kernel is as fast or faster
// (26 vs 28 us, 85 vs 82 us).  A3_OPT_RESIDUAL_T: 0 never, 1 by that rule (default), 2 whenever the shape allows.
bool residual_t_usable(const a3_handle* h, const GemmArgs& a) {
  const int g_residual_t = h->opt[A3_OPT_RESIDUAL_T];
  if (g_residual_t == 0 || a.M <= 0 || a.K % (SP_SUB * TC_BK) != 0 || a.nseg != 1 || a.seg[0].n % 32 != 0 || a.seg[0].bias != nullptr)
    return false;
  if (g_residual_t == 2) return true;
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
  return cdiv(a.seg[0].n, 4 * SP_FEAT) * cdiv(a.M, 256) > sms / 2;
}

// Token tiling of a launch: `tiles` tiles of `n` tokens (a multiple of 16, at most 256) that divide the row count
// evenly.  The tile count is the one with the cheapest rounds: the CTA pairs take the units (feature block x token
// tile) round by round, and a unit of n token columns costs, per k-block, the larger of its tensor time (2 n clocks:
// four instructions of n / 2) and the time its operands take to arrive (16 KiB of weights + 64 n bytes of tokens per
// CTA at about 64 bytes per clock: 256 + n clocks), plus a fixed part.  By that measure every unit narrower than 256
// waits for its operands, and the measurements agree: 804 rows x 112 feature blocks as five tiles of 176 (or as
// 4 x 176 + 112 with the narrow units last, which a count of token columns alone prefers) took 160-165 us against 147
// for 4 x 208.  Examples: 4 952 rows x 16 feature blocks -> 23 x 224 (five rounds of 224 instead of five of 256:
// 536 vs 591 us for both residual GEMMs of a layer), x 112 -> 20 x 256 as before; 804 rows x 24 head pairs -> 6 x 144
// (two rounds) instead of 4 x 208 (two rounds).  A3_OPT_GEMM_TILING = 1 keeps ceil(M / 256) tiles (comparisons).
// Feature blocks per group of the unit order: 8 when the token matrix (M x K bf16) is too large to stay in L2 beside
// the weights and the output that stream through it, else 1.
static int unit_group(int M, int K) { return (long long)M * K * 2 > (64ll << 20) ? 8 : 1; }

struct SpTiling {
  int tiles, n;
};
static SpTiling choose_tiling(const a3_handle* h, int M, int n_fblocks, int pairs) {
  SpTiling best{cdiv(M, 256), 0};
  best.n = cdiv(cdiv(M, best.tiles), 16) * 16;  // 804 rows -> 4 x 208
  if (h->opt[A3_OPT_GEMM_TILING] == 1) return best;
  auto load = [&](int tiles, int n) {
    const long long unit = (long long)(2 * n > 256 + n ? 2 * n : 256 + n) + 32;
    return (long long)cdiv((long long)n_fblocks * tiles, pairs) * unit;
  };
  long long best_load = load(best.tiles, best.n);
  for (int tiles = best.tiles + 1; tiles <= best.tiles + 64 && tiles <= cdiv(M, 96); ++tiles) {
    const int n = cdiv(cdiv(M, tiles), 16) * 16;
    const long long l = load(tiles, n);
    if (l < best_load) {
      best_load = l;
      best = SpTiling{tiles, n};
    }
  }
  return best;
}

template <int EPI>
static int launch_pair_t(const a3_handle* h, const GemmArgs& a, cudaStream_t st) {
  constexpr int ROWS = EPI == EPI_SWIGLU ? SP_FEAT : 2 * SP_FEAT;  // output features per CTA
  constexpr int XCH = EPI == EPI_SWIGLU ? SP_XCH_BYTES : 0;
  SpParams p{};
  p.M = a.M;
  p.K = a.K;
  p.F = a.seg[0].n;
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
  p.n_fblocks = cdiv(p.F, 2 * ROWS);
  const SpTiling til = choose_tiling(h, a.M, p.n_fblocks, sms / 2);
  p.tok_tiles = til.tiles;
  p.tok_n = til.n;
  p.n_units = p.n_fblocks * p.tok_tiles;
  p.group = unit_group(a.M, a.K);
  p.n_pairs = p.n_units < sms / 2 ? p.n_units : sms / 2;
  p.C = a.C;
  p.ldc = a.ldc;
  p.status = h->dev_status;
  // as many ring stages as fit beside the exchange buffers
  p.sub_bytes = SP_A_BYTES + (int)align_up((size_t)(p.tok_n / 2) * TC_BK * 2, 1024);
  p.stage_bytes = SP_SUB * p.sub_bytes;
  p.stages = (SP_SMEM_LIMIT - XCH - 256 - 1024) / p.stage_bytes;
  if (p.stages > SP_MAX_STAGES) p.stages = SP_MAX_STAGES;
  const int smem_bytes = p.stages * p.stage_bytes + XCH + 256 + 1024;
  CUtensorMap tX, tG, tU;
  A3_TRY(make_tmap(&tX, a.A, a.M, a.K, p.tok_n / 2));
  A3_TRY(make_tmap(&tG, a.seg[0].B, p.F, a.K, ROWS));
  if (EPI == EPI_SWIGLU) A3_TRY(make_tmap(&tU, a.B2, p.F, a.K, ROWS));
  else tU = tG;
  static SmemAttrOnce attr;
  A3_TRY(smem_attr_once(attr, h->device, pair_t_kernel<EPI>, SP_SMEM_LIMIT));
  ProfScope prof(h, EPI == EPI_SWIGLU ? A3_K_GEMM_SWIGLU : A3_K_GEMM_RESIDUAL, st);
  A3_CUDA(launch_pdl(pair_t_kernel<EPI>, dim3(2 * p.n_pairs), dim3(SP_THREADS), (size_t)smem_bytes, st, tX, tG, tU, tU, p));
  A3_LAUNCHED();
  return A3_OK;
}

// QKV projection on the same kernel: one head (128 features) per CTA of a pair, token tiles chosen so that the units
// fill whole rounds of the CTA pairs.  A3_OPT_QKV_T: 0 never, 1 whenever the shape allows (default).
bool qkv_t_usable(const a3_handle* h, const GemmArgs& a) {
  if (h->opt[A3_OPT_QKV_T] == 0 || h->m.head_dim != 128 || a.M <= 0 || a.K % (SP_SUB * TC_BK) != 0 || a.nseg < 1 || a.nseg > 3) return false;
  for (int s = 0; s < a.nseg; ++s)
    if (a.seg[s].n % 128 != 0 || a.seg[s].n <= 0) return false;
  return true;
}

int gemm_qkv_t(const a3_handle* h, const GemmArgs& a, cudaStream_t st) {
  SpParams p{};
  p.M = a.M;
  p.K = a.K;
  int heads = 0;
  for (int s = 0; s < 3; ++s) {
    if (s < a.nseg) {
      heads += a.seg[s].n / 128;
      p.kind[s] = a.seg[s].kind;
      p.bias[s] = a.seg[s].bias;
    }
    p.seg_heads_end[s] = heads;
  }
  p.n_heads = heads;
  const int head_pairs = cdiv(heads, 2);
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
  const int pairs = sms / 2;
  const SpTiling til = choose_tiling(h, a.M, head_pairs, pairs);
  p.tok_tiles = til.tiles;
  p.tok_n = til.n;
  p.n_fblocks = head_pairs;
  p.group = unit_group(a.M, a.K);
  p.n_units = head_pairs * p.tok_tiles;
  p.n_pairs = p.n_units < pairs ? p.n_units : pairs;
  p.status = h->dev_status;
  p.q_out = a.q_out;
  p.k_cache = a.k_cache;
  p.v_cache = a.v_cache;
  p.pos = a.pos;
  p.kv_len = a.kv_len;
  p.Hq = h->m.n_q_heads;
  p.Hkv = h->m.n_kv_heads;
  p.layout = h->m.rope_layout;
  p.max_pos = h->m.max_positions;
  p.tab = h->rope_tab;
  p.sub_bytes = SP_A_BYTES + (int)align_up((size_t)(p.tok_n / 2) * TC_BK * 2, 1024);
  p.stage_bytes = SP_SUB * p.sub_bytes;
  p.stages = (SP_SMEM_LIMIT - SP_QKV_EXTRA - 256 - 1024) / p.stage_bytes;
  if (p.stages > SP_MAX_STAGES) p.stages = SP_MAX_STAGES;
  const int smem_bytes = p.stages * p.stage_bytes + SP_QKV_EXTRA + 256 + 1024;
  CUtensorMap tX, tW[3];
  A3_TRY(make_tmap(&tX, a.A, a.M, a.K, p.tok_n / 2));
  for (int s = 0; s < 3; ++s) {
    if (s < a.nseg) A3_TRY(make_tmap(&tW[s], a.seg[s].B, a.seg[s].n, a.K, 128));
    else tW[s] = tW[0];
  }
  static SmemAttrOnce attr;
  A3_TRY(smem_attr_once(attr, h->device, pair_t_kernel<EPI_QKV>, SP_SMEM_LIMIT));
  ProfScope prof(h, A3_K_GEMM_QKV, st);
  A3_CUDA(launch_pdl(pair_t_kernel<EPI_QKV>, dim3(2 * p.n_pairs), dim3(SP_THREADS), (size_t)smem_bytes, st, tX, tW[0], tW[1], tW[2], p));
  A3_LAUNCHED();
  return A3_OK;
}

int gemm_swiglu_pair(const a3_handle* h, const GemmArgs& a, cudaStream_t st) { return launch_pair_t<EPI_SWIGLU>(h, a, st); }
int gemm_residual_t(const a3_handle* h, const GemmArgs& a, cudaStream_t st) { return launch_pair_t<EPI_RESIDUAL>(h, a, st); }

}  // namespace a3

// The gate/up GEMM of one layer alone (a3_swiglu_rows): out[M][d_ff] = silu(x Wg^T) * (x Wu^T), x [M][d_model].
extern "C" int a3_swiglu_rows(const a3_handle* h, int layer, const void* x, void* out, int M, a3_stream stream) {
  if (!h || layer < 0 || layer >= h->m.n_layers || M < 0) return A3_EINVAL;
  if (M == 0) return A3_OK;
  if (!x || !out || (((uintptr_t)x | (uintptr_t)out) & 15)) return A3_EINVAL;
  a3::GemmArgs u{};
  u.A = (const bf16*)x;
  u.M = M;
  u.K = h->m.d_model;
  u.nseg = 1;
  u.seg[0] = {(const bf16*)h->layers[layer].w_gate, nullptr, h->m.d_ff, 0};
  u.B2 = (const bf16*)h->layers[layer].w_up;
  u.C = (bf16*)out;
  u.ldc = h->m.d_ff;
  return a3::gemm_bf16(h, a3::EPI_SWIGLU, u, (cudaStream_t)stream);
}

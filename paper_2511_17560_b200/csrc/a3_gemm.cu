// Projection / MLP GEMMs of the recompute path (Eq. 5: Q_l = X_l W^q, K <- X_l W^k, V <- X_l W^v; H(.)) on the
// 5th-generation tensor cores:  C[M][N] = A[M][K] * B[N][K]^T, bf16 operands (both K-major), fp32 accumulators in
// tensor memory, fused epilogues:
//   EPI_RESIDUAL  C <- C + A B^T                       (output projection and MLP down projection)
//   EPI_SWIGLU    C <- silu(A Bg^T) * (A Bu^T)         (gate and up rows interleaved per tile: BN/2 + BN/2 columns)
//   EPI_QKV       +bias, RoPE of q/k at pos[m], q -> q_out, k/v -> cache rows pos[m] (the scatter of Eq. 5)
//
// One CTA computes one 128 x BN tile.  Warp 0 (one lane) feeds a ring of shared-memory stages with TMA
// (cp.async.bulk.tensor, 128-byte swizzle); warp 1 (one lane) issues tcgen05.mma (128 x BN x 16) on the stages and
// commits them back to the producer through mbarriers; warps 2..5 read the accumulator with tcgen05.ld (each thread
// owns one output row) and run the epilogue straight out of registers.  A second kernel shares a 256 x 256 tile
// between the two CTAs of a cluster (tcgen05 cta_group::2, see below).  No load uses cluster multicast.
// Every barrier wait is bounded: after half a second a waiter raises the CTA's abort flag and the device status bit
// A3_DEV_WAIT_EXHAUSTED, all roles leave their loops, in-flight copies are given time to land, tensor memory is
// released and the CTA returns.
#include <cuda.h>

#include "a3_internal.cuh"
#include "a3_tc.cuh"

namespace a3 {

template <int BN, int STAGES>
struct TcLayout {
  static constexpr int A_BYTES = TC_BM * TC_BK * 2;
  static constexpr int B_BYTES = BN * TC_BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFFSET + 256 + 1024;  // barriers + slack for the 1024-byte alignment
};

// QKV epilogue of one row: bias, RoPE with the prefetched (cos, sin) row, q -> buffer, k/v -> cache row pos[m].
template <int BN, int D>
__device__ __forceinline__ void tc_epilogue_qkv_row(const TcParams& p, uint32_t trow, int gr, bool row_ok, int seg, int nb0,
                                                    const uint4* pre, int qkv_pos) {
  const int kind = p.kind[seg];
  constexpr int half = D / 2;
  const bf16* bias = p.bias[seg];
  // the row's position was read and checked, and its cos/sin row fetched into `pre`, while the main loop ran
  const bool ok = row_ok && qkv_pos >= 0;
  const int ps = ok ? qkv_pos : 0;
  const float2* cs_row = reinterpret_cast<const float2*>(pre);
  bf16* dst;
  if (kind == 0) dst = p.q_out + (size_t)(row_ok ? gr : 0) * (p.Hq * D) + nb0;
  else if (kind == 1) dst = p.k_cache + (size_t)ps * (p.Hkv * D) + nb0;
  else dst = p.v_cache + (size_t)ps * (p.Hkv * D) + nb0;
  // pairs of 32-column chunks that hold the two halves of the rotation pairs (same chunk twice for the
  // interleaved layout and for V, which is not rotated)
  const int pair_stride = (p.layout == 0) ? half / 32 : 0;  // D=128: 2 chunks; D=64: 1 chunk
#pragma unroll
  for (int c = 0; c < BN / 32; ++c) {
    const int in_head = (c * 32) % D;  // static after unrolling: `pre` stays in registers
    if (p.layout == 0 && in_head >= half) continue;  // handled together with its low half
    __syncwarp();
    float a[32], b[32];
    tc_ld32(trow + c * 32, a);
    if (p.layout == 0) tc_ld32(trow + (c + pair_stride) * 32, b);
    tc_wait_ld();
    if (!ok) continue;
    const int ca = c * 32, cb = (c + pair_stride) * 32;
    if (bias) {
      float t[32];
      load32_bf16(bias + nb0 + ca, t);
#pragma unroll
      for (int e = 0; e < 32; ++e) a[e] += t[e];
      if (p.layout == 0) {
        load32_bf16(bias + nb0 + cb, t);
#pragma unroll
        for (int e = 0; e < 32; ++e) b[e] += t[e];
      }
    }
    if (kind != 2) {
      if (p.layout == 0) {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float2 cs = cs_row[in_head + e];
          const float x = a[e], y = b[e];
          a[e] = x * cs.x - y * cs.y;
          b[e] = x * cs.y + y * cs.x;
        }
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float2 cs = cs_row[in_head / 2 + e];
          const float x = a[2 * e], y = a[2 * e + 1];
          a[2 * e] = x * cs.x - y * cs.y;
          a[2 * e + 1] = x * cs.y + y * cs.x;
        }
      }
    }
    store32_bf16(dst + ca, a);
    if (p.layout == 0) store32_bf16(dst + cb, b);
  }
}

// Epilogue of one accumulator row (thread = row `gr` of the output, `trow` its tensor-memory address), straight out
// of registers.  For EPI_RESIDUAL the row's old values arrive in `pre` (see tc_prefetch_residual).
template <int EPI, int BN>
__device__ __forceinline__ void tc_epilogue_row(const TcParams& p, uint32_t trow, int gr, bool row_ok, int nt, int seg, int nb0,
                                                const uint4* pre, int qkv_pos, int g_cols = BN / 2) {
    if (EPI == EPI_RESIDUAL) {
      // the old values of C were fetched while the main loop ran (`pre`): only tensor memory is waited for here
      const int n0 = nt * BN;
#pragma unroll
      for (int c = 0; c < BN / 32; ++c) {
        float acc[32];
        tc_ld32(trow + c * 32, acc);
        tc_wait_ld();
        if (row_ok && n0 + c * 32 < p.N) {  // tiles need not divide N: TMA zero-fills, stores are cut
          float old[32];
#pragma unroll
          for (int i = 0; i < 4; ++i) unpack8(pre[c * 4 + i], old + 8 * i);
#pragma unroll
          for (int e = 0; e < 32; ++e) acc[e] += old[e];
          store32_bf16(p.C + (size_t)gr * p.ldc + n0 + c * 32, acc);
        }
      }
    } else if (EPI == EPI_SWIGLU) {
      // gate columns 0..g_cols-1, up columns g_cols..2 g_cols-1 of the accumulator; the tile's first feature is nb0
      const int n0 = nb0;
      // 32 columns at a time; a narrow tile's remainder, and a last tile that reaches the end of the matrix (its
      // loads beyond it were zero-filled), 8 at a time.  The branch depends on the tile only: uniform for the warp.
      const int n8 = g_cols / 8;
      int c8 = 0;
#pragma unroll 1
      while (c8 < n8) {
        __syncwarp();
        const int col = n0 + c8 * 8;
        if (c8 + 4 <= n8 && col + 32 <= p.N) {
          float g[32], u[32];
          tc_ld32(trow + c8 * 8, g);
          tc_ld32(trow + g_cols + c8 * 8, u);
          tc_wait_ld();
          if (row_ok) {
#pragma unroll
            for (int e = 0; e < 32; ++e) g[e] = silu_mul(g[e], u[e]);
            store32_bf16(p.C + (size_t)gr * p.ldc + col, g);
          }
          c8 += 4;
        } else {
          float g[8], u[8];
          tc_ld8(trow + c8 * 8, g);
          tc_ld8(trow + g_cols + c8 * 8, u);
          tc_wait_ld();
          if (row_ok && col + 8 <= p.N) {
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = silu_mul(g[e], u[e]);
            *reinterpret_cast<uint4*>(p.C + (size_t)gr * p.ldc + col) = pack8(g);
          }
          c8 += 1;
        }
      }
    } else {
      if (p.D == 128) tc_epilogue_qkv_row<BN, 128>(p, trow, gr, row_ok, seg, nb0, pre, qkv_pos);
      else tc_epilogue_qkv_row<BN, 64>(p, trow, gr, row_ok, seg, nb0, pre, qkv_pos);
    }
}

// Old values of this thread's row of C for the residual epilogue: issued before the accumulator is waited for, so
// the global-memory latency (a row per lane: uncoalesced, L2-resident) hides behind the main loop.
// Position of this thread's row (checked; -1 if unusable) and, for q and k tiles, the row's D/2 (cos, sin) pairs into
// `pre`: issued before the accumulator is waited for, like the residual rows below.
__device__ __forceinline__ int tc_prefetch_rope(const TcParams& p, int gr, bool row_ok, int seg, uint4 (&pre)[32]) {
  if (!row_ok) return -1;
  const int ps = p.pos[gr];
  if (ps < 0 || ps >= p.kv_len || ps >= p.max_pos) {
    atomicOr(p.status, A3_DEV_BAD_POSITION);
    return -1;
  }
  if (p.kind[seg] != 2) {
    const uint4* src = reinterpret_cast<const uint4*>(p.tab + (size_t)ps * (p.D / 2));
    const int nvec = p.D / 4;  // D/2 float2 = D/4 16-byte vectors (at most 32)
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (i < nvec) pre[i] = __ldg(src + i);
  }
  return ps;
}

template <int BN>
__device__ __forceinline__ void tc_prefetch_residual(const TcParams& p, int gr, bool row_ok, int nt, uint4 (&pre)[BN / 8]) {
  const int n0 = nt * BN;
#pragma unroll
  for (int c = 0; c < BN / 32; ++c) {
    const bool col_ok = row_ok && n0 + c * 32 < p.N;
    const uint4* src = reinterpret_cast<const uint4*>(p.C + (size_t)(col_ok ? gr : 0) * p.ldc + (col_ok ? n0 + c * 32 : 0));
#pragma unroll
    for (int i = 0; i < 4; ++i) pre[c * 4 + i] = col_ok ? __ldg(src + i) : make_uint4(0, 0, 0, 0);
  }
}

// QKV tiles made of whole heads of 128 columns (BN = 384: three heads), which may straddle the q/k/v matrices:
// head g of the concatenated [q | k | v] output -> its matrix (segment) and its first row there.
__device__ __forceinline__ void qkv_head_of(const TcParams& p, int g, int& seg, int& row0) {
  seg = (g >= p.seg_heads_end[0]) + (g >= p.seg_heads_end[1]);
  row0 = (g - (seg == 0 ? 0 : p.seg_heads_end[seg - 1])) * 128;
}

template <int EPI, int BN, int STAGES>
__global__ void __launch_bounds__(TC_THREADS)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
               const __grid_constant__ CUtensorMap tmN0, const __grid_constant__ CUtensorMap tmN1, const TcParams p) {
  using L = TcLayout<BN, STAGES>;
  constexpr int TMEM_COLS = BN <= 128 ? 128 : (BN <= 256 ? 256 : 512);  // allocations are powers of two
  // head tiles: the tile is BN/128 whole heads, each loaded from its own matrix (QKV at head dimension 128 only)
  constexpr bool HEAD_TILES = (EPI == EPI_QKV && BN > 256);
  constexpr int HEADS = BN / 128;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + L::BAR_OFFSET;  // full[S], empty[S], tmem_full: 8 bytes each
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::BAR_OFFSET + 8 * (2 * STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::BAR_OFFSET + 8 * (2 * STAGES + 1) + 8);
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bars + 8u * (2 * STAGES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * TC_BM;
  const int nt = blockIdx.y;
  const int KT = p.K / TC_BK;

  int seg = 0, seg_tile0 = 0;
  if (EPI == EPI_QKV && !HEAD_TILES) {
    while (seg < 2 && nt >= p.seg_tiles_end[seg]) {
      seg_tile0 = p.seg_tiles_end[seg];
      ++seg;
    }
  }
  // first B row of this tile within its matrix (for SwiGLU: within gate and within up)
  int nb0 = (EPI == EPI_SWIGLU) ? nt * (BN / 2) : (nt - seg_tile0) * BN;
  // SwiGLU: features per tile; the column tiles from y_wide on are narrower (maps tmN0/tmN1, box g_narrow rows)
  int g_cols = BN / 2;
  const bool narrow = EPI == EPI_SWIGLU && p.g_narrow > 0 && nt >= p.y_wide;
  if (narrow) {
    g_cols = p.g_narrow;
    nb0 = p.y_wide * (BN / 2) + (nt - p.y_wide) * g_cols;
  }
  // head tiles: heads nt*HEADS .. of [q | k | v]; the last tile may hold fewer
  const int heads_here = HEAD_TILES ? min(HEADS, p.seg_heads_end[2] - nt * HEADS) : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(tmem_full_bar, 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;  // never raised: lets the drain below wait on its own clock only
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();  // everything above overlapped the previous kernel's tail; from here on its results are read
  pdl_launch_dependents();

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      const CUtensorMap* mapB = seg == 0 ? &tmB0 : (seg == 1 ? &tmB1 : &tmB2);
      const CUtensorMap* head_map[HEADS];
      int head_row0[HEADS];
      if (HEAD_TILES) {
#pragma unroll
        for (int j = 0; j < HEADS; ++j) {
          int sj = 0;
          head_row0[j] = 0;
          if (j < heads_here) qkv_head_of(p, nt * HEADS + j, sj, head_row0[j]);
          head_map[j] = sj == 0 ? &tmB0 : (sj == 1 ? &tmB1 : &tmB2);
        }
        tmap_prefetch(&tmB0);
        tmap_prefetch(&tmB1);
        tmap_prefetch(&tmB2);
      }
      tmap_prefetch(&tmA);
      tmap_prefetch(mapB);
      if (EPI == EPI_SWIGLU) tmap_prefetch(&tmB1);
      if (narrow) {
        tmap_prefetch(&tmN0);
        tmap_prefetch(&tmN1);
      }
      int issued = 0;
      for (int kb = 0; kb < KT; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, p.status)) break;
        const uint32_t sa = base + s * L::STAGE_BYTES, sb = sa + L::A_BYTES;
        mbar_expect_tx(full_bar(s), HEAD_TILES ? L::A_BYTES + heads_here * (L::B_BYTES / HEADS)
                                    : (EPI == EPI_SWIGLU ? L::A_BYTES + 2 * g_cols * TC_BK * 2 : L::STAGE_BYTES));
        tma_load_2d(sa, &tmA, kb * TC_BK, m0, full_bar(s));
        if (HEAD_TILES) {
#pragma unroll
          for (int j = 0; j < HEADS; ++j)
            if (j < heads_here) tma_load_2d(sb + j * (L::B_BYTES / HEADS), head_map[j], kb * TC_BK, head_row0[j], full_bar(s));
        } else if (EPI == EPI_SWIGLU) {
          // gate rows, then up rows (g_cols is a multiple of 8, so the up block starts on a 1024-byte boundary)
          tma_load_2d(sb, narrow ? &tmN0 : &tmB0, kb * TC_BK, nb0, full_bar(s));
          tma_load_2d(sb + g_cols * TC_BK * 2, narrow ? &tmN1 : &tmB1, kb * TC_BK, nb0, full_bar(s));
        } else {
          tma_load_2d(sb, mapB, kb * TC_BK, nb0, full_bar(s));
        }
        issued = kb + 1;
      }
      if (*abort_flag) {
        // let the copies already issued land before the CTA can exit (bounded)
        for (int kb = max(0, issued - STAGES); kb < issued; ++kb)
          mbar_wait(full_bar(kb % STAGES), (kb / STAGES) & 1, abort_flag + 1, p.status, 2000000ull);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = EPI == EPI_SWIGLU ? idesc_bf16(2 * g_cols) : idesc_bf16(BN > 256 ? 256 : BN);
      // head tiles: an instruction spans at most 256 columns, so heads 0-1 and head 2 are separate instructions
      const uint32_t idesc_lo = heads_here >= 2 ? idesc_bf16(256) : idesc_bf16(128);
      constexpr uint32_t idesc_hi = idesc_bf16(128);
      bool ok = true;
      for (int kb = 0; kb < KT && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(full_bar(s), ph, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = base + s * L::STAGE_BYTES, sb = sa + L::A_BYTES;
        const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
        if (HEAD_TILES) {
          const uint64_t db_hi = smem_desc_sw128(sb + 2 * (L::B_BYTES / HEADS));
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k) {
            tc_mma_f16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc_lo, (kb | k) != 0);
            if (heads_here > 2) tc_mma_f16(tmem_base + 256, da + (uint64_t)(2 * k), db_hi + (uint64_t)(2 * k), idesc_hi, (kb | k) != 0);
          }
        } else {
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)  // +32 bytes per 16-element K step inside the 128-byte swizzle row
            tc_mma_f16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0);
        }
        tc_commit(empty_bar(s));  // arrives once the MMAs above have finished reading this stage
      }
      if (ok) tc_commit(tmem_full_bar);
    }
  } else {
    // ---------------- epilogue: warps 2..5, warp w may touch TMEM lanes 32*(w%4) .. +31
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int gr = m0 + row;
    const bool row_ok = gr < p.M;
    const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16);
    uint4 pre[EPI == EPI_RESIDUAL ? BN / 8 : (EPI == EPI_QKV ? 32 : 1)];
    int qkv_pos = -1;
    if (EPI == EPI_RESIDUAL) tc_prefetch_residual<BN>(p, gr, row_ok, nt, *reinterpret_cast<uint4(*)[BN / 8]>(pre));
    if (EPI == EPI_QKV) {
      int seg_first = seg;  // head tiles: q/k heads come first in a tile, so the first head tells whether RoPE is needed
      if (HEAD_TILES) {
        int r0;
        qkv_head_of(p, nt * HEADS, seg_first, r0);
      }
      qkv_pos = tc_prefetch_rope(p, gr, row_ok, seg_first, *reinterpret_cast<uint4(*)[32]>(pre));
    }
    const bool ready = mbar_wait(tmem_full_bar, 0, abort_flag, p.status);
    tc_fence_after();
    if (ready) {
      if (HEAD_TILES) {
#pragma unroll 1
        for (int j = 0; j < heads_here; ++j) {
          int sj, r0;
          qkv_head_of(p, nt * HEADS + j, sj, r0);
          tc_epilogue_qkv_row<128, 128>(p, trow + j * 128, gr, row_ok, sj, r0, pre, qkv_pos);
        }
      } else {
        tc_epilogue_row<EPI, BN>(p, trow, gr, row_ok, nt, seg, nb0, pre, qkv_pos, g_cols);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

// ---------------------------------------------------------------- CTA-pair kernel (tcgen05 cta_group::2)
// With one CTA per tile every SM pulls A (128 x 64) and B (256 x 64) of each k-block through its own 64-byte-per-
// clock L2 port: 48 KiB per 512 clocks of MMA, i.e. the port, not the tensor core, sets the pace.  Here two CTAs of
// a cluster (two SMs) share one 256 x 256 output tile: each loads its own 128 rows of A and HALF of the B tile
// (32 KiB per k-block per SM), the leader CTA issues tcgen05.mma.cta_group::2 (M = 256, N = 256), which reads both
// halves of B from the two SMs' shared memory and leaves rows 0..127 of the accumulator in the leader's tensor
// memory and rows 128..255 in its peer's.  Both CTAs then run the same epilogues as the single-CTA kernel.
// Loads are plain per-CTA TMA copies (no multicast); the peer's copies complete on the leader's "full" barrier;
// tcgen05.commit with a CTA mask releases a stage (and, at the end, publishes the accumulator) in both CTAs.
constexpr int PAIR_BN = 256;
template <int STAGES>
struct PairLayout {
  static constexpr int A_BYTES = TC_BM * TC_BK * 2;
  static constexpr int B_BYTES = (PAIR_BN / 2) * TC_BK * 2;  // this CTA's half of the B tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFFSET + 256 + 1024;
};
template <int EPI, int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                 const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, const TcParams p) {
  using L = PairLayout<STAGES>;
  constexpr int BN = PAIR_BN;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // same offset in both CTAs of the pair
  unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + L::BAR_OFFSET;  // full[S] (used in the leader), empty[S], tmem_full: 8 bytes each
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::BAR_OFFSET + 8 * (2 * STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::BAR_OFFSET + 8 * (2 * STAGES + 1) + 8);
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bars + 8u * (2 * STAGES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int m0 = blockIdx.x * TC_BM;  // CTAs 2i and 2i+1 of a row of the grid form a pair: consecutive row tiles
  const int nt = blockIdx.y;
  const int KT = p.K / TC_BK;

  int seg = 0, seg_tile0 = 0;
  if (EPI == EPI_QKV) {
    while (seg < 2 && nt >= p.seg_tiles_end[seg]) {
      seg_tile0 = p.seg_tiles_end[seg];
      ++seg;
    }
  }
  // first output column of this tile within its matrix (for SwiGLU: within gate and within up)
  const int nb0 = (EPI == EPI_SWIGLU) ? nt * (BN / 2) : (nt - seg_tile0) * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(tmem_full_bar, 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // the same warp of both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(256) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();  // the peer's barriers exist before anything is signalled on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs): own rows of A, own half of B
    if (lane == 0) {
      const CUtensorMap* mapB;
      int brow0;
      if (EPI == EPI_SWIGLU) {
        mapB = leader ? &tmB0 : &tmB1;  // accumulator columns 0..127 = gate (leader's half), 128..255 = up (peer's half)
        brow0 = nb0;
      } else {
        mapB = seg == 0 ? &tmB0 : (seg == 1 ? &tmB1 : &tmB2);
        brow0 = nb0 + (int)rank * (BN / 2);
      }
      tmap_prefetch(&tmA);
      tmap_prefetch(mapB);
      int issued = 0;
      for (int kb = 0; kb < KT; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, p.status)) break;
        const uint32_t sa = base + s * L::STAGE_BYTES, sb = sa + L::A_BYTES;
        const uint32_t full_leader = full_bar(s) & PAIR_LEADER_MASK;
        // The leader announces the bytes of both CTAs.  A copy of the peer may complete before that: the phase
        // cannot end early, because the leader's own arrival is still pending until its expect_tx.
        if (leader) mbar_expect_tx(full_bar(s), 2 * L::STAGE_BYTES);
        tma_load_2d_pair(sa, &tmA, kb * TC_BK, m0, full_leader);
        tma_load_2d_pair(sb, mapB, kb * TC_BK, brow0, full_leader);
        issued = kb + 1;
      }
      if (*abort_flag) {
        // let the copies already issued land before the CTA can exit (bounded)
        if (leader) {
          for (int kb = max(0, issued - STAGES); kb < issued; ++kb)
            mbar_wait(full_bar(kb % STAGES), (kb / STAGES) & 1, abort_flag + 1, p.status, 2000000ull);
        } else {
          const unsigned long long t0 = global_ns();
          while (global_ns() - t0 < 200000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: the leader alone, for both CTAs
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = idesc_bf16_pair(BN);
      bool ok = true;
      for (int kb = 0; kb < KT && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(full_bar(s), ph, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = base + s * L::STAGE_BYTES, sb = sa + L::A_BYTES;
        const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
#pragma unroll
        for (int k = 0; k < TC_BK / 16; ++k)
          tc_mma_pair_f16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0);
        tc_commit_pair(empty_bar(s), 3);  // frees this stage in both CTAs once the MMAs above have read it
      }
      if (ok) tc_commit_pair(tmem_full_bar, 3);
    }
  } else {
    // ---------------- epilogue: warps 2..5 of both CTAs, each CTA its own 128 rows
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int gr = m0 + row;
    const bool row_ok = gr < p.M;
    const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16);
    uint4 pre[EPI == EPI_RESIDUAL ? BN / 8 : (EPI == EPI_QKV ? 32 : 1)];
    int qkv_pos = -1;
    if (EPI == EPI_RESIDUAL) tc_prefetch_residual<BN>(p, gr, row_ok, nt, *reinterpret_cast<uint4(*)[BN / 8]>(pre));
    if (EPI == EPI_QKV) qkv_pos = tc_prefetch_rope(p, gr, row_ok, seg, *reinterpret_cast<uint4(*)[32]>(pre));
    const bool ready = mbar_wait(tmem_full_bar, 0, abort_flag, p.status);
    tc_fence_after();
    if (ready) tc_epilogue_row<EPI, BN>(p, trow, gr, row_ok, nt, seg, nb0, pre, qkv_pos);
  }
  tc_fence_before();
  cluster_sync_all();  // neither CTA releases tensor or shared memory while the other may still use it
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256) : "memory");
}

// ---------------------------------------------------------------- host side
template <int EPI, int BN, int STAGES>
static int launch_tc(const a3_handle* h, const GemmArgs& a, const TcParams& p, int tiles, cudaStream_t st) {
  using L = TcLayout<BN, STAGES>;
  CUtensorMap tA, tB[3], tN[2];
  A3_TRY(make_tmap(&tA, a.A, a.M, a.K, TC_BM));
  if (EPI == EPI_SWIGLU) {
    A3_TRY(make_tmap(&tB[0], a.seg[0].B, a.seg[0].n, a.K, BN / 2));
    A3_TRY(make_tmap(&tB[1], a.B2, a.seg[0].n, a.K, BN / 2));
    tB[2] = tB[0];
    if (p.g_narrow > 0) {
      A3_TRY(make_tmap(&tN[0], a.seg[0].B, a.seg[0].n, a.K, p.g_narrow));
      A3_TRY(make_tmap(&tN[1], a.B2, a.seg[0].n, a.K, p.g_narrow));
    }
  } else {
    for (int s = 0; s < 3; ++s) {
      // head tiles (QKV, BN > 256) load one 128-row head per copy
      if (s < a.nseg) A3_TRY(make_tmap(&tB[s], a.seg[s].B, a.seg[s].n, a.K, (EPI == EPI_QKV && BN > 256) ? 128 : BN));
      else tB[s] = tB[0];
    }
  }
  static SmemAttrOnce attr;
  A3_TRY(smem_attr_once(attr, h->device, gemm_tc_kernel<EPI, BN, STAGES>, L::SMEM_BYTES));
  dim3 grid(cdiv(a.M, TC_BM), tiles);
  ProfScope prof(h, EPI == EPI_RESIDUAL ? A3_K_GEMM_RESIDUAL : EPI == EPI_SWIGLU ? A3_K_GEMM_SWIGLU : A3_K_GEMM_QKV, st);
  if (!(EPI == EPI_SWIGLU && p.g_narrow > 0)) tN[0] = tN[1] = tB[0];
  A3_CUDA(launch_pdl(gemm_tc_kernel<EPI, BN, STAGES>, grid, dim3(TC_THREADS), (size_t)L::SMEM_BYTES, st, tA, tB[0], tB[1], tB[2], tN[0], tN[1], p));
  A3_LAUNCHED();
  return A3_OK;
}

template <int EPI, int STAGES>
static int launch_pair(const a3_handle* h, const GemmArgs& a, const TcParams& p, int tiles, cudaStream_t st) {
  using L = PairLayout<STAGES>;
  CUtensorMap tA, tB[3];
  A3_TRY(make_tmap(&tA, a.A, a.M, a.K, TC_BM));
  if (EPI == EPI_SWIGLU) {
    A3_TRY(make_tmap(&tB[0], a.seg[0].B, a.seg[0].n, a.K, PAIR_BN / 2));
    A3_TRY(make_tmap(&tB[1], a.B2, a.seg[0].n, a.K, PAIR_BN / 2));
    tB[2] = tB[0];
  } else {
    for (int s = 0; s < 3; ++s) {
      if (s < a.nseg) A3_TRY(make_tmap(&tB[s], a.seg[s].B, a.seg[s].n, a.K, PAIR_BN / 2));
      else tB[s] = tB[0];
    }
  }
  static SmemAttrOnce attr;
  A3_TRY(smem_attr_once(attr, h->device, gemm_pair_kernel<EPI, STAGES>, L::SMEM_BYTES));
  dim3 grid(2 * cdiv(cdiv(a.M, TC_BM), 2), tiles);  // whole pairs: a last odd row tile gets an all-padding partner
  ProfScope prof(h, EPI == EPI_RESIDUAL ? A3_K_GEMM_RESIDUAL : EPI == EPI_SWIGLU ? A3_K_GEMM_SWIGLU : A3_K_GEMM_QKV, st);
  A3_CUDA(launch_pdl(gemm_pair_kernel<EPI, STAGES>, grid, dim3(TC_THREADS), (size_t)L::SMEM_BYTES, st, tA, tB[0], tB[1], tB[2], p));
  A3_LAUNCHED();
  return A3_OK;
}

// Tile width / pipeline depth per epilogue [EPI_RESIDUAL, EPI_SWIGLU, EPI_QKV] -> {BN, STAGES}; BN = 0 lets the
// launcher choose (a3_set_option pins a choice on a handle for cross-checks).  Measured on B200 at Llama-8B width:
// two co-resident CTAs per SM (256/2, 128/3) overlap one tile's epilogue with the other's main loop and win when
// the grid has several waves.  The CTA-pair kernel wins for the residual GEMMs (N = d_model: few tiles, one CTA per
// SM); for SwiGLU and QKV its extra all-padding row tile at 804 rows (7 -> 8) costs more than the halved B traffic
// saves: under the power cap the tensor work, not the L2 port, sets the pace.
// A3_OPT_SWIGLU_NARROW: 0: no narrower last wave in the SwiGLU grid; 1: choose; 16..120: that width on half the tiles.

template <int EPI>
static int dispatch_tc(const a3_handle* h, const GemmArgs& a, const TcParams& p, int tiles, int bn, int stages, cudaStream_t st) {
  if (bn == 512 && stages == 3) return launch_pair<EPI, 3>(h, a, p, tiles, st);
  if (bn == 512) return launch_pair<EPI, 6>(h, a, p, tiles, st);
  if constexpr (EPI == EPI_QKV) {
    if (bn == 384) return launch_tc<EPI, 384, 3>(h, a, p, tiles, st);
  }
  if (bn == 256 && stages == 4) return launch_tc<EPI, 256, 4>(h, a, p, tiles, st);
  if (bn == 256 && stages == 3) return launch_tc<EPI, 256, 3>(h, a, p, tiles, st);
  if (bn == 256 && stages == 2) return launch_tc<EPI, 256, 2>(h, a, p, tiles, st);
  if (bn == 224 && stages == 4) return launch_tc<EPI, 224, 4>(h, a, p, tiles, st);
  if (bn == 192 && stages == 4) return launch_tc<EPI, 192, 4>(h, a, p, tiles, st);
  if (bn == 128 && stages == 3) return launch_tc<EPI, 128, 3>(h, a, p, tiles, st);
  if (bn == 128 && stages == 6) return launch_tc<EPI, 128, 6>(h, a, p, tiles, st);
  return launch_tc<EPI, 128, 4>(h, a, p, tiles, st);
}

int gemm_bf16(const a3_handle* h, GemmEpilogue epi, const GemmArgs& a, cudaStream_t st) {
  if (a.M <= 0) return A3_OK;
  if (a.K % TC_BK) return A3_EUNSUPPORTED;
  if (epi == EPI_SWIGLU && swiglu_pair_usable(h, a)) return gemm_swiglu_pair(h, a, st);
  const int g_tc_narrow = h->opt[A3_OPT_SWIGLU_NARROW];
  int bn = h->opt[A3_OPT_GEMM_BN_RESIDUAL + (int)epi];
  int stages = h->opt[A3_OPT_GEMM_STAGES_RESIDUAL + (int)epi];
  if (epi == EPI_RESIDUAL && bn == 0 && residual_t_usable(h, a)) return gemm_residual_t(h, a, st);
  if (epi == EPI_QKV && bn == 0 && qkv_t_usable(h, a)) return gemm_qkv_t(h, a, st);

  if (bn == 0) {
    const int m_tiles = cdiv(a.M, TC_BM), sms = h->sm_count > 0 ? h->sm_count : 148;
    if (epi == EPI_RESIDUAL) {
      // the CTA-pair kernel (bn 512 selects it): measured 5-7 % faster than one CTA per 128 x 224/256 tile at
      // Llama-8B width for 804 and 5 152 rows
      (void)m_tiles;
      (void)sms;
      bn = 512;
      stages = 6;
    } else {
      bn = 256;
      stages = 4;
      // QKV at head dimension 128: tiles of two or three whole heads, whichever needs less tensor time per SM
      // (rounds of the grid x heads per tile).  804 rows of Llama-8B: 7 x 24 two-head tiles are two rounds on 148
      // SMs (4 head-times), 7 x 16 three-head tiles are one (3 head-times).
      if (epi == EPI_QKV && h->m.head_dim == 128 && a.nseg == 3) {
        bool whole = true;
        int heads = 0;
        for (int s = 0; s < 3; ++s) {
          whole = whole && a.seg[s].n % 128 == 0;
          heads += a.seg[s].n / 128;
        }
        if (whole && cdiv(m_tiles * cdiv(heads, 3), sms) * 3 < cdiv(m_tiles * cdiv(heads, 2), sms) * 2) {
          bn = 384;
          stages = 3;
        }
      }
    }
  }
  // output columns per tile; QKV tiles must hold whole heads and divide every segment
  bool pair = bn == 512;  // the CTA-pair kernel: 256 accumulator columns over two CTAs
  if (pair) {
    bn = PAIR_BN;
    if (epi != EPI_RESIDUAL)
      for (int s = 0; s < a.nseg; ++s)
        if (a.seg[s].n % (epi == EPI_SWIGLU ? PAIR_BN / 2 : PAIR_BN)) pair = false;  // falls back to one CTA per tile
    if (!pair) stages = 4;
  }
  int out_cols = epi == EPI_SWIGLU ? bn / 2 : bn;
  const bool head_tiles = epi == EPI_QKV && bn == 384;
  if (head_tiles) {
    if (h->m.head_dim != 128 || a.nseg != 3) return A3_EUNSUPPORTED;
    for (int s = 0; s < 3; ++s)
      if (a.seg[s].n % 128) return A3_EUNSUPPORTED;
  } else if (epi == EPI_QKV) {
    for (int s = 0; s < a.nseg; ++s)
      if (a.seg[s].n % out_cols) {
        bn = out_cols = 128;
        stages = 3;
      }
  }
  TcParams p{};
  p.M = a.M;
  p.K = a.K;
  int tiles = 0, heads = 0;
  for (int s = 0; s < 3; ++s) {
    if (s < a.nseg) heads += a.seg[s].n / 128;
    p.seg_heads_end[s] = heads;
  }
  for (int s = 0; s < 3; ++s) {
    if (s < a.nseg) {
      if (epi != EPI_RESIDUAL && !head_tiles && a.seg[s].n % out_cols) return A3_EUNSUPPORTED;
      if (a.seg[s].n % 32) return A3_EUNSUPPORTED;
      p.bias[s] = a.seg[s].bias;
      p.kind[s] = a.seg[s].kind;
      tiles += cdiv(a.seg[s].n, out_cols);
    }
    p.seg_tiles_end[s] = tiles;
  }
  if (head_tiles) tiles = cdiv(heads, 3);
  // SwiGLU with two CTAs per SM: the grid runs in waves of 2 x SMs tiles and a partly filled last wave costs a whole
  // one (measured: 58 us per wave at Llama-8B width whatever its fill).  The column tiles of the last wave are
  // therefore made narrower, so that they all fit into it: a wave's time follows the bytes its tiles pull through
  // the SM's L2 port (A: 128 rows, B: 2 g rows per k-block), i.e. (128 + 2 g) / 384 of a full one.
  if (epi == EPI_SWIGLU && bn == 256 && stages == 2 && g_tc_narrow && a.seg[0].n % 128 == 0) {
    const int m_tiles = cdiv(a.M, TC_BM), slots = 2 * (h->sm_count > 0 ? h->sm_count : 148), ct = a.seg[0].n / 128;
    const int total = m_tiles * ct, waves_full = total / slots;
    if (g_tc_narrow >= 16 && g_tc_narrow < 128 && g_tc_narrow % 8 == 0 && ct >= 2) {  // forced (tests): half the tiles narrow
      p.y_wide = ct / 2;
      p.g_narrow = g_tc_narrow;
      tiles = p.y_wide + cdiv(a.seg[0].n - p.y_wide * 128, p.g_narrow);
    } else if (waves_full >= 1 && total % slots) {
      const int y_wide = waves_full * slots / m_tiles;
      const int rest = a.seg[0].n - y_wide * 128;
      const int per_row = (slots + waves_full * slots - y_wide * m_tiles) / m_tiles;
      const int rnd = 16;  // measured at 804..2 000 rows: widths that are multiples of 16 features never lose
      const int g = per_row > 0 ? cdiv(cdiv(rest, per_row), rnd) * rnd : 128;
      if (g >= 16 && g < 128) {
        p.y_wide = y_wide;
        p.g_narrow = g;
        tiles = y_wide + cdiv(rest, g);
      }
    }
  }
  p.N = a.seg[0].n;
  p.C = a.C;
  p.ldc = a.ldc;
  p.q_out = a.q_out;
  p.k_cache = a.k_cache;
  p.v_cache = a.v_cache;
  p.pos = a.pos;
  p.kv_len = a.kv_len;
  p.Hq = h->m.n_q_heads;
  p.Hkv = h->m.n_kv_heads;
  p.D = h->m.head_dim;
  p.layout = h->m.rope_layout;
  p.max_pos = h->m.max_positions;
  p.tab = h->rope_tab;
  p.status = h->dev_status;
  if (pair) bn = 512;
  if (epi == EPI_RESIDUAL) return dispatch_tc<EPI_RESIDUAL>(h, a, p, tiles, bn, stages, st);
  if (epi == EPI_SWIGLU) return dispatch_tc<EPI_SWIGLU>(h, a, p, tiles, bn, stages, st);
  return dispatch_tc<EPI_QKV>(h, a, p, tiles, bn, stages, st);
}

}  // namespace a3


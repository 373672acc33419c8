// Question->context relevance scores (Eq. 3): s_i = sum over question rows j and query heads h of
// Softmax_row(q_{j,h} K^T / sqrt(D))[i].  Question row j sits at global position q_pos[j] and sees slots 0..q_pos[j].
//
// The G = Hq/Hkv query heads that share one KV head are packed into one operand (flat row r -> token r / G, head
// r % G), so a K tile is read once per group rather than once per head.  The probability matrix is never
// materialised: the kernels take the rows' log-sum-exps (emitted by the attention kernel's statistics pass), form
// exp2(logit * scale - lse) in fp32 and add it up per cache slot in a fixed order, which makes the scores
// bit-reproducible from run to run.
//
// scores_tc_kernel (the one in use): tcgen05.  The product is taken TRANSPOSED, S^T = K_tile Q_g^T: the 128 cache
// slots of the CTA's key tile are the M side (one tensor-memory lane each), the packed question rows of KV head g
// the N side (up to 256 columns per instruction).  A thread of the accumulating warps therefore owns one cache
// slot and finds all of that slot's logits in its own lane: the sum over question rows and heads of Eq. 3 is a
// plain loop over its columns, with no exchange between threads; the row's log-sum-exp and position are the same
// for the whole warp and come from a small table in shared memory.
//   warp 0 (one lane)  TMA: the K tile of head g (two slots) and chunks of <= 256 packed question rows (two slots;
//                      a 3-D box over q seen as [nq][Hq][D] lands as the packed K-major operand)
//   warp 1 (one lane)  tcgen05.mma, accumulators double-buffered in tensor memory (2 x 256 columns)
//   warps 2..5         one cache slot per thread: p = ex2(s * scale - lse), masked where slot > position, summed
// scores_mma_kernel: the earlier warp-level mma.sync kernel, kept as the cross-check and for shapes the tcgen05
// kernel does not take (more than 16 query heads per KV head, more than 4096 (row, head) pairs).
#include <cuda.h>

#include "a3_internal.cuh"
#include "a3_attn.cuh"

namespace a3 {

constexpr int AT_THREADS = 128;  // 4 warps x 16 rows
constexpr int AT_BM = 64, AT_BN = 64;
constexpr float LOG2E = 1.4426950408889634f;

// byte offset of 16-byte chunk c of row r in a [rows][D] bf16 tile (row pitch D*2 bytes), XOR-swizzled
template <int D>
__device__ __forceinline__ uint32_t tswz(int r, int c) {
  return (uint32_t)(r * (D * 2) + ((c ^ (r & 7)) << 4));
}

// copies a [64][D] tile; row i comes from base + row_index(i)*stride (elements); invalid rows are zero-filled
template <int D, typename RowFn>
__device__ __forceinline__ void load_tile(uint32_t sdst, const bf16* safe, RowFn row_ptr) {
  constexpr int CPR = D / 8;
#pragma unroll
  for (int i = 0; i < (64 * CPR) / AT_THREADS; ++i) {
    int idx = threadIdx.x + i * AT_THREADS;
    int r = idx / CPR, c = idx % CPR;
    const bf16* src = row_ptr(r);
    cp_async16(sdst + tswz<D>(r, c), src ? src + c * 8 : safe, src != nullptr);
  }
}

template <int D>
__device__ __forceinline__ void load_q_frags(uint32_t sq, int warp, int lane, uint32_t (&qf)[D / 16][4]) {
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    int c = ks * 2 + (lane >> 4);
    ldmatrix_x4(sq + tswz<D>(r, c), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
  }
}

// S(16 x 64) = Q(16 x D) K_tile(64 x D)^T for this warp
template <int D>
__device__ __forceinline__ void qk_tile(uint32_t sk, int lane, const uint32_t (&qf)[D / 16][4], float (&s)[8][4]) {
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) s[j][e] = 0.f;
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      uint32_t b0, b1, b2, b3;
      int r = jj * 16 + (lane & 7) + (lane >> 4) * 8;
      int c = ks * 2 + ((lane >> 3) & 1);
      ldmatrix_x4(sk + tswz<D>(r, c), b0, b1, b2, b3);
      mma_bf16(s[2 * jj], qf[ks], b0, b1);
      mma_bf16(s[2 * jj + 1], qf[ks], b2, b3);
    }
  }
}

// ------------------------------------------------------------------ relevance scores (Eq. 3)
// One CTA per tile of 64 cache slots.  It loops over the KV heads and, per head, over blocks of 64 packed
// question rows; column sums stay on chip and are added in a fixed order.
template <int D>
__global__ void __launch_bounds__(AT_THREADS)
scores_mma_kernel(const bf16* __restrict__ q, const int32_t* __restrict__ q_pos, int nq, const bf16* __restrict__ k,
              int kv_len, int cand_begin, int cand_end, const float* __restrict__ lse, float* __restrict__ scores,
              int Hq, int Hkv, float scale_log2, float* __restrict__ per_head) {
  __shared__ __align__(128) unsigned char smem[2 * 64 * D * 2];
  __shared__ float colpart[4][AT_BN];
  const uint32_t sq = smem_u32(smem), sk = sq + 64 * D * 2;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gq = lane >> 2, tq = lane & 3;
  const int G = Hq / Hkv;
  const int key0 = blockIdx.x * AT_BN;
  const int rows_total = nq * G;
  const int nrb = (rows_total + AT_BM - 1) / AT_BM;
  const int kvrow = Hkv * D;
  float total = 0.f;  // thread c < 64 owns cache slot key0 + c
  float head_total = 0.f;

  // gridDim.y == 1: this CTA walks all KV heads (their sum is Eq. 3's score); gridDim.y == Hkv: one KV head per CTA
  // (the per-head votes of the eviction step, where no sum over heads is wanted)
  const int g_begin = gridDim.y == 1 ? 0 : blockIdx.y, g_end = gridDim.y == 1 ? Hkv : blockIdx.y + 1;
  for (int g = g_begin; g < g_end; ++g) {
    __syncthreads();  // previous users of sk / sq are done
    load_tile<D>(sk, k, [&](int r) -> const bf16* {
      int key = key0 + r;
      return key < kv_len ? k + (size_t)key * kvrow + g * D : nullptr;
    });
    for (int rb = 0; rb < nrb; ++rb) {
      const int r0 = rb * AT_BM;
      if (rb > 0) __syncthreads();
      load_tile<D>(sq, q, [&](int r) -> const bf16* {
        int fr = r0 + r;
        if (fr >= rows_total) return nullptr;
        return q + ((size_t)(fr / G) * Hq + g * G + fr % G) * D;
      });
      cp_async_commit();
      cp_async_wait<0>();
      __syncthreads();
      uint32_t qf[D / 16][4];
      load_q_frags<D>(sq, warp, lane, qf);
      float s[8][4];
      qk_tile<D>(sk, lane, qf, s);
      int lim[2];
      float l2[2];
#pragma unroll
      for (int hlf = 0; hlf < 2; ++hlf) {
        int fr = r0 + warp * 16 + gq + hlf * 8;
        if (fr < rows_total) {
          int t = fr / G, hq = g * G + fr % G;
          lim[hlf] = min(q_pos[t], kv_len - 1);
          l2[hlf] = lse[(size_t)t * Hq + hq] * LOG2E;
        } else {
          lim[hlf] = -1;
          l2[hlf] = 0.f;
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float c0 = 0.f, c1 = 0.f;  // columns j*8 + 2*tq, +1: rows gq and gq+8
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
          int key = key0 + j * 8 + 2 * tq;
          float p0 = key <= lim[hlf] ? exp2f(s[j][2 * hlf] * scale_log2 - l2[hlf]) : 0.f;
          float p1 = key + 1 <= lim[hlf] ? exp2f(s[j][2 * hlf + 1] * scale_log2 - l2[hlf]) : 0.f;
          c0 += p0;
          c1 += p1;
        }
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
          c0 += __shfl_xor_sync(0xffffffffu, c0, off);
          c1 += __shfl_xor_sync(0xffffffffu, c1, off);
        }
        if (gq == 0) {
          colpart[warp][j * 8 + 2 * tq] = c0;
          colpart[warp][j * 8 + 2 * tq + 1] = c1;
        }
      }
      __syncthreads();
      if (tid < AT_BN) {
        const float part = (colpart[0][tid] + colpart[1][tid]) + (colpart[2][tid] + colpart[3][tid]);
        total += part;
        head_total += part;
      }
    }
    if (per_head) {  // the votes of this KV head's query heads alone (eviction step)
      const int key = key0 + tid;
      if (tid < AT_BN && key < kv_len) per_head[(size_t)g * kv_len + key] = (key >= cand_begin && key < cand_end) ? head_total : 0.f;
      head_total = 0.f;
    }
  }
  if (tid < AT_BN) {
    int key = key0 + tid;
    if (key < kv_len && scores) scores[key] = (key >= cand_begin && key < cand_end) ? total : 0.f;
  }
}

// ------------------------------------------------------------------ relevance scores on tcgen05
constexpr int STC_THREADS = 192;
constexpr int STC_MAX_PAIRS = 4096;  // (question row, query head) pairs whose log-sum-exps fit the shared-memory table

struct StcParams {
  const int32_t* q_pos;
  const float* lse;
  float* scores;
  float* per_head;
  int nq, kv_len, cand_begin, cand_end, Hq, Hkv;
  int nq_tile;   // question rows per chunk (multiple of 16); a chunk has N = G * nq_tile packed rows
  int n_chunks;  // chunks per KV head
  float scale_log2;
  uint32_t* status;
};

// dynamic shared memory: [K slot 0][K slot 1][Q slot 0][Q slot 1][l2 table][position table][barriers]
template <int D>
struct StcLayout {
  static constexpr int K_SLOT = (D / 64) * 128 * 128;  // [128 slots][64] bf16 sub-tiles
  __host__ __device__ static constexpr int q_slot(int n_cols) { return (D / 64) * n_cols * 128; }
  static constexpr int TAB_BYTES = STC_MAX_PAIRS * 4 + STC_MAX_PAIRS * 4;  // l2[Hkv][rows_g], position per packed row
  static int smem_bytes(int n_cols) { return 2 * K_SLOT + 2 * q_slot(n_cols) + TAB_BYTES + 256 + 1024; }
};

template <int D>
__global__ void __launch_bounds__(STC_THREADS, 1)
scores_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ, const StcParams p) {
  using L = StcLayout<D>;
  using namespace atc;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int G = p.Hq / p.Hkv;
  const int N = G * p.nq_tile;     // columns of one instruction (multiple of 16, at most 256)
  const int rows_g = p.nq * G;     // packed question rows of one KV head
  const int q_slot = L::q_slot(N);
  const uint32_t k_off = 0, q_off = 2 * L::K_SLOT, tab_off = q_off + 2 * q_slot, bar_off = tab_off + L::TAB_BYTES;
  float* l2tab = reinterpret_cast<float*>(base_ptr + tab_off);                  // [Hkv][rows_g]: lse * log2(e)
  int* postab = reinterpret_cast<int*>(base_ptr + tab_off + STC_MAX_PAIRS * 4);  // [rows_g]: position of the packed row
  const uint32_t bars = base + bar_off;
  auto k_full = [&](int s) { return bars + 8u * s; };
  auto k_empty = [&](int s) { return bars + 8u * (2 + s); };
  auto q_full = [&](int s) { return bars + 8u * (4 + s); };
  auto q_empty = [&](int s) { return bars + 8u * (6 + s); };
  auto t_full = [&](int b) { return bars + 8u * (8 + b); };
  auto t_empty = [&](int b) { return bars + 8u * (10 + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + bar_off + 8 * 12);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + bar_off + 8 * 12 + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int key0 = blockIdx.x * 128;
  // gridDim.y == 1: all KV heads, summed (Eq. 3); gridDim.y == Hkv: one KV head per CTA (per-head votes only)
  const int g_begin = gridDim.y == 1 ? 0 : blockIdx.y, g_end = gridDim.y == 1 ? p.Hkv : blockIdx.y + 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(k_full(i), 1);
      mbar_init(k_empty(i), 1);
      mbar_init(q_full(i), 1);
      mbar_init(q_empty(i), 1);
      mbar_init(t_full(i), 1);
      mbar_init(t_empty(i), 4);  // one arrival per accumulating warp
    }
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
  pdl_wait();  // everything above overlapped the previous kernel's tail; the log-sum-exps and K are read below
  pdl_launch_dependents();
  // tables: log-sum-exps in the exp2 domain in packed order per KV head, and each packed row's position
  for (int i = threadIdx.x; i < p.Hkv * rows_g; i += STC_THREADS) {
    const int g = i / rows_g, r = i - g * rows_g;
    l2tab[i] = p.lse[(size_t)(r / G) * p.Hq + g * G + r % G] * ATC_LOG2E;
  }
  for (int r = threadIdx.x; r < rows_g; r += STC_THREADS) postab[r] = min(p.q_pos[r / G], p.kv_len - 1);
  __syncthreads();

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQ) : "memory");
      uint32_t st = 0, gi = 0;
      bool ok = true;
      for (int g = g_begin; g < g_end && ok; ++g, ++gi) {
        const int ks = gi & 1;
        ok = mbar_wait(k_empty(ks), ((gi >> 1) & 1) ^ 1, abort_flag, p.status);
        if (!ok) break;
        mbar_expect_tx(k_full(ks), L::K_SLOT);
#pragma unroll
        for (int j = 0; j < D / 64; ++j) tma_load_2d(base + k_off + ks * L::K_SLOT + j * (128 * 128), &tmK, g * D + 64 * j, key0, k_full(ks));
        for (int c = 0; c < p.n_chunks; ++c, ++st) {
          const int qs = st & 1;
          ok = mbar_wait(q_empty(qs), ((st >> 1) & 1) ^ 1, abort_flag, p.status);
          if (!ok) break;
          mbar_expect_tx(q_full(qs), (uint32_t)q_slot);
#pragma unroll
          for (int j = 0; j < D / 64; ++j) {
            const uint32_t dst = base + q_off + qs * q_slot + j * (N * 128);
            asm volatile("cp.async.bulk.tensor.3d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                         ::"r"(dst), "l"(&tmQ), "r"(64 * j), "r"(g * G), "r"(c * p.nq_tile), "r"(q_full(qs))
                         : "memory");
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: S^T (128 slots x N packed rows) = K_tile Q_chunk^T
    if (lane == 0) {
      const uint32_t id = idesc(N, 0);
      uint32_t st = 0, gi = 0;
      bool ok = true;
      for (int g = g_begin; g < g_end && ok; ++g, ++gi) {
        const int ks = gi & 1;
        ok = mbar_wait(k_full(ks), (gi >> 1) & 1, abort_flag, p.status);
        for (int c = 0; c < p.n_chunks && ok; ++c, ++st) {
          const int b = st & 1;
          ok = mbar_wait(q_full(b), (st >> 1) & 1, abort_flag, p.status) &&
               mbar_wait(t_empty(b), ((st >> 1) & 1) ^ 1, abort_flag, p.status);
          if (!ok) break;
          fence_after();
          const uint32_t sk = base + k_off + ks * L::K_SLOT, sq = base + q_off + b * q_slot;
#pragma unroll
          for (int k = 0; k < D / 16; ++k)
            mma_f16(tmem_base + b * 256, desc_k_sw128(sk + (k / 4) * (128 * 128) + (k % 4) * 32),
                    desc_k_sw128(sq + (k / 4) * (N * 128) + (k % 4) * 32), id, k != 0);
          commit(t_full(b));
          commit(q_empty(b));
          if (c == p.n_chunks - 1) commit(k_empty(ks));
        }
      }
    }
  } else {
    // ---------------- accumulation: one cache slot per thread
    const int quarter = warp & 3;
    const int key = key0 + quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    // question rows sit behind the context, so only the key tiles that reach past the first question row need a mask
    const bool need_mask = key0 + 127 > postab[0];
    const bool vec_ok = (rows_g & 3) == 0;  // the table rows of every head start on a 16-byte boundary
    const bool cand = key >= p.cand_begin && key < p.cand_end;
    float total = 0.f;
    uint32_t st = 0;
    bool ok = true;
    for (int g = g_begin; g < g_end && ok; ++g) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const float* l2g = l2tab + g * rows_g;
      for (int c = 0; c < p.n_chunks; ++c, ++st) {
        const int b = st & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(t_full(b), (st >> 1) & 1, abort_flag, p.status));
        if (!ok) break;
        fence_after();
        const int r0 = c * N;
        const int n_valid = min(N, rows_g - r0);  // packed rows beyond the question are zero-filled operands: skipped
        const int n32 = (n_valid + 31) >> 5;
#pragma unroll 1
        for (int cc = 0; cc < n32; ++cc) {
          float x[32];
          ld32(tmem_base + b * 256 + lane_addr + cc * 32, x);
          wait_ld();
          const int rb = r0 + cc * 32;
          const bool whole = rb + 32 <= r0 + n_valid && vec_ok;  // 32 live packed rows, tables readable as vectors
          if (whole && !need_mask) {
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              const float4 l4 = *reinterpret_cast<const float4*>(l2g + rb + e);
              acc[0] += ex2_approx(fmaf(x[e], p.scale_log2, -l4.x));
              acc[1] += ex2_approx(fmaf(x[e + 1], p.scale_log2, -l4.y));
              acc[2] += ex2_approx(fmaf(x[e + 2], p.scale_log2, -l4.z));
              acc[3] += ex2_approx(fmaf(x[e + 3], p.scale_log2, -l4.w));
            }
          } else if (whole) {
            // the key tiles around the question: a slot counts for a row only up to the row's own position
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              const float4 l4 = *reinterpret_cast<const float4*>(l2g + rb + e);
              const int4 m4 = *reinterpret_cast<const int4*>(postab + rb + e);
              const float p0 = ex2_approx(fmaf(x[e], p.scale_log2, -l4.x)), p1 = ex2_approx(fmaf(x[e + 1], p.scale_log2, -l4.y));
              const float p2 = ex2_approx(fmaf(x[e + 2], p.scale_log2, -l4.z)), p3 = ex2_approx(fmaf(x[e + 3], p.scale_log2, -l4.w));
              acc[0] += key <= m4.x ? p0 : 0.f;
              acc[1] += key <= m4.y ? p1 : 0.f;
              acc[2] += key <= m4.z ? p2 : 0.f;
              acc[3] += key <= m4.w ? p3 : 0.f;
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int r = rb + e;
              const bool live = r < r0 + n_valid;
              const float l2v = live ? l2g[r] : 0.f;
              const int lim = live ? postab[r] : -1;
              const float pv = ex2_approx(fmaf(x[e], p.scale_log2, -l2v));
              acc[e & 3] += key <= lim ? pv : 0.f;
            }
          }
        }
        // this warp has read its part of the accumulator: hand it back to the MMA issuer
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(t_empty(b));
      }
      const float head_total = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      total += head_total;
      if (p.per_head && key < p.kv_len) p.per_head[(size_t)g * p.kv_len + key] = cand ? head_total : 0.f;
    }
    if (ok && p.scores && key < p.kv_len) p.scores[key] = cand ? total : 0.f;
  }
  fence_before();
  __syncthreads();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

typedef CUresult (*EncodeTiledFn3)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn3 stc_encode_fn() {
  static EncodeTiledFn3 fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn3)ptr;
  }
  return fn;
}

// The shapes the tcgen05 kernel takes: nq_tile question rows per chunk such that G * nq_tile <= 256 columns.
static bool stc_shape(const a3_handle* h, int nq, int* nq_tile, int* n_chunks) {
  const int Hq = h->m.n_q_heads, G = Hq / h->m.n_kv_heads;
  if (nq <= 0 || G > 16 || (long long)nq * Hq > STC_MAX_PAIRS) return false;
  int t = (256 / G) / 16 * 16;                 // multiple of 16, so that N = G * t is one too
  const int need = (nq + 15) / 16 * 16;
  if (t > need) t = need;
  if (t <= 0) return false;
  *nq_tile = t;
  *n_chunks = (nq + t - 1) / t;
  return true;
}

template <int D>
static int launch_scores_tc(const a3_handle* h, const bf16* q, const int32_t* q_pos, int nq, const bf16* k, int kv_len, int cand_begin,
                            int cand_end, const float* lse, float* scores, float* per_head, int nq_tile, int n_chunks, cudaStream_t st) {
  using L = StcLayout<D>;
  const int Hq = h->m.n_q_heads, Hkv = h->m.n_kv_heads, G = Hq / Hkv;
  EncodeTiledFn3 fn = stc_encode_fn();
  if (!fn) return A3_ECUDA;
  CUtensorMap tK, tQ;
  {
    cuuint64_t dims[2] = {(cuuint64_t)Hkv * D, (cuuint64_t)kv_len};
    cuuint64_t strides[1] = {(cuuint64_t)Hkv * D * 2};
    cuuint32_t box[2] = {64, 128}, estr[2] = {1, 1};
    CUresult r = fn(&tK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(k), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
      g_last_cuda_error = (int)r;
      return A3_ECUDA;
    }
  }
  {
    // q [nq][Hq][D] as a 3-D tensor; a box of 64 channels x G heads x nq_tile rows is the packed operand of one KV head
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)nq};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hq * D * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)nq_tile}, estr[3] = {1, 1, 1};
    CUresult r = fn(&tQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(q), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
      g_last_cuda_error = (int)r;
      return A3_ECUDA;
    }
  }
  StcParams p{};
  p.q_pos = q_pos;
  p.lse = lse;
  p.scores = scores;
  p.per_head = per_head;
  p.nq = nq;
  p.kv_len = kv_len;
  p.cand_begin = cand_begin;
  p.cand_end = cand_end;
  p.Hq = Hq;
  p.Hkv = Hkv;
  p.nq_tile = nq_tile;
  p.n_chunks = n_chunks;
  p.scale_log2 = LOG2E / sqrtf((float)D);
  p.status = h->dev_status;
  const int smem = L::smem_bytes(G * nq_tile);
  static SmemAttrOnce attr;
  A3_TRY(smem_attr_once(attr, h->device, scores_tc_kernel<D>, L::smem_bytes(256)));
  dim3 grid(cdiv(kv_len, 128), (per_head && !scores) ? Hkv : 1);
  A3_CUDA(launch_pdl(scores_tc_kernel<D>, grid, dim3(STC_THREADS), (size_t)smem, st, tK, tQ, p));
  A3_LAUNCHED();
  return A3_OK;
}

int scores_pass(const a3_handle* h, const bf16* q, const int32_t* q_pos, int nq, const bf16* k, int kv_len,
                int cand_begin, int cand_end, const float* lse, float* scores, cudaStream_t st, float* per_head) {
  if (kv_len <= 0) return A3_OK;
  const int Hq = h->m.n_q_heads, Hkv = h->m.n_kv_heads, D = h->m.head_dim;
  ProfScope prof(h, A3_K_SCORES, st);
  int nq_tile = 0, n_chunks = 0;
  const int variant = h->opt[A3_OPT_SCORES_KERNEL];
  if (variant != 2 && stc_shape(h, nq, &nq_tile, &n_chunks)) {
    if (D == 128) return launch_scores_tc<128>(h, q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, per_head, nq_tile, n_chunks, st);
    return launch_scores_tc<64>(h, q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, per_head, nq_tile, n_chunks, st);
  }
  const float scale_log2 = LOG2E / sqrtf((float)D);
  dim3 grid(cdiv(kv_len, AT_BN), (per_head && !scores) ? Hkv : 1);
  if (D == 128) scores_mma_kernel<128><<<grid, AT_THREADS, 0, st>>>(q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, Hq, Hkv, scale_log2, per_head);
  else scores_mma_kernel<64><<<grid, AT_THREADS, 0, st>>>(q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, Hq, Hkv, scale_log2, per_head);
  A3_LAUNCHED();
  return A3_OK;
}

}  // namespace a3

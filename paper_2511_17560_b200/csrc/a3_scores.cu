// Question->context relevance scores (Eq. 3): s_i = sum over question rows j and query heads h of
// Softmax_row(q_{j,h} K^T / sqrt(D))[i].  Question row j sits at global position q_pos[j] and sees slots 0..q_pos[j].
//
// The G = Hq/Hkv query heads that share one KV head are packed into the row dimension of the tile (flat row r ->
// token r / G, head r % G), so a K tile is read once per group rather than once per head.  The probability matrix
// is never materialised: the kernel takes the rows' log-sum-exps (emitted by the attention kernel), forms
// exp2(logit - lse) from warp-level tensor-core QK^T fragments, reduces it down the rows with warp shuffles and
// adds heads in a fixed order, which makes the scores bit-reproducible from run to run.
#include "a3_internal.cuh"

namespace a3 {

constexpr int AT_THREADS = 128;  // 4 warps x 16 rows
constexpr int AT_BM = 64, AT_BN = 64;
constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;

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
scores_kernel(const bf16* __restrict__ q, const int32_t* __restrict__ q_pos, int nq, const bf16* __restrict__ k,
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

int scores_pass(const a3_handle* h, const bf16* q, const int32_t* q_pos, int nq, const bf16* k, int kv_len,
                int cand_begin, int cand_end, const float* lse, float* scores, cudaStream_t st, float* per_head) {
  if (kv_len <= 0) return A3_OK;
  const int Hq = h->m.n_q_heads, Hkv = h->m.n_kv_heads, D = h->m.head_dim;
  const float scale_log2 = LOG2E / sqrtf((float)D);
  dim3 grid(cdiv(kv_len, AT_BN), (per_head && !scores) ? Hkv : 1);
  ProfScope prof(h, A3_K_SCORES, st);
  if (D == 128) scores_kernel<128><<<grid, AT_THREADS, 0, st>>>(q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, Hq, Hkv, scale_log2, per_head);
  else scores_kernel<64><<<grid, AT_THREADS, 0, st>>>(q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, Hq, Hkv, scale_log2, per_head);
  A3_LAUNCHED();
  return A3_OK;
}

}  // namespace a3

// Attention of the carried rows over the fused GQA cache (Eq. 4, Eq. 5) and the question->context relevance
// scores (Eq. 3).  Row m sits at global position pos[m] and sees cache slots 0..pos[m].
//
// Both kernels pack the G = Hq/Hkv query heads that share one KV head into the row dimension of the tile
// (flat row r -> token r / G, head r % G), so a K/V tile is read once per group rather than once per head.
// Softmax statistics are fp32 in the exp2 domain; the score kernel never materialises the probability
// matrix: it reduces exp(logit - lse) down the rows with warp shuffles and sums heads in a fixed order,
// which makes the scores bit-reproducible from run to run.
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

// ------------------------------------------------------------------ attention
template <int D>
__global__ void __launch_bounds__(AT_THREADS)
attention_kernel(const bf16* __restrict__ q, const int32_t* __restrict__ pos, int M, const bf16* __restrict__ k,
                 const bf16* __restrict__ v, int kv_len, bf16* __restrict__ o, float* __restrict__ lse, int Hq, int Hkv,
                 float scale_log2) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int TILE = 64 * D * 2;
  const uint32_t sq = smem_u32(smem);
  const uint32_t skv = sq + TILE;  // [stage][K,V]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = Hq / Hkv;
  const int g = blockIdx.y;
  const int tile = gridDim.x - 1 - blockIdx.x;  // heaviest (latest) row tiles first
  const int r0 = tile * AT_BM;
  const int rows_total = M * G;
  const int kvrow = Hkv * D;

  auto q_row = [&](int r) -> const bf16* {
    int fr = r0 + r;
    if (fr >= rows_total) return nullptr;
    int t = fr / G, hg = fr % G;
    return q + ((size_t)t * Hq + g * G + hg) * D;
  };
  int last_tok = min(M - 1, (r0 + AT_BM - 1) / G);
  int maxpos = min(pos[last_tok], kv_len - 1);
  const int minpos = pos[r0 / G];
  const int nkt = maxpos < 0 ? 0 : maxpos / AT_BN + 1;

  auto load_kv = [&](int stage, int kt) {
    const int key0 = kt * AT_BN;
    load_tile<D>(skv + stage * 2 * TILE, k, [&](int r) -> const bf16* {
      int key = key0 + r;
      return key <= maxpos ? k + (size_t)key * kvrow + g * D : nullptr;
    });
    load_tile<D>(skv + stage * 2 * TILE + TILE, v, [&](int r) -> const bf16* {
      int key = key0 + r;
      return key <= maxpos ? v + (size_t)key * kvrow + g * D : nullptr;
    });
  };

  load_tile<D>(sq, q, q_row);
  if (nkt > 0) load_kv(0, 0);
  cp_async_commit();

  // row limits of the two rows this thread owns in the accumulator layout
  const int gq = lane >> 2, tq = lane & 3;
  int lim[2];
#pragma unroll
  for (int hlf = 0; hlf < 2; ++hlf) {
    int fr = r0 + warp * 16 + gq + hlf * 8;
    lim[hlf] = fr < rows_total ? min(pos[fr / G], kv_len - 1) : -1;
  }

  uint32_t qf[D / 16][4];
  float oacc[D / 8][4];
#pragma unroll
  for (int j = 0; j < D / 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[j][e] = 0.f;
  float mx[2] = {-INFINITY, -INFINITY}, lsum[2] = {0.f, 0.f};

  for (int kt = 0; kt < nkt; ++kt) {
    if (kt + 1 < nkt) load_kv((kt + 1) & 1, kt + 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (kt == 0) load_q_frags<D>(sq, warp, lane, qf);
    const uint32_t sk = skv + (kt & 1) * 2 * TILE, sv = sk + TILE;

    float s[8][4];
    qk_tile<D>(sk, lane, qf, s);

    const int key0 = kt * AT_BN;
    const bool need_mask = key0 + AT_BN - 1 > minpos;
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float x = s[j][e] * scale_log2;
        if (need_mask) {
          int key = key0 + j * 8 + 2 * tq + (e & 1);
          if (key > lim[e >> 1]) x = -INFINITY;
        }
        s[j][e] = x;
        tmax[e >> 1] = fmaxf(tmax[e >> 1], x);
      }
    float alpha[2], mref[2];
#pragma unroll
    for (int hlf = 0; hlf < 2; ++hlf) {
      tmax[hlf] = fmaxf(tmax[hlf], __shfl_xor_sync(0xffffffffu, tmax[hlf], 1));
      tmax[hlf] = fmaxf(tmax[hlf], __shfl_xor_sync(0xffffffffu, tmax[hlf], 2));
      float mnew = fmaxf(mx[hlf], tmax[hlf]);
      mref[hlf] = mnew == -INFINITY ? 0.f : mnew;
      alpha[hlf] = exp2f(mx[hlf] - mref[hlf]);  // mx = -inf -> 0
      mx[hlf] = mnew;
      lsum[hlf] *= alpha[hlf];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float pe = exp2f(s[j][e] - mref[e >> 1]);
        s[j][e] = pe;
        lsum[e >> 1] += pe;
      }
#pragma unroll
    for (int j = 0; j < D / 8; ++j) {
      oacc[j][0] *= alpha[0];
      oacc[j][1] *= alpha[0];
      oacc[j][2] *= alpha[1];
      oacc[j][3] *= alpha[1];
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < AT_BN / 16; ++kk) {
      uint32_t pa[4];
      pa[0] = pack2(s[2 * kk][0], s[2 * kk][1]);
      pa[1] = pack2(s[2 * kk][2], s[2 * kk][3]);
      pa[2] = pack2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      pa[3] = pack2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
      for (int jd = 0; jd < D / 16; ++jd) {
        uint32_t b0, b1, b2, b3;
        int mi = lane >> 3;
        int r = kk * 16 + (lane & 7) + (mi & 1) * 8;
        int c = jd * 2 + (mi >> 1);
        ldmatrix_x4_trans(sv + tswz<D>(r, c), b0, b1, b2, b3);
        mma_bf16(oacc[2 * jd], pa, b0, b1);
        mma_bf16(oacc[2 * jd + 1], pa, b2, b3);
      }
    }
    __syncthreads();  // everyone is done with this stage before it is refilled
  }
  cp_async_wait<0>();

#pragma unroll
  for (int hlf = 0; hlf < 2; ++hlf) {
    lsum[hlf] += __shfl_xor_sync(0xffffffffu, lsum[hlf], 1);
    lsum[hlf] += __shfl_xor_sync(0xffffffffu, lsum[hlf], 2);
  }
#pragma unroll
  for (int hlf = 0; hlf < 2; ++hlf) {
    int fr = r0 + warp * 16 + gq + hlf * 8;
    if (fr >= rows_total) continue;
    int t = fr / G, hq = g * G + fr % G;
    float inv = lsum[hlf] > 0.f ? 1.f / lsum[hlf] : 0.f;
    if (o) {
      bf16* orow = o + ((size_t)t * Hq + hq) * D;
#pragma unroll
      for (int j = 0; j < D / 8; ++j)
        *reinterpret_cast<uint32_t*>(orow + j * 8 + 2 * tq) = pack2(oacc[j][2 * hlf] * inv, oacc[j][2 * hlf + 1] * inv);
    }
    if (lse && tq == 0) lse[(size_t)t * Hq + hq] = lsum[hlf] > 0.f ? (mx[hlf] + log2f(lsum[hlf])) * LN2 : -INFINITY;
  }
}

int attention_rows_tc(const a3_handle* h, const bf16* q, const int32_t* pos, int M, const bf16* k, const bf16* v,
                      int kv_len, bf16* o, float* lse, void* part, size_t part_bytes, cudaStream_t st);
// 0: tcgen05 kernel (a3_attention_tc.cu); 1: the warp-level mma.sync kernel in this file (cross-check for bring-up)
int g_attn_impl = 0;

int attention_rows(const a3_handle* h, const bf16* q, const int32_t* pos, int M, const bf16* k, const bf16* v,
                   int kv_len, bf16* o, float* lse, void* part, size_t part_bytes, cudaStream_t st) {
  if (M <= 0) return A3_OK;
  if (g_attn_impl == 0) return attention_rows_tc(h, q, pos, M, k, v, kv_len, o, lse, part, part_bytes, st);
  const int Hq = h->m.n_q_heads, Hkv = h->m.n_kv_heads, D = h->m.head_dim;
  const int G = Hq / Hkv;
  dim3 grid(cdiv((long long)M * G, AT_BM), Hkv);
  const float scale_log2 = LOG2E / sqrtf((float)D);
  const int smem = 5 * 64 * D * 2;
  static bool attr_set = false;
  if (!attr_set) {
    A3_CUDA(cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 5 * 64 * 128 * 2));
    A3_CUDA(cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 5 * 64 * 64 * 2));
    attr_set = true;
  }
  ProfScope prof(h, A3_K_ATTENTION, st);
  if (D == 128) attention_kernel<128><<<grid, AT_THREADS, smem, st>>>(q, pos, M, k, v, kv_len, o, lse, Hq, Hkv, scale_log2);
  else attention_kernel<64><<<grid, AT_THREADS, smem, st>>>(q, pos, M, k, v, kv_len, o, lse, Hq, Hkv, scale_log2);
  A3_LAUNCHED();
  return A3_OK;
}

// ------------------------------------------------------------------ relevance scores (Eq. 3)
// One CTA per tile of 64 cache slots.  It loops over the KV heads and, per head, over blocks of 64 packed
// question rows; column sums stay on chip and are added in a fixed order.
template <int D>
__global__ void __launch_bounds__(AT_THREADS)
scores_kernel(const bf16* __restrict__ q, const int32_t* __restrict__ q_pos, int nq, const bf16* __restrict__ k,
              int kv_len, int cand_begin, int cand_end, const float* __restrict__ lse, float* __restrict__ scores,
              int Hq, int Hkv, float scale_log2) {
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

  for (int g = 0; g < Hkv; ++g) {
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
      if (tid < AT_BN) total += (colpart[0][tid] + colpart[1][tid]) + (colpart[2][tid] + colpart[3][tid]);
    }
  }
  if (tid < AT_BN) {
    int key = key0 + tid;
    if (key < kv_len) scores[key] = (key >= cand_begin && key < cand_end) ? total : 0.f;
  }
}

int scores_pass(const a3_handle* h, const bf16* q, const int32_t* q_pos, int nq, const bf16* k, int kv_len,
                int cand_begin, int cand_end, const float* lse, float* scores, cudaStream_t st) {
  if (kv_len <= 0) return A3_OK;
  const int Hq = h->m.n_q_heads, Hkv = h->m.n_kv_heads, D = h->m.head_dim;
  const float scale_log2 = LOG2E / sqrtf((float)D);
  dim3 grid(cdiv(kv_len, AT_BN));
  ProfScope prof(h, A3_K_SCORES, st);
  if (D == 128) scores_kernel<128><<<grid, AT_THREADS, 0, st>>>(q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, Hq, Hkv, scale_log2);
  else scores_kernel<64><<<grid, AT_THREADS, 0, st>>>(q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, Hq, Hkv, scale_log2);
  A3_LAUNCHED();
  return A3_OK;
}

}  // namespace a3

extern "C" void a3_internal_set_attn_impl(int impl) { a3::g_attn_impl = impl; }

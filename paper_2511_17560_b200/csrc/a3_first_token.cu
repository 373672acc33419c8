// First token after fusion: final RMSNorm of one hidden row, vocabulary projection, greedy choice.
// (The quantity behind the paper's time-to-first-token figures; Inference paragraph of the Experiments.)
//
// The projection is a matrix-vector product over a [vocab][d] bf16 matrix read exactly once (1 GiB at
// Llama-3-8B size): bound by HBM.  Every CTA normalises the row itself (8 KiB, from L2) into shared memory as
// fp32 holding the bf16-rounded values a bf16 pipeline would store; a warp then walks four vocabulary rows at a
// time with sixteen 16-byte streaming loads in flight per lane, reduces with shuffles, writes the fp32 logits and keeps
// its best (value, lowest id).  The last CTA to finish (ticket counter) reduces the per-CTA candidates, so the
// whole step is one launch and its result does not depend on the order in which CTAs finish.
#include "a3_internal.cuh"

namespace a3 {

constexpr int FT_THREADS = 256;
constexpr int FT_WARPS = FT_THREADS / 32;

struct FtBest {
  float v;
  int i;
};
// total order: larger value first, then lower id; NaN never wins
__device__ __forceinline__ bool ft_better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

__global__ void __launch_bounds__(FT_THREADS, 2)
first_token_kernel(const bf16* __restrict__ x, const bf16* __restrict__ gain, const uint4* __restrict__ w, int d, int vocab,
                   float eps, float* __restrict__ logits, int32_t* __restrict__ token, FtBest* __restrict__ cand,
                   unsigned int* __restrict__ ticket, uint32_t* status) {
  extern __shared__ float sa[];  // [d] normalised row
  __shared__ float red[FT_WARPS];
  __shared__ FtBest sbest[FT_WARPS];
  __shared__ bool last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // final RMSNorm (fp32 statistics, result rounded to bf16 as a stored activation would be)
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += FT_THREADS) {
    const float v = __bfloat162float(x[i]);
    sa[i] = v;
    ss += v * v;
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (lane == 0) red[warp] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < FT_WARPS; ++i) tot += red[i];
  const float rstd = rsqrtf(tot / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += FT_THREADS)
    sa[i] = __bfloat162float(__float2bfloat16(sa[i] * rstd * __bfloat162float(gain[i])));
  __syncthreads();

  const int nchunk = d / 8;  // 16-byte chunks per vocabulary row
  const float4* sa4 = reinterpret_cast<const float4*>(sa);
  float best_v = -INFINITY;
  int best_i = 0x7fffffff;
  bool bad = false;
  constexpr int R = 4;  // vocabulary rows a warp walks together: 4 x 4 loads of 16 bytes in flight per lane
  const int n_groups = (vocab + R - 1) / R;
  for (int gr = blockIdx.x * FT_WARPS + warp; gr < n_groups; gr += gridDim.x * FT_WARPS) {
    const int r0 = R * gr;
    const uint4* wr[R];
    float acc[R];
#pragma unroll
    for (int j = 0; j < R; ++j) {
      wr[j] = w + (size_t)min(r0 + j, vocab - 1) * nchunk;  // rows beyond the last repeat it; their results are dropped
      acc[j] = 0.f;
    }
    for (int c0 = lane; c0 < nchunk; c0 += 128) {
      uint4 pk[R][4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + 32 * u;
#pragma unroll
        for (int j = 0; j < R; ++j) pk[j][u] = c < nchunk ? __ldcs(wr[j] + c) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + 32 * u;
        if (c < nchunk) {
          const float4 a0 = sa4[2 * c], a1 = sa4[2 * c + 1];
#pragma unroll
          for (int j = 0; j < R; ++j) {
            float f[8];
            unpack8(pk[j][u], f);
            acc[j] += f[0] * a0.x + f[1] * a0.y + f[2] * a0.z + f[3] * a0.w + f[4] * a1.x + f[5] * a1.y + f[6] * a1.z + f[7] * a1.w;
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
#pragma unroll
      for (int j = 0; j < R; ++j) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
    }
    if (lane == 0) {
#pragma unroll
      for (int j = 0; j < R; ++j) {
        const int rj = r0 + j;
        if (rj < vocab) {
          if (logits) logits[rj] = acc[j];
          bad = bad || !isfinite(acc[j]);
          if (ft_better(acc[j], rj, best_v, best_i)) best_v = acc[j], best_i = rj;
        }
      }
    }
  }
  if (lane == 0) {
    sbest[warp] = FtBest{best_v, best_i};
    if (bad) atomicOr(status, A3_DEV_NONFINITE_SCORE);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    FtBest b = sbest[0];
    for (int i = 1; i < FT_WARPS; ++i)
      if (ft_better(sbest[i].v, sbest[i].i, b.v, b.i)) b = sbest[i];
    cand[blockIdx.x] = b;
    __threadfence();
    last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!last) return;
  // the last CTA: every candidate is visible (each writer fenced before taking its ticket)
  __threadfence();
  FtBest b{-INFINITY, 0x7fffffff};
  const volatile FtBest* vc = cand;
  for (int i = threadIdx.x; i < (int)gridDim.x; i += FT_THREADS) {
    const float cv = vc[i].v;
    const int ci = vc[i].i;
    if (ft_better(cv, ci, b.v, b.i)) b.v = cv, b.i = ci;
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, b.v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, b.i, o);
    if (ft_better(ov, oi, b.v, b.i)) b.v = ov, b.i = oi;
  }
  if (lane == 0) sbest[warp] = b;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < FT_WARPS; ++i)
      if (ft_better(sbest[i].v, sbest[i].i, b.v, b.i)) b = sbest[i];
    *token = b.i == 0x7fffffff ? 0 : b.i;  // every logit NaN: token 0, flagged above
    *ticket = 0;                           // ready for the next call
  }
}

}  // namespace a3

using namespace a3;

extern "C" size_t a3_first_token_workspace_bytes(const a3_handle* h) {
  if (!h) return 0;
  return 256 + sizeof(FtBest) * (size_t)h->sm_count * 2;
}

extern "C" int a3_first_token(const a3_handle* h, const void* x_row, const void* final_norm, const void* lm_head, int vocab,
                              float* logits_out, int32_t* token_out, void* ws, size_t ws_bytes, a3_stream stream) {
  if (!h || !x_row || !final_norm || !lm_head || !token_out || !ws) return A3_EINVAL;
  const int d = h->m.d_model;
  if (vocab <= 0 || d % 8 != 0) return A3_EINVAL;
  if (((uintptr_t)lm_head & 15) || ((uintptr_t)ws & 255)) return A3_EINVAL;
  if (ws_bytes < a3_first_token_workspace_bytes(h)) return A3_EWORKSPACE;
  if ((size_t)d * 4 > 96 * 1024) return A3_EUNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned int* ticket = (unsigned int*)ws;
  FtBest* cand = (FtBest*)((char*)ws + 256);
  // The ticket must be zero when the kernel starts; the kernel leaves it at zero, but the workspace is the
  // caller's and may have been used for something else in between.
  A3_CUDA(cudaMemsetAsync(ticket, 0, 4, st));
  const size_t smem = (size_t)d * 4;
  if (smem > 48 * 1024) A3_CUDA(cudaFuncSetAttribute(first_token_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
  int grid = h->sm_count * 2;
  const int need = cdiv((vocab + 3) / 4, FT_WARPS);
  if (grid > need) grid = need;
  {
    ProfScope prof(h, A3_K_FIRST_TOKEN, st);
    first_token_kernel<<<grid, FT_THREADS, smem, st>>>((const bf16*)x_row, (const bf16*)final_norm, (const uint4*)lm_head, d, vocab,
                                                       h->m.rms_eps, logits_out, token_out, cand, ticket, h->dev_status);
  }
  return launched();
}

// Selection Re = top_p(s) (Eq. 3): block-radix select on the order-preserving integer image of the fp32 scores.
// One CTA per score array.  Four 8-bit histogram passes find the key of the k-th largest score; one ordered
// pass then emits every slot above that key plus, in slot order, as many slots equal to it as are still needed.
// The result is exact: ties go to the lower slot and the output is ascending.
#include "a3_internal.cuh"

namespace a3 {

constexpr int TK_THREADS = 1024;

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // larger float <=> larger key
}

__global__ void __launch_bounds__(TK_THREADS)
topk_select_kernel(const float* __restrict__ scores, int cand_begin, int n, int k, int32_t* __restrict__ idx_out, uint32_t* status,
                   size_t score_stride, size_t idx_stride) {
  // one CTA per independent selection (the per-head selections of the eviction step; a single one for Eq. 3)
  scores += blockIdx.x * score_stride;
  idx_out += blockIdx.x * idx_stride;
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_prefix, s_remaining;
  __shared__ unsigned int warp_gt[TK_THREADS / 32], warp_eq[TK_THREADS / 32];
  __shared__ unsigned int run_gt, run_eq;
  const float* s = scores + cand_begin;
  const int tid = threadIdx.x;

  // ---- radix select: after the loop `prefix` is the key of the k-th largest element
  uint32_t prefix = 0, mask = 0;
  unsigned int remaining = (unsigned int)k;  // rank (1-based, from the top) inside the current bucket
  bool nonfinite = false;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += TK_THREADS) {
      float v = s[i];
      if (shift == 24 && !(fabsf(v) <= 3.0e38f)) nonfinite = true;
      uint32_t key = score_key(v);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned int acc = 0;
      int d = 255;
      for (; d > 0; --d) {
        if (acc + hist[d] >= remaining) break;
        acc += hist[d];
      }
      s_prefix = prefix | ((uint32_t)d << shift);
      s_remaining = remaining - acc;
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= 255u << shift;
    __syncthreads();
  }
  if (nonfinite) atomicOr(status, A3_DEV_NONFINITE_SCORE);
  // `remaining` = how many elements equal to the threshold key are taken (lowest slots first)
  const uint32_t thr = prefix;
  const unsigned int need_eq = remaining;
  if (tid == 0) {
    run_gt = 0;
    run_eq = 0;
  }
  __syncthreads();

  // ---- ordered emission, 1024 slots per trip
  const int lane = tid & 31, warp = tid >> 5;
  for (int base = 0; base < n; base += TK_THREADS) {
    const int i = base + tid;
    uint32_t key = 0;
    bool gt = false, eq = false;
    if (i < n) {
      key = score_key(s[i]);
      gt = key > thr;
      eq = key == thr;
    }
    const unsigned int bgt = __ballot_sync(0xffffffffu, gt), beq = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) {
      warp_gt[warp] = __popc(bgt);
      warp_eq[warp] = __popc(beq);
    }
    __syncthreads();
    unsigned int pre_gt = run_gt, pre_eq = run_eq;
    for (int w = 0; w < warp; ++w) {
      pre_gt += warp_gt[w];
      pre_eq += warp_eq[w];
    }
    const unsigned int lt_mask = (1u << lane) - 1u;
    const unsigned int my_gt = pre_gt + __popc(bgt & lt_mask);  // greater-than elements before me
    const unsigned int my_eq = pre_eq + __popc(beq & lt_mask);  // equal elements before me
    if (gt || (eq && my_eq < need_eq)) {
      const unsigned int eq_taken_before = my_eq < need_eq ? my_eq : need_eq;
      const unsigned int o = my_gt + eq_taken_before;
      if (o < (unsigned int)k) idx_out[o] = cand_begin + i;
    }
    __syncthreads();
    if (tid == TK_THREADS - 1) {
      run_gt = my_gt + (gt ? 1u : 0u);
      run_eq = my_eq + (eq ? 1u : 0u);
    }
    __syncthreads();
  }
}

}  // namespace a3

using namespace a3;

extern "C" int a3_topk_select(const a3_handle* h, const float* scores, int cand_begin, int cand_end, int k,
                              int32_t* idx_out, a3_stream stream) {
  if (!h || cand_begin < 0 || cand_end < cand_begin || k < 0) return A3_EINVAL;
  const int n = cand_end - cand_begin;
  if (k > n) k = n;
  if (k == 0) return A3_OK;
  if (!scores || !idx_out) return A3_EINVAL;
  ProfScope prof(h, A3_K_TOPK, (cudaStream_t)stream);
  topk_select_kernel<<<1, TK_THREADS, 0, (cudaStream_t)stream>>>(scores, cand_begin, n, k, idx_out, h->dev_status, 0, 0);
  A3_LAUNCHED();
  return A3_OK;
}

int a3::topk_batched(const a3_handle* h, const float* scores, size_t score_stride, int batches, int cand_begin, int cand_end,
                     int k, int32_t* idx_out, size_t idx_stride, cudaStream_t st) {
  const int n = cand_end - cand_begin;
  if (k > n) k = n;
  if (k <= 0 || batches <= 0) return A3_OK;
  ProfScope prof(h, A3_K_TOPK, st);
  topk_select_kernel<<<batches, TK_THREADS, 0, st>>>(scores, cand_begin, n, k, idx_out, h->dev_status, score_stride, idx_stride);
  A3_LAUNCHED();
  return A3_OK;
}

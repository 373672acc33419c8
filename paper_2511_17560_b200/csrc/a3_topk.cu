// Selection Re = top_p(s) (Eq. 3): block-radix select on the order-preserving integer image of the fp32 scores.
// One CTA per score array.  The scores are read from global memory once, as integer keys into shared memory (up to
// TK_SMEM_KEYS of them; longer arrays are re-read from global memory in every pass).  Four 8-bit histogram passes
// find the key of the k-th largest score: the warps count into TK_HISTS private histograms (a warp whose lanes all
// hold the same digit - the rule in the first pass, since the scores of one request share their leading bits - adds
// 32 with one instruction instead of serialising 32 atomics on one bin), the histograms are summed, and the bin of
// the k-th element is found by a parallel suffix sum over the 256 bins.  The emission is
// ordered: every warp owns a contiguous span of the slots, counts what it will emit, and after one exchange of the
// 32 warp totals writes every slot above the threshold key plus, in slot order, as many slots equal to it as are
// still needed.  The result is exact: ties go to the lower slot and the output is ascending.
#include "a3_internal.cuh"

namespace a3 {

constexpr int TK_THREADS = 1024;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int TK_HISTS = 16;              // private histograms (warp w counts into number w % TK_HISTS)
constexpr int TK_SMEM_KEYS = 48 * 1024;  // 192 KiB of keys

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // larger float <=> larger key
}

template <bool IN_SMEM>
__device__ __forceinline__ void topk_body(const float* __restrict__ s, uint32_t* __restrict__ keys, int cand_begin, int n, int k,
                                          int32_t* __restrict__ idx_out, uint32_t* status) {
  __shared__ unsigned int hist[256];
  __shared__ unsigned int whist[TK_HISTS][256];
  __shared__ unsigned int warp_tot[8];
  __shared__ unsigned int s_prefix, s_remaining;
  __shared__ unsigned int warp_gt[TK_WARPS], warp_eq[TK_WARPS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  auto key_at = [&](int i) -> uint32_t { return IN_SMEM ? keys[i] : score_key(s[i]); };

  // ---- load: scores -> keys (shared memory), non-finite scores flagged
  bool nonfinite = false;
#pragma unroll 4
  for (int i = tid; i < n; i += TK_THREADS) {
    const float v = s[i];
    if (!(fabsf(v) <= 3.0e38f)) nonfinite = true;
    if (IN_SMEM) keys[i] = score_key(v);
  }
  if (nonfinite) atomicOr(status, A3_DEV_NONFINITE_SCORE);

  // ---- radix select: after the loop `prefix` is the key of the k-th largest element
  uint32_t prefix = 0, mask = 0;
  unsigned int remaining = (unsigned int)k;  // rank (1-based, from the top) inside the current bucket
  const int n_round = (n + 31) & ~31;        // whole warps walk the array, so that the lanes can vote together
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < TK_HISTS * 256; i += TK_THREADS) (&whist[0][0])[i] = 0;
    __syncthreads();
    unsigned int* mine = whist[warp % TK_HISTS];
    for (int i = tid; i < n_round; i += TK_THREADS) {
      uint32_t digit = 0xFFFFFFFFu;  // lanes with nothing to count
      if (i < n) {
        const uint32_t key = key_at(i);
        if ((key & mask) == prefix) digit = (key >> shift) & 255u;
      }
      const uint32_t first = __shfl_sync(0xffffffffu, digit, 0);
      if (__all_sync(0xffffffffu, digit == first)) {
        if (lane == 0 && digit != 0xFFFFFFFFu) atomicAdd(&mine[digit], 32u);
      } else if (digit != 0xFFFFFFFFu) {
        atomicAdd(&mine[digit], 1u);
      }
    }
    __syncthreads();
    if (tid < 256) {
      unsigned int v = 0;
#pragma unroll
      for (int w = 0; w < TK_HISTS; ++w) v += whist[w][tid];
      hist[tid] = v;
    }
    __syncthreads();
    // suffix sums over the bins: S[d] = count of elements with digit >= d; the k-th element's digit is the largest d
    // with S[d] >= remaining
    if (tid < 256) {
      unsigned int v = hist[tid];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int t = __shfl_down_sync(0xffffffffu, v, o);
        if (lane + o < 32) v += t;
      }
      if (lane == 0) warp_tot[warp] = v;
      __syncwarp();
      hist[tid] = v;  // suffix sum within this warp's 32 bins
    }
    __syncthreads();
    if (tid < 256) {
      unsigned int above = 0;  // elements in the bins of higher warps
      for (int w = warp + 1; w < 8; ++w) above += warp_tot[w];
      const unsigned int S_d = hist[tid] + above;
      const unsigned int S_next = lane == 31 ? above : hist[tid + 1] + above;  // S[d + 1]
      if (S_d >= remaining && S_next < remaining) {
        s_prefix = prefix | ((uint32_t)tid << shift);
        s_remaining = remaining - S_next;
      }
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= 255u << shift;
  }
  // `remaining` = how many elements equal to the threshold key are taken (lowest slots first)
  const uint32_t thr = prefix;
  const unsigned int need_eq = remaining;

  // ---- ordered emission: warp w owns slots [w * span, (w + 1) * span)
  const int span = ((n + TK_WARPS - 1) / TK_WARPS + 31) & ~31;
  const int b0 = warp * span, b1 = min(n, b0 + span);
  unsigned int cnt_gt = 0, cnt_eq = 0;
  for (int base = b0; base < b1; base += 32) {
    const int i = base + lane;
    const uint32_t key = i < b1 ? key_at(i) : 0u;
    cnt_gt += __popc(__ballot_sync(0xffffffffu, i < b1 && key > thr));
    cnt_eq += __popc(__ballot_sync(0xffffffffu, i < b1 && key == thr));
  }
  if (lane == 0) {
    warp_gt[warp] = cnt_gt;
    warp_eq[warp] = cnt_eq;
  }
  __syncthreads();
  unsigned int run_gt = 0, run_eq = 0;
  for (int w = 0; w < warp; ++w) {
    run_gt += warp_gt[w];
    run_eq += warp_eq[w];
  }
  const unsigned int lt_mask = (1u << lane) - 1u;
  for (int base = b0; base < b1; base += 32) {
    const int i = base + lane;
    const uint32_t key = i < b1 ? key_at(i) : 0u;
    const bool gt = i < b1 && key > thr, eq = i < b1 && key == thr;
    const unsigned int bgt = __ballot_sync(0xffffffffu, gt), beq = __ballot_sync(0xffffffffu, eq);
    const unsigned int my_gt = run_gt + __popc(bgt & lt_mask);  // greater-than elements before me
    const unsigned int my_eq = run_eq + __popc(beq & lt_mask);  // equal elements before me
    if (gt || (eq && my_eq < need_eq)) {
      const unsigned int o = my_gt + (my_eq < need_eq ? my_eq : need_eq);
      if (o < (unsigned int)k) idx_out[o] = cand_begin + i;
    }
    run_gt += __popc(bgt);
    run_eq += __popc(beq);
  }
}

__global__ void __launch_bounds__(TK_THREADS)
topk_select_kernel(const float* __restrict__ scores, int cand_begin, int n, int k, int32_t* __restrict__ idx_out, uint32_t* status,
                   size_t score_stride, size_t idx_stride, int in_smem) {
  extern __shared__ uint32_t tk_keys[];
  pdl_wait();
  pdl_launch_dependents();
  // one CTA per independent selection (the per-head selections of the eviction step; a single one for Eq. 3)
  const float* s = scores + blockIdx.x * score_stride + cand_begin;
  int32_t* out = idx_out + blockIdx.x * idx_stride;
  if (in_smem) topk_body<true>(s, tk_keys, cand_begin, n, k, out, status);
  else topk_body<false>(s, tk_keys, cand_begin, n, k, out, status);
}

static int launch_topk(const a3_handle* h, const float* scores, size_t score_stride, int batches, int cand_begin, int n, int k,
                       int32_t* idx_out, size_t idx_stride, cudaStream_t st) {
  const int in_smem = n <= TK_SMEM_KEYS ? 1 : 0;
  const size_t smem = in_smem ? (size_t)n * 4 : 0;
  static SmemAttrOnce attr;
  A3_TRY(smem_attr_once(attr, h->device, topk_select_kernel, TK_SMEM_KEYS * 4));
  ProfScope prof(h, A3_K_TOPK, st);
  A3_CUDA(launch_pdl(topk_select_kernel, dim3(batches), dim3(TK_THREADS), smem, st, scores, cand_begin, n, k, idx_out, h->dev_status,
                     score_stride, idx_stride, in_smem));
  A3_LAUNCHED();
  return A3_OK;
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
  return launch_topk(h, scores, 0, 1, cand_begin, n, k, idx_out, 0, (cudaStream_t)stream);
}

int a3::topk_batched(const a3_handle* h, const float* scores, size_t score_stride, int batches, int cand_begin, int cand_end,
                     int k, int32_t* idx_out, size_t idx_stride, cudaStream_t st) {
  const int n = cand_end - cand_begin;
  if (k > n) k = n;
  if (k <= 0 || batches <= 0) return A3_OK;
  return launch_topk(h, scores, score_stride, batches, cand_begin, n, k, idx_out, idx_stride, st);
}

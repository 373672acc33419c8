// `ex`: eviction after fusion (Extension subsection).  The system prompt S and the question Q are kept whole;
// per layer and per KV head the C - |S| - |Q| document tokens with the most question-window attention are kept
// (SnapKV's strategy) and the layer's cache is compacted.
//
// One layer = four launches: per-head votes (the score kernel of Eq. 3 without the sum over KV heads, fed with
// the question rows' queries and log-sum-exps of that layer), optional max pooling, one top-k CTA per KV head,
// and a gather that writes the compact cache [C'][Hkv][D] (bound by HBM: each kept row is read and written once).
#include "a3_internal.cuh"

namespace a3 {

// running maximum over `width` candidates centred on each candidate, cut at the candidate range
__global__ void __launch_bounds__(256)
pool_scores_kernel(const float* __restrict__ in, float* __restrict__ out, int kv_len, int cand_begin, int cand_end, int half_width) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= kv_len) return;
  const float* row = in + (size_t)blockIdx.y * kv_len;
  float v = 0.f;
  if (i >= cand_begin && i < cand_end) {
    const int lo = max(cand_begin, i - half_width), hi = min(cand_end - 1, i + half_width);
    v = row[lo];
    for (int j = lo + 1; j <= hi; ++j) v = fmaxf(v, row[j]);
  }
  out[(size_t)blockIdx.y * kv_len + i] = v;
}

// kept slot c of head g: S, then the selected documents (ascending), then Q
__device__ __forceinline__ int evict_source(int c, int g, const int32_t* __restrict__ sel, int k, int n_system, int n_ctx) {
  if (c < n_system) return c;
  if (c < n_system + k) return sel[(size_t)g * k + (c - n_system)];
  return n_ctx + (c - n_system - k);
}

// grid: kept slots; a CTA moves the K and V rows of all heads of one compact slot (Hkv * D * 2 bytes each)
__global__ void __launch_bounds__(128)
evict_gather_kernel(const uint4* __restrict__ kc, const uint4* __restrict__ vc, int kv_len, const int32_t* __restrict__ sel, int k,
                    int n_system, int n_ctx, int Hkv, int head_vecs, uint4* __restrict__ k_out, uint4* __restrict__ v_out,
                    int32_t* __restrict__ kept, int C, uint32_t* status) {
  const int c = blockIdx.x;
  const int row_vecs = Hkv * head_vecs;
  for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
    const int g = v / head_vecs;
    const int src = evict_source(c, g, sel, k, n_system, n_ctx);
    if (src < 0 || src >= kv_len) {
      if (v % head_vecs == 0) atomicOr(status, A3_DEV_BAD_POSITION);
      continue;
    }
    k_out[(size_t)c * row_vecs + v] = __ldcs(kc + (size_t)src * row_vecs + v);
    v_out[(size_t)c * row_vecs + v] = __ldcs(vc + (size_t)src * row_vecs + v);
    if (kept && v % head_vecs == 0) kept[(size_t)g * C + c] = src;
  }
}

}  // namespace a3

using namespace a3;

extern "C" int a3_evict_count(int capacity, int n_system, int n_ctx, int n_question) {
  int k = capacity - n_system - n_question;
  if (k > n_ctx - n_system) k = n_ctx - n_system;
  return k < 0 ? 0 : k;
}

extern "C" size_t a3_evict_workspace_bytes(const a3_handle* h, int kv_len) {
  if (!h || kv_len < 0) return 0;
  const size_t per = align_up((size_t)h->m.n_kv_heads * kv_len * 4, 256);
  return 3 * per;  // votes, pooled votes, selected slots
}

extern "C" int a3_evict_layer(const a3_handle* h, const void* q_window, const int32_t* q_pos, int nq, const float* lse,
                              const void* k_layer, const void* v_layer, int kv_len, int n_system, int n_ctx, int capacity,
                              int pool, void* k_out, void* v_out, int32_t* kept_out, void* ws, size_t ws_bytes,
                              a3_stream stream) {
  if (!h || nq < 0 || kv_len < 0 || n_system < 0 || n_ctx < n_system || n_ctx + nq != kv_len) return A3_EINVAL;
  if (pool < 1 || pool % 2 == 0 || capacity < 0) return A3_EINVAL;
  if (kv_len == 0) return A3_OK;
  if (!k_layer || !v_layer || !k_out || !v_out || !ws) return A3_EINVAL;
  if (nq > 0 && (!q_window || !q_pos || !lse)) return A3_EINVAL;
  if (((uintptr_t)k_layer | (uintptr_t)v_layer | (uintptr_t)k_out | (uintptr_t)v_out | (uintptr_t)ws) & 15) return A3_EINVAL;
  if (ws_bytes < a3_evict_workspace_bytes(h, kv_len)) return A3_EWORKSPACE;
  const a3_model_desc& m = h->m;
  cudaStream_t st = (cudaStream_t)stream;
  const int k = a3_evict_count(capacity, n_system, n_ctx, nq);
  const int C = n_system + k + nq;
  const size_t per = align_up((size_t)m.n_kv_heads * kv_len * 4, 256);
  float* votes = (float*)ws;
  float* pooled = (float*)((char*)ws + per);
  int32_t* sel = (int32_t*)((char*)ws + 2 * per);
  if (k > 0 && k < n_ctx - n_system) {
    if (nq > 0) A3_TRY(scores_pass(h, (const bf16*)q_window, q_pos, nq, (const bf16*)k_layer, kv_len, n_system, n_ctx, lse, nullptr, st, votes));
    else A3_CUDA(cudaMemsetAsync(votes, 0, (size_t)m.n_kv_heads * kv_len * 4, st));
    const float* src = votes;
    if (pool > 1) {
      ProfScope prof(h, A3_K_ROWS, st);
      pool_scores_kernel<<<dim3(cdiv(kv_len, 256), m.n_kv_heads), 256, 0, st>>>(votes, pooled, kv_len, n_system, n_ctx, pool / 2);
      A3_LAUNCHED();
      src = pooled;
    }
    A3_TRY(topk_batched(h, src, (size_t)kv_len, m.n_kv_heads, n_system, n_ctx, k, sel, (size_t)k, st));
  } else if (k > 0) {
    // everything fits: the selection is every document slot (no votes needed)
    for (int g = 0; g < m.n_kv_heads; ++g) A3_TRY(iota_rows(h, sel + (size_t)g * k, n_system, k, st));
  }
  if (C == 0) return A3_OK;
  {
    ProfScope prof(h, A3_K_ROWS, st);
    evict_gather_kernel<<<C, 128, 0, st>>>((const uint4*)k_layer, (const uint4*)v_layer, kv_len, sel, k, n_system, n_ctx, m.n_kv_heads,
                                           m.head_dim / 8, (uint4*)k_out, (uint4*)v_out, kept_out, C, h->dev_status);
    A3_LAUNCHED();
  }
  return A3_OK;
}

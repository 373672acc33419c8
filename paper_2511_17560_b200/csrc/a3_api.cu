// Handle lifetime, workspace carving and the orchestration of the fusion request (host code only).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "a3_internal.cuh"

namespace a3 {
int build_rope_table(float2* tab, int max_pos, int D, double base, cudaStream_t st);

// Workspace of one a3_recompute_layer call, carved from a caller-provided buffer.
struct LayerWs {
  bf16 *a, *q, *o, *hmid;
  float* lse;
  void* attn_part;
  size_t attn_part_bytes;
  size_t bytes;
};
static LayerWs carve_layer_ws(const a3_handle* h, int rows, void* base) {
  const a3_model_desc& m = h->m;
  LayerWs w;
  char* p = (char*)base;
  size_t off = 0;
  auto take = [&](size_t b) {
    char* r = p ? p + off : nullptr;
    off += align_up(b, 256);
    return r;
  };
  const size_t R = (size_t)(rows > 0 ? rows : 1);
  w.a = (bf16*)take(R * m.d_model * 2);
  w.q = (bf16*)take(R * m.n_q_heads * m.head_dim * 2);
  w.o = (bf16*)take(R * m.n_q_heads * m.head_dim * 2);
  w.hmid = (bf16*)take(R * m.d_ff * 2);
  w.lse = (float*)take(R * m.n_q_heads * 4);
  w.attn_part_bytes = attention_part_bytes(h);
  w.attn_part = take(w.attn_part_bytes);
  w.bytes = off;
  return w;
}

struct RequestWs {
  bf16* x_all;
  int32_t* all_pos;
  float* lse_q;
  void* evict;  // scratch of a3_evict_layer
  size_t evict_bytes;
  void* layer;
  size_t bytes;
};
static RequestWs carve_request_ws(const a3_handle* h, int n, void* base) {
  const a3_model_desc& m = h->m;
  RequestWs w;
  char* p = (char*)base;
  size_t off = 0;
  auto take = [&](size_t b) {
    char* r = p ? p + off : nullptr;
    off += align_up(b, 256);
    return r;
  };
  const size_t N = (size_t)(n > 0 ? n : 1);
  w.x_all = (bf16*)take(N * m.d_model * 2);
  w.all_pos = (int32_t*)take(N * 4);
  w.lse_q = (float*)take(N * m.n_q_heads * 4);
  w.evict_bytes = a3_evict_workspace_bytes(h, n);
  w.evict = take(w.evict_bytes);
  w.layer = take(carve_layer_ws(h, n, nullptr).bytes);
  w.bytes = off;
  return w;
}
}  // namespace a3

using namespace a3;

extern "C" const char* a3_status_string(int s) {
  switch (s) {
    case A3_OK: return "ok";
    case A3_EINVAL: return "invalid argument";
    case A3_EUNSUPPORTED: return "unsupported shape";
    case A3_EWORKSPACE: return "workspace too small";
    case A3_ECUDA: return "CUDA call failed";
    case A3_EDEVICE: return "device status word set";
    case A3_ETOOLARGE: return "size exceeds a fixed built-in limit";
    default: return "unknown status";
  }
}

extern "C" int a3_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" uint64_t a3_launch_count(int reset) {
  uint64_t v = g_launches;
  if (reset) g_launches = 0;
  return v;
}

extern "C" int a3_chunk_edge_rows(const int32_t* chunk_len, int n_chunks, int m, int n_system, int32_t* rows_out, int capacity) {
  if (!chunk_len || n_chunks <= 0 || m <= 0) return 0;
  int count = 0, o = 0;
  for (int c = 0; c < n_chunks; ++c) {
    const int t = chunk_len[c] > 0 ? chunk_len[c] : 0;
    for (int i = 0; i < t; ++i) {
      if ((i < m || i >= t - m) && o + i >= n_system) {
        if (rows_out && count < capacity) rows_out[count] = o + i;
        ++count;
      }
      if (i == m - 1 && t - m > m) i = t - m - 1;  // jump over the middle of a long chunk
    }
    o += t;
  }
  return count;
}

extern "C" int a3_random_rows(uint64_t seed, int cand_begin, int cand_end, int k, int32_t* rows_out, int capacity) {
  if (cand_begin < 0 || cand_end <= cand_begin || k <= 0) return 0;
  const int n = cand_end - cand_begin;
  if (k > n) k = n;
  int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
  if (!idx) return 0;
  for (int i = 0; i < n; ++i) idx[i] = i;
  for (int i = 0; i < k; ++i) {
    uint64_t z = seed + (uint64_t)i + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    const int j = i + (int)(z % (uint64_t)(n - i));
    const int32_t t = idx[i];
    idx[i] = idx[j];
    idx[j] = t;
  }
  // ascending order of the k chosen slots (insertion into a bitmap would do as well; k log k is nothing here)
  qsort(idx, (size_t)k, sizeof(int32_t), [](const void* a, const void* b) { return (*(const int32_t*)a > *(const int32_t*)b) - (*(const int32_t*)a < *(const int32_t*)b); });
  if (rows_out)
    for (int i = 0; i < k && i < capacity; ++i) rows_out[i] = cand_begin + idx[i];
  free(idx);
  return k;
}

extern "C" int a3_recompute_count(double ratio, int n, int n_candidates) {
  if (n_candidates <= 0 || n <= 0 || !(ratio > 0.0)) return 0;
  double p = floor(ratio * (double)n + 1e-9);
  if (p > (double)n_candidates) return n_candidates;
  return (int)p;
}

extern "C" int a3_create(a3_handle** out, const a3_model_desc* m, const a3_layer_weights* layers) {
  if (!out || !m || !layers) return A3_EINVAL;
  *out = nullptr;
  if (m->n_layers <= 0 || m->d_model <= 0 || m->n_q_heads <= 0 || m->n_kv_heads <= 0 || m->d_ff <= 0 ||
      m->max_positions <= 0 || !(m->rope_theta > 0.0) || !(m->rms_eps >= 0.f))
    return A3_EINVAL;
  if (m->head_dim != 64 && m->head_dim != 128) return A3_EUNSUPPORTED;
  if (m->rope_layout != 0 && m->rope_layout != 1) return A3_EUNSUPPORTED;
  if (m->n_q_heads % m->n_kv_heads) return A3_EUNSUPPORTED;
  if (m->d_model % 128 || (m->n_q_heads * m->head_dim) % 128 || (m->n_kv_heads * m->head_dim) % 128 || m->d_ff % 128)
    return A3_EUNSUPPORTED;
  for (int l = 0; l < m->n_layers; ++l) {
    const a3_layer_weights& w = layers[l];
    const void* req[] = {w.attn_norm, w.wq, w.wk, w.wv, w.wo, w.mlp_norm, w.w_gate, w.w_up, w.w_down};
    for (const void* p : req)
      if (!p || ((uintptr_t)p & 15)) return A3_EINVAL;
    const void* opt[] = {w.bq, w.bk, w.bv};
    for (const void* p : opt)
      if (p && ((uintptr_t)p & 15)) return A3_EINVAL;
  }
  a3_handle* h = (a3_handle*)calloc(1, sizeof(a3_handle));
  if (!h) return A3_EINVAL;
  h->m = *m;
  h->opt[A3_OPT_ATTN_PAIR] = -1;
  h->opt[A3_OPT_SWIGLU_NARROW] = 1;
  h->opt[A3_OPT_SWIGLU_PAIR] = 1;
  h->opt[A3_OPT_RESIDUAL_T] = 1;
  h->opt[A3_OPT_QKV_T] = 1;
  h->opt[A3_OPT_GEMM_BN_SWIGLU] = 256;  // the one-CTA gate/up kernel runs two CTAs per SM: 256 columns, 2 stages
  h->opt[A3_OPT_GEMM_STAGES_SWIGLU] = 2;
  h->layers = (a3_layer_weights*)malloc(sizeof(a3_layer_weights) * m->n_layers);
  memcpy(h->layers, layers, sizeof(a3_layer_weights) * m->n_layers);
  cudaError_t e = cudaGetDevice(&h->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
  if (e == cudaSuccess) e = cudaMalloc((void**)&h->rope_tab, (size_t)m->max_positions * (m->head_dim / 2) * sizeof(float2));
  if (e == cudaSuccess) e = cudaMalloc((void**)&h->dev_status, 256);
  if (e == cudaSuccess) e = cudaMemset(h->dev_status, 0, 256);
  if (e != cudaSuccess) {
    a3_destroy(h);
    return cuda_fail(e);
  }
  int s = build_rope_table(h->rope_tab, m->max_positions, m->head_dim, m->rope_theta, 0);
  if (s == A3_OK) {
    e = cudaStreamSynchronize(0);
    if (e != cudaSuccess) s = cuda_fail(e);
  }
  if (s != A3_OK) {
    a3_destroy(h);
    return s;
  }
  *out = h;
  return A3_OK;
}

extern "C" int a3_set_option(a3_handle* h, int option, int value) {
  if (!h || option < 0 || option >= A3_OPT_COUNT) return A3_EINVAL;
  h->opt[option] = value;
  return A3_OK;
}

extern "C" int a3_profile_enable(a3_handle* h, int max_records) {
  if (!h || max_records < 0) return A3_EINVAL;
  if (h->prof) {
    for (int i = 0; i < 2 * h->prof->capacity; ++i) cudaEventDestroy(h->prof->ev[i]);
    free(h->prof->ev);
    free(h->prof->cls);
    free(h->prof);
    h->prof = nullptr;
  }
  if (max_records == 0) return A3_OK;
  Profiler* p = (Profiler*)calloc(1, sizeof(Profiler));
  p->ev = (cudaEvent_t*)calloc(2 * (size_t)max_records, sizeof(cudaEvent_t));
  p->cls = (int*)calloc(max_records, sizeof(int));
  p->capacity = max_records;
  for (int i = 0; i < 2 * max_records; ++i) {
    cudaError_t e = cudaEventCreate(&p->ev[i]);
    if (e != cudaSuccess) {
      p->capacity = i / 2;
      break;
    }
  }
  h->prof = p;
  return A3_OK;
}

extern "C" int a3_profile_read(a3_handle* h, a3_profile_entry* out, a3_stream stream) {
  if (!h || !out) return A3_EINVAL;
  for (int k = 0; k < A3_K_CLASSES; ++k) out[k] = a3_profile_entry{0, 0.0};
  A3_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  Profiler* p = h->prof;
  if (!p) return A3_OK;
  for (int i = 0; i < p->used; ++i) {
    float ms = 0.f;
    A3_CUDA(cudaEventElapsedTime(&ms, p->ev[2 * i], p->ev[2 * i + 1]));
    out[p->cls[i]].launches += 1;
    out[p->cls[i]].ms += ms;
  }
  p->used = 0;
  return A3_OK;
}

extern "C" const char* a3_kernel_class_name(int cls) {
  static const char* names[A3_K_CLASSES] = {"rerotate", "rmsnorm", "gemm_qkv", "attention", "gemm_residual",
                                            "gemm_swiglu", "scores", "topk", "rows", "first_token"};
  return cls >= 0 && cls < A3_K_CLASSES ? names[cls] : "?";
}

namespace a3 { static void host_pipe_destroy(a3_handle* h); }

extern "C" void a3_destroy(a3_handle* h) {
  if (!h) return;
  a3_profile_enable(h, 0);
  host_pipe_destroy(h);
  if (h->rope_tab) cudaFree(h->rope_tab);
  if (h->dev_status) cudaFree(h->dev_status);
  free(h->layers);
  free(h);
}

extern "C" size_t a3_layer_workspace_bytes(const a3_handle* h, int max_rows) {
  if (!h || max_rows < 0) return 0;
  return carve_layer_ws(h, max_rows, nullptr).bytes;
}

extern "C" size_t a3_request_workspace_bytes(const a3_handle* h, int n) {
  if (!h || n < 0) return 0;
  return carve_request_ws(h, n, nullptr).bytes;
}

extern "C" int a3_device_status(const a3_handle* h, uint32_t* bits_out, a3_stream stream) {
  if (!h || !bits_out) return A3_EINVAL;
  cudaStream_t st = (cudaStream_t)stream;
  A3_CUDA(cudaStreamSynchronize(st));
  uint32_t v = 0;
  A3_CUDA(cudaMemcpy(&v, h->dev_status, 4, cudaMemcpyDeviceToHost));
  if (v) A3_CUDA(cudaMemset(h->dev_status, 0, 4));
  *bits_out = v;
  return A3_OK;
}

// ------------------------------------------------------------------ one layer (Eq. 5)
namespace a3 {
// rows_kv: rows whose k/v are projected and written to the cache (all M); rows_q: q is projected for rows
// [q_first, M) only (the selection layer needs the question rows' queries, not the context rows').
static int qkv_project(const a3_handle* h, int layer, const bf16* a, const int32_t* pos, int M, int q_first, bf16* q_out,
                       bf16* kc, bf16* vc, int kv_len, cudaStream_t st) {
  const a3_model_desc& m = h->m;
  const a3_layer_weights& w = h->layers[layer];
  const int qd = m.n_q_heads * m.head_dim, kvd = m.n_kv_heads * m.head_dim;
  GemmArgs g{};
  g.K = m.d_model;
  g.q_out = q_out;
  g.k_cache = kc;
  g.v_cache = vc;
  g.kv_len = kv_len;
  if (q_first == 0) {
    g.A = a;
    g.M = M;
    g.pos = pos;
    g.nseg = 3;
    g.seg[0] = {(const bf16*)w.wq, (const bf16*)w.bq, qd, 0};
    g.seg[1] = {(const bf16*)w.wk, (const bf16*)w.bk, kvd, 1};
    g.seg[2] = {(const bf16*)w.wv, (const bf16*)w.bv, kvd, 2};
    return gemm_bf16(h, EPI_QKV, g, st);
  }
  g.A = a;
  g.M = M;
  g.pos = pos;
  g.nseg = 2;
  g.seg[0] = {(const bf16*)w.wk, (const bf16*)w.bk, kvd, 1};
  g.seg[1] = {(const bf16*)w.wv, (const bf16*)w.bv, kvd, 2};
  A3_TRY(gemm_bf16(h, EPI_QKV, g, st));
  if (q_first < M) {
    g.A = a + (size_t)q_first * m.d_model;
    g.M = M - q_first;
    g.pos = pos + q_first;
    g.nseg = 1;
    g.seg[0] = {(const bf16*)w.wq, (const bf16*)w.bq, qd, 0};
    A3_TRY(gemm_bf16(h, EPI_QKV, g, st));
  }
  return A3_OK;
}

static int recompute_layer_impl(const a3_handle* h, int layer, bf16* x, const int32_t* pos, int M, bf16* kc, bf16* vc,
                                int kv_len, float* lse_out, const LayerWs& w, cudaStream_t st) {
  const a3_model_desc& m = h->m;
  const a3_layer_weights& lw = h->layers[layer];
  const int qd = m.n_q_heads * m.head_dim;
  A3_TRY(rmsnorm_rows(h, x, (const bf16*)lw.attn_norm, m.rms_eps, M, m.d_model, w.a, st));
  A3_TRY(qkv_project(h, layer, w.a, pos, M, 0, w.q, kc, vc, kv_len, st));
  A3_TRY(attention_rows(h, w.q, pos, M, kc, vc, kv_len, w.o, lse_out, w.attn_part, w.attn_part_bytes, st));
  GemmArgs g{};
  g.A = w.o;
  g.M = M;
  g.K = qd;
  g.nseg = 1;
  g.seg[0] = {(const bf16*)lw.wo, nullptr, m.d_model, 0};
  g.C = x;
  g.ldc = m.d_model;
  A3_TRY(gemm_bf16(h, EPI_RESIDUAL, g, st));
  A3_TRY(rmsnorm_rows(h, x, (const bf16*)lw.mlp_norm, m.rms_eps, M, m.d_model, w.a, st));
  GemmArgs u{};
  u.A = w.a;
  u.M = M;
  u.K = m.d_model;
  u.nseg = 1;
  u.seg[0] = {(const bf16*)lw.w_gate, nullptr, m.d_ff, 0};
  u.B2 = (const bf16*)lw.w_up;
  u.C = w.hmid;
  u.ldc = m.d_ff;
  A3_TRY(gemm_bf16(h, EPI_SWIGLU, u, st));
  GemmArgs d{};
  d.A = w.hmid;
  d.M = M;
  d.K = m.d_ff;
  d.nseg = 1;
  d.seg[0] = {(const bf16*)lw.w_down, nullptr, m.d_model, 0};
  d.C = x;
  d.ldc = m.d_model;
  A3_TRY(gemm_bf16(h, EPI_RESIDUAL, d, st));
  return A3_OK;
}
}  // namespace a3

extern "C" int a3_recompute_layer(const a3_handle* h, int layer, void* x_rows, const int32_t* pos, int M, void* k_layer,
                                  void* v_layer, int kv_len, float* lse_out, void* ws, size_t ws_bytes, a3_stream stream) {
  if (!h || layer < 0 || layer >= h->m.n_layers || M < 0 || kv_len < 0) return A3_EINVAL;
  if (M == 0) return A3_OK;
  if (!x_rows || !pos || !k_layer || !v_layer || !ws) return A3_EINVAL;
  if (kv_len > h->m.max_positions || M > kv_len) return A3_EINVAL;
  if (((uintptr_t)x_rows | (uintptr_t)k_layer | (uintptr_t)v_layer | (uintptr_t)ws) & 15) return A3_EINVAL;
  LayerWs w = carve_layer_ws(h, M, ws);
  if (w.bytes > ws_bytes) return A3_EWORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  A3_TRY(check_rows(h, pos, M, kv_len, st));
  return recompute_layer_impl(h, layer, (bf16*)x_rows, pos, M, (bf16*)k_layer, (bf16*)v_layer, kv_len, lse_out, w, st);
}

// ------------------------------------------------------------------ scores (Eq. 3)
extern "C" size_t a3_scores_workspace_bytes(const a3_handle* h, int nq) {
  if (!h || nq < 0) return 0;
  return align_up((size_t)(nq > 0 ? nq : 1) * h->m.n_q_heads * 4, 256) + stats_part_bytes(h, nq);
}

namespace a3 {
// Row log-sum-exps of the question rows (statistics pass of the attention kernel, keys split over the SMs), then the
// score pass.  `part` may be null (no split: one CTA per row tile and KV head).
int scores_with_stats(const a3_handle* h, const bf16* q, const int32_t* q_pos, int nq, const bf16* k, int kv_len, int cand_begin,
                      int cand_end, float* lse, void* part, size_t part_bytes, float* scores, cudaStream_t st) {
  if (nq > 0) A3_TRY(attention_rows(h, q, q_pos, nq, k, k, kv_len, nullptr, lse, part, part_bytes, st));
  return scores_pass(h, q, q_pos, nq, k, kv_len, cand_begin, cand_end, lse, scores, st);
}
}  // namespace a3

extern "C" int a3_query_scores(const a3_handle* h, const void* q_rows, const int32_t* q_pos, int nq, const void* k_layer,
                               int kv_len, int cand_begin, int cand_end, const float* lse, float* scores, void* ws,
                               size_t ws_bytes, a3_stream stream) {
  if (!h || nq < 0 || kv_len < 0 || cand_begin < 0 || cand_end < cand_begin || cand_end > kv_len) return A3_EINVAL;
  if (kv_len == 0) return A3_OK;
  if (!scores || !k_layer) return A3_EINVAL;
  if (nq > 0 && (!q_rows || !q_pos)) return A3_EINVAL;
  if (((uintptr_t)q_rows | (uintptr_t)k_layer) & 15) return A3_EINVAL;
  if (kv_len > h->m.max_positions) return A3_EINVAL;
  cudaStream_t st = (cudaStream_t)stream;
  A3_TRY(check_rows(h, q_pos, nq, kv_len, st));  // the key range of a row tile is taken from its first and last row
  if (!lse && nq > 0) {
    const size_t lse_bytes = align_up((size_t)nq * h->m.n_q_heads * 4, 256);
    if (!ws || ((uintptr_t)ws & 15) || ws_bytes < lse_bytes + stats_part_bytes(h, nq)) return A3_EWORKSPACE;
    return scores_with_stats(h, (const bf16*)q_rows, q_pos, nq, (const bf16*)k_layer, kv_len, cand_begin, cand_end, (float*)ws,
                             (char*)ws + lse_bytes, stats_part_bytes(h, nq), scores, st);
  }
  return scores_pass(h, (const bf16*)q_rows, q_pos, nq, (const bf16*)k_layer, kv_len, cand_begin, cand_end, lse, scores, st);
}

// ------------------------------------------------------------------ the whole request
namespace a3 {
// The host-buffer entry feeds the request: layer_ready[l] is the event after which layer l's chunk caches are in device
// memory; position recovery of layer l is queued behind it, just before the layer needs the cache.  The copies
// themselves are queued a few layers ahead of the compute launches that need them (queue_layer), not all up front:
// thousands of small copies take the host tens of milliseconds to queue, which would otherwise delay the first launch.
// The first full block walks a long input in row panels (same panels whatever the entry point, so that every entry
// point arrives at the same bits): the host-buffer entry copies the embeddings panel by panel and the block starts
// on the first panel while the others are still on their way.
constexpr int X0_PANELS = 4;
constexpr int X0_PANEL_MIN_ROWS = 16384;  // shorter inputs: one panel
static inline int x0_panels(int n) { return n >= X0_PANEL_MIN_ROWS ? X0_PANELS : 1; }
static inline int x0_panel_begin(int n, int i, int panels) { return i >= panels ? n : (int)((long long)n * i / panels) & ~127; }

struct HostFeed {
  const cudaEvent_t* layer_ready;  // [n_layers]
  const cudaEvent_t* x0_ready;     // [x0_panels(n)]: the embeddings of a panel of rows are on the device
  void* ctx;
  int (*queue_layer)(void* ctx, int layer);  // queues the copies of one layer on the copy stream, records layer_ready[layer]
  int next;                                  // first layer whose copies are not queued yet
};
static int fuse_impl(const a3_handle* h, const a3_request* r, void* ws, size_t ws_bytes, a3_stream stream, HostFeed* feed);
}

extern "C" int a3_fuse_request(const a3_handle* h, const a3_request* r, void* ws, size_t ws_bytes, a3_stream stream) {
  return fuse_impl(h, r, ws, ws_bytes, stream, nullptr);
}

// ---------------------------------------------------------------- the request as a CUDA graph
struct a3_graph {
  cudaGraph_t graph;
  cudaGraphExec_t exec;
  int kernels;
};

extern "C" int a3_graph_capture(const a3_handle* h, const a3_request* req, void* ws, size_t ws_bytes, a3_stream stream,
                                a3_graph** out) {
  if (!h || !req || !ws || !out || !stream || h->prof) return A3_EINVAL;
  *out = nullptr;
  cudaStream_t st = (cudaStream_t)stream;
  // once for real: every kernel's one-time attribute set-up happens here, outside the capture
  A3_TRY(a3_fuse_request(h, req, ws, ws_bytes, stream));
  const unsigned long long before = g_launches;
  A3_CUDA(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
  const int status = a3_fuse_request(h, req, ws, ws_bytes, stream);
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(st, &graph);  // always ends the capture, also after a failed request
  const int kernels = (int)(g_launches - before);
  g_launches = before;  // nothing ran during the capture
  if (status != A3_OK || e != cudaSuccess || !graph) {
    if (graph) cudaGraphDestroy(graph);
    if (status != A3_OK) return status;
    return cuda_fail(e != cudaSuccess ? e : cudaErrorUnknown);
  }
  cudaGraphExec_t exec = nullptr;
  const cudaError_t ei = cudaGraphInstantiate(&exec, graph, 0);
  if (ei != cudaSuccess) {
    cudaGraphDestroy(graph);
    return cuda_fail(ei);
  }
  a3_graph* g = (a3_graph*)calloc(1, sizeof(a3_graph));
  if (!g) {
    cudaGraphExecDestroy(exec);
    cudaGraphDestroy(graph);
    return A3_EINVAL;
  }
  g->graph = graph;
  g->exec = exec;
  g->kernels = kernels;
  *out = g;
  return A3_OK;
}

extern "C" int a3_graph_launch(const a3_graph* g, a3_stream stream) {
  if (!g || !g->exec) return A3_EINVAL;
  A3_CUDA(cudaGraphLaunch(g->exec, (cudaStream_t)stream));
  g_launches += (unsigned long long)g->kernels;
  return A3_OK;
}

extern "C" int a3_graph_kernel_count(const a3_graph* g) { return g ? g->kernels : 0; }

extern "C" void a3_graph_destroy(a3_graph* g) {
  if (!g) return;
  if (g->exec) cudaGraphExecDestroy(g->exec);
  if (g->graph) cudaGraphDestroy(g->graph);
  free(g);
}

static int a3::fuse_impl(const a3_handle* h, const a3_request* r, void* ws, size_t ws_bytes, a3_stream stream, HostFeed* feed) {
  if (!h || !r || !ws) return A3_EINVAL;
  const cudaEvent_t* layer_ready = feed ? feed->layer_ready : nullptr;
  const cudaEvent_t* x0_ready = feed ? feed->x0_ready : nullptr;
  // copies of the layers up to `upto` are on their way (host-buffer entry only)
  auto feed_to = [&](int upto) -> int {
    while (feed && feed->next <= upto && feed->next < h->m.n_layers) {
      A3_TRY(feed->queue_layer(feed->ctx, feed->next));
      ++feed->next;
    }
    return A3_OK;
  };
  constexpr int FEED_AHEAD = 3;
  const a3_model_desc& m = h->m;
  if (r->n_ctx < 0 || r->n_question < 0 || r->n_system < 0 || r->n_system > r->n_ctx || r->n_chunks < 0) return A3_EINVAL;
  const int n = r->n_ctx + r->n_question;
  if (n == 0) return A3_OK;
  if (n > m.max_positions) return A3_EINVAL;
  if (r->select_layer < 0 || r->select_layer >= m.n_layers) return A3_EINVAL;
  if (r->score_source != A3_SCORES_TRUE_KEYS && r->score_source != A3_SCORES_CACHED_KEYS) return A3_EINVAL;
  if (r->score_source == A3_SCORES_CACHED_KEYS && layer_ready) return A3_EUNSUPPORTED;
  if (r->selector != A3_SELECT_ATTENTION && r->selector != A3_SELECT_VALUE_DEVIATION) return A3_EINVAL;
  // the value-deviation selector compares true with cached values: it needs the true ones and device-resident chunks
  if (r->selector == A3_SELECT_VALUE_DEVIATION && (r->score_source != A3_SCORES_TRUE_KEYS || layer_ready)) return A3_EUNSUPPORTED;
  const int n_cand = r->n_ctx - r->n_system;
  if (r->n_recompute < 0 || r->n_recompute > n_cand) return A3_EINVAL;
  if (!r->x0 || !r->k_fused || !r->v_fused || !r->rows_out || !r->scores_out || !r->x_out) return A3_EINVAL;
  if (r->n_chunks > 0 && !r->chunks) return A3_EINVAL;
  const size_t layer_bytes = (size_t)n * m.n_kv_heads * m.head_dim * 2;
  if (r->layer_stride < layer_bytes || (r->layer_stride & 15)) return A3_EINVAL;
  if (((uintptr_t)r->x0 | (uintptr_t)r->k_fused | (uintptr_t)r->v_fused | (uintptr_t)r->x_out | (uintptr_t)ws) & 15) return A3_EINVAL;
  RequestWs w = carve_request_ws(h, n, ws);
  if (w.bytes > ws_bytes) return A3_EWORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const int p = r->n_recompute, nq = r->n_question, M = p + nq, ls = r->select_layer;
  LayerWs lw = carve_layer_ws(h, n, w.layer);
  auto kl = [&](int l) { return (bf16*)((char*)r->k_fused + (size_t)l * r->layer_stride); };
  auto vl = [&](int l) { return (bf16*)((char*)r->v_fused + (size_t)l * r->layer_stride); };
  // `ex`: compact copy of every layer's cache, taken right after the layer with its question rows as the window
  const bool evict = r->evict_capacity > 0;
  const int pool = r->evict_pool > 1 ? r->evict_pool : 1;
  const int c_evicted = r->n_system + a3_evict_count(r->evict_capacity, r->n_system, r->n_ctx, nq) + nq;
  if (evict) {
    if (!r->k_evicted || !r->v_evicted || pool % 2 == 0) return A3_EINVAL;
    if (r->evicted_layer_stride < (uint64_t)c_evicted * m.n_kv_heads * m.head_dim * 2 || (r->evicted_layer_stride & 15)) return A3_EINVAL;
    if (((uintptr_t)r->k_evicted | (uintptr_t)r->v_evicted) & 15) return A3_EINVAL;
  }
  // one layer for rows whose last nq entries are the question rows, then (optionally) its eviction
  auto layer_step = [&](int l, bf16* x, const int32_t* pos, int rows) -> int {
    A3_TRY(recompute_layer_impl(h, l, x, pos, rows, kl(l), vl(l), n, evict ? lw.lse : nullptr, lw, st));
    if (!evict) return A3_OK;
    const size_t first_q = (size_t)(rows - nq);
    return a3_evict_layer(h, lw.q + first_q * m.n_q_heads * m.head_dim, pos + first_q, nq, lw.lse + first_q * m.n_q_heads, kl(l), vl(l), n,
                          r->n_system, r->n_ctx, r->evict_capacity, pool, (char*)r->k_evicted + (size_t)l * r->evicted_layer_stride,
                          (char*)r->v_evicted + (size_t)l * r->evicted_layer_stride,
                          r->kept_out ? r->kept_out + (size_t)l * m.n_kv_heads * c_evicted : nullptr, w.evict, w.evict_bytes, stream);
  };

  if (r->score_source == A3_SCORES_CACHED_KEYS) {
    // Scores against the recovered cached keys: every layer is position-recovered; only the question rows pass
    // through the leading blocks; rows [Re, Q] are recomputed through every layer from the embeddings.
    A3_TRY(a3_rope_rerotate(h, r->chunks, r->n_chunks, r->max_chunk_len, r->k_fused, r->v_fused, r->layer_stride, r->n_ctx, 0, m.n_layers, stream));
    A3_TRY(iota_rows(h, w.all_pos, 0, n, st));
    const int32_t* q_pos = w.all_pos + r->n_ctx;
    A3_CUDA(cudaMemsetAsync(r->scores_out, 0, (size_t)n * 4, st));
    if (nq > 0) {
      bf16* xq = w.x_all;  // [nq][d] scratch for the question rows
      A3_CUDA(cudaMemcpyAsync(xq, (const bf16*)r->x0 + (size_t)r->n_ctx * m.d_model, (size_t)nq * m.d_model * 2, cudaMemcpyDeviceToDevice, st));
      for (int l = 0; l < ls; ++l) A3_TRY(recompute_layer_impl(h, l, xq, q_pos, nq, kl(l), vl(l), n, nullptr, lw, st));
      A3_TRY(rmsnorm_rows(h, xq, (const bf16*)h->layers[ls].attn_norm, m.rms_eps, nq, m.d_model, lw.a, st));
      A3_TRY(qkv_project(h, ls, lw.a, q_pos, nq, 0, lw.q, kl(ls), vl(ls), n, st));
      A3_TRY(scores_with_stats(h, lw.q, q_pos, nq, kl(ls), n, r->n_system, r->n_ctx, w.lse_q, lw.attn_part, lw.attn_part_bytes,
                               r->scores_out, st));
    }
    if (p > 0) {
      if (r->forced_re) A3_CUDA(cudaMemcpyAsync(r->rows_out, r->forced_re, (size_t)p * 4, cudaMemcpyDeviceToDevice, st));
      else A3_TRY(a3_topk_select(h, r->scores_out, r->n_system, r->n_ctx, p, r->rows_out, stream));
    }
    A3_TRY(iota_rows(h, r->rows_out + p, r->n_ctx, nq, st));
    if (M == 0) return A3_OK;
    A3_TRY(check_rows(h, r->rows_out, M, n, st));
    A3_TRY(a3_gather_rows(h, r->x0, n, r->rows_out, M, m.d_model, r->x_out, stream));
    for (int l = 0; l < m.n_layers; ++l) A3_TRY(layer_step(l, (bf16*)r->x_out, r->rows_out, M));
    return A3_OK;
  }

  // Position recovery (Eq. 2) in one launch.  Layers up to the selection layer are skipped: every row of their
  // caches is rewritten with true values below (full blocks; K/V of all rows at the selection layer), so the
  // recovered values would never be read.
  if (!layer_ready && ls + 1 < m.n_layers)
    A3_TRY(a3_rope_rerotate(h, r->chunks, r->n_chunks, r->max_chunk_len, r->k_fused, r->v_fused, r->layer_stride, r->n_ctx, ls + 1,
                            m.n_layers, stream));
  // leading full blocks: the whole input through layers 0..select_layer-1
  const int panels = x0_panels(n);
  A3_TRY(iota_rows(h, w.all_pos, 0, n, st));
  for (int i = 0; i < panels; ++i) {
    const int r0 = x0_panel_begin(n, i, panels), r1 = x0_panel_begin(n, i + 1, panels);
    if (x0_ready) A3_CUDA(cudaStreamWaitEvent(st, x0_ready[i], 0));
    A3_CUDA(cudaMemcpyAsync(w.x_all + (size_t)r0 * m.d_model, (const bf16*)r->x0 + (size_t)r0 * m.d_model, (size_t)(r1 - r0) * m.d_model * 2,
                            cudaMemcpyDeviceToDevice, st));
    if (ls > 0) {
      // block 0 on this panel of rows: they attend to the rows before them, whose K/V the earlier panels have written
      if (i == 0) A3_TRY(feed_to(ls + 1 + FEED_AHEAD));  // a full block is long: several layers' copies fit under it
      if (i + 1 < panels) A3_TRY(recompute_layer_impl(h, 0, w.x_all + (size_t)r0 * m.d_model, w.all_pos + r0, r1 - r0, kl(0), vl(0), n, nullptr, lw, st));
      else A3_TRY(layer_step(0, w.x_all + (size_t)r0 * m.d_model, w.all_pos + r0, r1 - r0));
    }
  }
  for (int l = 1; l < ls; ++l) {
    A3_TRY(feed_to(ls + 1 + FEED_AHEAD * (l + 1)));
    A3_TRY(layer_step(l, w.x_all, w.all_pos, n));
  }
  A3_TRY(feed_to(ls + 1 + FEED_AHEAD));
  // selection layer: true K, V for all rows, queries of the question rows, scores, Re (Eq. 3)
  A3_TRY(rmsnorm_rows(h, w.x_all, (const bf16*)h->layers[ls].attn_norm, m.rms_eps, n, m.d_model, lw.a, st));
  A3_TRY(qkv_project(h, ls, lw.a, w.all_pos, n, r->n_ctx, lw.q, kl(ls), vl(ls), n, st));
  A3_CUDA(cudaMemsetAsync(r->scores_out, 0, (size_t)n * 4, st));
  if (r->selector == A3_SELECT_VALUE_DEVIATION) {
    A3_TRY(value_deviation(h, r->chunks, r->n_chunks, r->max_chunk_len, ls, vl(ls), r->n_system, r->n_ctx, r->scores_out, st));
  } else if (nq > 0) {
    A3_TRY(scores_with_stats(h, lw.q, w.all_pos + r->n_ctx, nq, kl(ls), n, r->n_system, r->n_ctx, w.lse_q, lw.attn_part,
                             lw.attn_part_bytes, r->scores_out, st));
  }
  if (p > 0) {
    if (r->forced_re) A3_CUDA(cudaMemcpyAsync(r->rows_out, r->forced_re, (size_t)p * 4, cudaMemcpyDeviceToDevice, st));
    else A3_TRY(a3_topk_select(h, r->scores_out, r->n_system, r->n_ctx, p, r->rows_out, stream));
  }
  A3_TRY(iota_rows(h, r->rows_out + p, r->n_ctx, nq, st));
  if (M == 0) {
    A3_TRY(feed_to(m.n_layers));
    if (layer_ready)
      for (int l = ls + 1; l < m.n_layers; ++l) {
        A3_CUDA(cudaStreamWaitEvent(st, layer_ready[l], 0));
        A3_TRY(a3_rope_rerotate(h, r->chunks, r->n_chunks, r->max_chunk_len, r->k_fused, r->v_fused, r->layer_stride, r->n_ctx, l, l + 1, stream));
      }
    return A3_OK;
  }
  A3_TRY(check_rows(h, r->rows_out, M, n, st));
  A3_TRY(a3_gather_rows(h, w.x_all, n, r->rows_out, M, m.d_model, r->x_out, stream));
  // layers select_layer..L-1 on rows [Re, Q] only (Eq. 4, Eq. 5)
  for (int l = ls; l < m.n_layers; ++l) {
    A3_TRY(feed_to(l + FEED_AHEAD));
    if (layer_ready && l > ls) {
      A3_CUDA(cudaStreamWaitEvent(st, layer_ready[l], 0));
      A3_TRY(a3_rope_rerotate(h, r->chunks, r->n_chunks, r->max_chunk_len, r->k_fused, r->v_fused, r->layer_stride, r->n_ctx, l, l + 1, stream));
    }
    A3_TRY(layer_step(l, (bf16*)r->x_out, r->rows_out, M));
  }
  return A3_OK;
}

extern "C" int a3_precompute_chunk(const a3_handle* h, void* x_chunk, int T, void* k_chunk, void* v_chunk,
                                   uint64_t layer_stride, void* ws, size_t ws_bytes, a3_stream stream) {
  if (!h || T < 0) return A3_EINVAL;
  if (T == 0) return A3_OK;
  if (!x_chunk || !k_chunk || !v_chunk || !ws) return A3_EINVAL;
  const a3_model_desc& m = h->m;
  if (T > m.max_positions) return A3_EINVAL;
  if (layer_stride < (uint64_t)T * m.n_kv_heads * m.head_dim * 2 || (layer_stride & 15)) return A3_EINVAL;
  if (((uintptr_t)x_chunk | (uintptr_t)k_chunk | (uintptr_t)v_chunk | (uintptr_t)ws) & 15) return A3_EINVAL;
  RequestWs w = carve_request_ws(h, T, ws);
  if (w.bytes > ws_bytes) return A3_EWORKSPACE;
  LayerWs lw = carve_layer_ws(h, T, w.layer);
  cudaStream_t st = (cudaStream_t)stream;
  A3_TRY(iota_rows(h, w.all_pos, 0, T, st));
  for (int l = 0; l < m.n_layers; ++l)
    A3_TRY(recompute_layer_impl(h, l, (bf16*)x_chunk, w.all_pos, T, (bf16*)((char*)k_chunk + (size_t)l * layer_stride),
                                (bf16*)((char*)v_chunk + (size_t)l * layer_stride), T, nullptr, lw, st));
  return A3_OK;
}

extern "C" int a3_fuse_batch(const a3_handle* h, const a3_request* reqs, int n_requests, void* ws, size_t ws_bytes,
                             a3_stream stream) {
  if (!h || n_requests < 0 || (n_requests > 0 && !reqs)) return A3_EINVAL;
  for (int i = 0; i < n_requests; ++i) A3_TRY(a3_fuse_request(h, &reqs[i], ws, ws_bytes, stream));
  return A3_OK;
}

// ------------------------------------------------------------------ host-buffer entry
extern "C" size_t a3_host_staging_bytes(const a3_handle* h, int n_ctx, int n) {
  if (!h || n_ctx < 0 || n < n_ctx) return 0;
  const a3_model_desc& m = h->m;
  const size_t row = (size_t)m.n_kv_heads * m.head_dim * 2;
  // chunk K and V of all layers, embeddings, descriptors (one per token is an upper bound on chunks)
  return align_up(2 * (size_t)m.n_layers * n_ctx * row, 256) + align_up((size_t)n * m.d_model * 2, 256) +
         align_up((size_t)(n_ctx + 1) * sizeof(a3_chunk_ref), 256);
}

namespace a3 {
// copy stream and events of the host-buffer entry, created on first use and kept by the handle
struct HostPipe {
  cudaStream_t copy_stream;
  cudaEvent_t start, x0_ready[X0_PANELS];
  cudaEvent_t* layer_ready;
  int n_layers;
  a3_chunk_ref* href;  // host copy of the chunk descriptors of the last call
  int href_cap;
};
static int host_pipe(const a3_handle* h, HostPipe** out) {
  a3_handle* hm = const_cast<a3_handle*>(h);
  if (!hm->host_pipe) {
    HostPipe* p = (HostPipe*)calloc(1, sizeof(HostPipe));
    if (!p) return A3_EINVAL;
    p->n_layers = h->m.n_layers;
    p->layer_ready = (cudaEvent_t*)calloc(p->n_layers, sizeof(cudaEvent_t));
    cudaError_t e = cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->start, cudaEventDisableTiming);
    for (int i = 0; i < X0_PANELS && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&p->x0_ready[i], cudaEventDisableTiming);
    for (int l = 0; l < p->n_layers && e == cudaSuccess; ++l) e = cudaEventCreateWithFlags(&p->layer_ready[l], cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(e);
    hm->host_pipe = p;
  }
  *out = (HostPipe*)hm->host_pipe;
  return A3_OK;
}
static void host_pipe_destroy(a3_handle* h) {
  HostPipe* p = (HostPipe*)h->host_pipe;
  if (!p) return;
  for (int l = 0; l < p->n_layers; ++l)
    if (p->layer_ready[l]) cudaEventDestroy(p->layer_ready[l]);
  if (p->start) cudaEventDestroy(p->start);
  for (int i = 0; i < X0_PANELS; ++i)
    if (p->x0_ready[i]) cudaEventDestroy(p->x0_ready[i]);
  if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
  free(p->layer_ready);
  free(p->href);
  free(p);
  h->host_pipe = nullptr;
}
}  // namespace a3

// Copies run on the handle's own copy stream, layer by layer, while the compute stream works: the embeddings go
// first (the full block needs only them), then each layer's chunk caches; position recovery of a layer is queued
// behind that layer's copy.  Layers up to the selection layer are never copied: their caches are recomputed.
extern "C" int a3_fuse_request_host(const a3_handle* h, const a3_request* req, const a3_host_io* io, void* staging,
                                    size_t staging_bytes, void* ws, size_t ws_bytes, a3_stream stream) {
  if (!h || !req || !io || !staging) return A3_EINVAL;
  if (!io->x0 || !io->rows_out || !io->x_out) return A3_EINVAL;
  if (req->n_chunks > 0 && (!io->chunk_k || !io->chunk_v || !io->chunk_len)) return A3_EINVAL;
  const a3_model_desc& m = h->m;
  const int n = req->n_ctx + req->n_question;
  if (req->n_ctx < 0 || req->n_question < 0 || req->n_chunks < 0 || req->n_chunks > req->n_ctx + 1) return A3_EINVAL;
  if (req->select_layer < 0 || req->select_layer >= m.n_layers) return A3_EINVAL;
  if (a3_host_staging_bytes(h, req->n_ctx, n) > staging_bytes) return A3_EWORKSPACE;
  HostPipe* hp = nullptr;
  A3_TRY(host_pipe(h, &hp));
  cudaStream_t st = (cudaStream_t)stream, cs = hp->copy_stream;
  const size_t row = (size_t)m.n_kv_heads * m.head_dim * 2;
  char* base = (char*)staging;
  char* kv = base;
  char* x0 = base + align_up(2 * (size_t)m.n_layers * req->n_ctx * row, 256);
  a3_chunk_ref* dref = (a3_chunk_ref*)(x0 + align_up((size_t)n * m.d_model * 2, 256));
  // host copy of the descriptors: kept by the handle and grown on demand, so that a steady stream of calls allocates nothing
  if (hp->href_cap < req->n_chunks) {
    a3_chunk_ref* grown = (a3_chunk_ref*)realloc(hp->href, sizeof(a3_chunk_ref) * (size_t)req->n_chunks);
    if (!grown) return A3_EINVAL;
    hp->href = grown;
    hp->href_cap = req->n_chunks;
  }
  a3_chunk_ref* href = hp->href;
  int off = 0, maxlen = 0;
  size_t kvoff = 0;
  for (int c = 0; c < req->n_chunks; ++c) {
    const int len = io->chunk_len[c];
    if (len < 0 || off + len > req->n_ctx) return A3_EINVAL;
    const size_t bytes = (size_t)m.n_layers * len * row;
    href[c].k_src = kv + kvoff;
    href[c].v_src = kv + kvoff + bytes;
    href[c].src_layer_stride = (uint64_t)len * row;
    href[c].len = len;
    href[c].dst_offset = off;
    href[c].delta = off;
    href[c].token_step = 0;  // the host entry takes chunks stored at local positions
    kvoff += 2 * bytes;
    off += len;
    if (len > maxlen) maxlen = len;
  }
  if (off != req->n_ctx) return A3_EINVAL;
  // From here on copies are in flight: every exit waits for both streams first, so that the caller may reuse or free
  // its host buffers and the staging area whatever the status.
  int status = A3_OK;
  auto note = [&](cudaError_t e) {
    if (e != cudaSuccess && status == A3_OK) status = cuda_fail(e);
    return status == A3_OK;
  };
  // the copy stream starts after whatever the caller has already queued on `stream` (the staging area may be in use)
  note(cudaEventRecord(hp->start, st));
  if (status == A3_OK) note(cudaStreamWaitEvent(cs, hp->start, 0));
  // the descriptor array is pageable host memory: this copy returns only once it has been staged
  if (status == A3_OK && req->n_chunks > 0)
    note(cudaMemcpyAsync(dref, href, sizeof(a3_chunk_ref) * req->n_chunks, cudaMemcpyHostToDevice, cs));
  const int panels = x0_panels(n);
  for (int i = 0; i < panels && status == A3_OK; ++i) {
    const int r0 = x0_panel_begin(n, i, panels), r1 = x0_panel_begin(n, i + 1, panels);
    if (note(cudaMemcpyAsync(x0 + (size_t)r0 * m.d_model * 2, (const char*)io->x0 + (size_t)r0 * m.d_model * 2, (size_t)(r1 - r0) * m.d_model * 2,
                             cudaMemcpyHostToDevice, cs)))
      note(cudaEventRecord(hp->x0_ready[i], cs));
  }
  a3_request r = *req;
  r.chunks = dref;
  r.max_chunk_len = maxlen;
  r.x0 = x0;
  struct FeedCtx {
    const a3_chunk_ref* href;
    const a3_host_io* io;
    int n_chunks;
    size_t row;
    cudaStream_t cs;
    cudaEvent_t* layer_ready;
  } fc{href, io, req->n_chunks, row, cs, hp->layer_ready};
  HostFeed feed{hp->layer_ready, hp->x0_ready, &fc,
                [](void* ctx, int l) -> int {
                  FeedCtx* f = (FeedCtx*)ctx;
                  for (int c = 0; c < f->n_chunks; ++c) {
                    const size_t slice = (size_t)f->href[c].len * f->row;
                    A3_CUDA(cudaMemcpyAsync((char*)f->href[c].k_src + l * slice, (const char*)f->io->chunk_k[c] + l * slice, slice, cudaMemcpyHostToDevice, f->cs));
                    A3_CUDA(cudaMemcpyAsync((char*)f->href[c].v_src + l * slice, (const char*)f->io->chunk_v[c] + l * slice, slice, cudaMemcpyHostToDevice, f->cs));
                  }
                  A3_CUDA(cudaEventRecord(f->layer_ready[l], f->cs));
                  return A3_OK;
                },
                req->select_layer + 1};
  if (status == A3_OK) status = fuse_impl(h, &r, ws, ws_bytes, stream, &feed);
  const int M = r.n_recompute + r.n_question;
  if (status == A3_OK && M > 0) {
    if (note(cudaMemcpyAsync(io->rows_out, r.rows_out, (size_t)M * 4, cudaMemcpyDeviceToHost, st)))
      note(cudaMemcpyAsync(io->x_out, r.x_out, (size_t)M * m.d_model * 2, cudaMemcpyDeviceToHost, st));
  }
  note(cudaStreamSynchronize(cs));  // the copy stream first: the compute stream may be waiting on its events
  const cudaError_t es = cudaStreamSynchronize(st);
  if (es != cudaSuccess && status == A3_OK) status = cuda_fail(es);
  return status;
}

/*
 * a3.h - C ABI of the B200 (sm_100a) hot path of attention-aware KV-cache fusion (A^3).
 *
 * The library fuses KV caches that were prefilled chunk by chunk (Eq. 1) into one
 * cache for the concatenated input X = (S, D_1..D_k, Q): position recovery (Eq. 2),
 * question->context relevance scores and top-p selection (Eq. 3), and recomputation
 * of the selected rows [Re, Q] over the fused cache (Eq. 4, Eq. 5).
 *
 * Conventions
 *  - "dev" pointers are CUDA device pointers, "host" pointers ordinary host memory.
 *  - Tensors are bf16 (2 bytes, row-major) unless stated; scores and log-sum-exps are
 *    fp32; indices and positions int32.
 *  - A per-layer KV cache is [slots][n_kv_heads][head_dim]; a token's global position
 *    is its cache slot.  Linear maps are stored [out][in] (y = x W^T).
 *  - The caller owns every buffer (weights, chunk caches, fused cache, workspace,
 *    outputs).  The handle borrows the weight pointers for its lifetime and owns only
 *    its RoPE table, a small status block and tensor-map descriptors.
 *  - Hot calls allocate nothing, do not synchronise and copy nothing between host and
 *    device (a3_fuse_request_host excepted); all work is queued on `stream`
 *    (a cudaStream_t passed as void*).  Calls on different streams may overlap only if
 *    they use different workspaces.  A handle may be used from several host threads as
 *    long as the calls on it do not run at the same time (the launch counter, the
 *    profiling records and the lazily created copy stream are not locked); device
 *    memory and kernels are per call and need no such care.
 *  - Return value: A3_OK or a negative a3_status.  Host-detectable problems are
 *    rejected before any launch.  Problems only the device can see (a position outside
 *    the cache, a non-finite score, an exhausted bounded wait) set the handle's device
 *    status word and the kernel skips the offending access; read it with
 *    a3_device_status.  No kernel traps.
 *  - Supported shapes: head_dim 64 or 128; d_model, n_q_heads*head_dim,
 *    n_kv_heads*head_dim and d_ff multiples of 128; n_q_heads a multiple of n_kv_heads.
 *    Row counts, chunk lengths and cache lengths are arbitrary.
 */
#ifndef A3_H_
#define A3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct a3_handle a3_handle;
typedef void* a3_stream; /* cudaStream_t */

typedef enum {
  A3_OK = 0,
  A3_EINVAL = -1,       /* bad argument (null pointer, negative size, range) */
  A3_EUNSUPPORTED = -2, /* shape outside the supported set */
  A3_EWORKSPACE = -3,   /* workspace too small */
  A3_ECUDA = -4,        /* a CUDA call failed; see a3_last_cuda_error */
  A3_EDEVICE = -5,      /* a kernel recorded a problem in the device status word */
  A3_ETOOLARGE = -6     /* the request exceeds a fixed built-in limit (a3_query_scores_static) */
} a3_status;

/* Device status bits (a3_device_status). */
#define A3_DEV_BAD_POSITION 1u   /* a row position / slot was outside [0, kv_len) */
#define A3_DEV_NONFINITE_SCORE 2u
#define A3_DEV_WAIT_EXHAUSTED 4u /* a bounded barrier wait gave up */
#define A3_DEV_UNSORTED_ROWS 8u  /* row positions not strictly ascending */

typedef struct {
  int n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff;
  double rope_theta;  /* base of theta_i = base^(-2i/head_dim) (Position Recovery) */
  float rms_eps;
  int rope_layout;    /* 0: pairs (i, i+D/2); 1: pairs (2i, 2i+1) as the matrix before Eq. 2 */
  int max_positions;  /* RoPE table rows: largest global position + 1 ever used */
} a3_model_desc;

/* One decoder block; all dev pointers to bf16.  bq/bk/bv may be NULL. */
typedef struct {
  const void *attn_norm, *wq, *wk, *wv, *bq, *bk, *bv, *wo, *mlp_norm, *w_gate, *w_up, *w_down;
} a3_layer_weights;

/* One precomputed chunk (Eq. 1): K_i, V_i of all layers.  Position recovery (Eq. 2) rotates the key of token t
 * by delta + token_step * t positions:
 *   stored at local positions 0..len-1 (the default):            delta = dst_offset, token_step = 0
 *   stored without positional embedding (Eq. 2 as printed):      delta = dst_offset, token_step = 1
 *   converting local-position storage to storage without one:    delta = 0,          token_step = -1 */
typedef struct {
  const void* k_src;          /* dev, [n_layers][len][Hkv][D], layer l at k_src + l*src_layer_stride */
  const void* v_src;          /* dev, same layout */
  uint64_t src_layer_stride;  /* bytes between consecutive layers of this chunk */
  int32_t len;                /* tokens in the chunk */
  int32_t dst_offset;         /* first slot of the chunk in the fused cache (o_c) */
  int32_t delta;              /* rotation of token 0: global minus stored position (= dst_offset for local storage) */
  int32_t token_step;         /* additional rotation per token index: 0, +1 or -1 (see above) */
} a3_chunk_ref;

/* Which keys the relevance scores (Eq. 3) are taken against.
 * A3_SCORES_TRUE_KEYS: the Attention Recovery subsection as written - the whole input passes through the blocks
 *   below select_layer, K_true of every row is formed at select_layer, rows [Re, Q] are recomputed from there on.
 * A3_SCORES_CACHED_KEYS: only the question rows pass through the leading blocks (over the position-recovered
 *   cache); their queries are scored against the recovered cached keys of select_layer; rows [Re, Q] are then
 *   recomputed through every layer from the embeddings.  Skips the full blocks (about 15 % of the work at
 *   10 x 512 tokens, r = 0.15); not supported by a3_fuse_request_host. */
#define A3_SCORES_TRUE_KEYS 0
#define A3_SCORES_CACHED_KEYS 1

/* What ranks the candidates.  A3_SELECT_ATTENTION is Eq. 3.  A3_SELECT_VALUE_DEVIATION is the comparison method
 * of the Baselines paragraph (CacheBlend): score = squared distance between a token's cached value and its true
 * value at select_layer, over all KV heads and channels (needs A3_SCORES_TRUE_KEYS, which forms the true values);
 * scores_out then holds these distances.  Index-only selections (chunk edges - a3_chunk_edge_rows -, random -
 * a3_random_rows -) are passed through forced_re. */
#define A3_SELECT_ATTENTION 0
#define A3_SELECT_VALUE_DEVIATION 1

/* One fusion request.  Slots [0, n_ctx) are the chunks in input order, [n_ctx, n_ctx+n_question)
 * the question.  Slots [0, n_system) (a system prompt) are attendable but never candidates. */
typedef struct {
  const a3_chunk_ref* chunks; /* dev array [n_chunks] */
  int32_t n_chunks, max_chunk_len;
  int32_t n_ctx, n_question, n_system;
  int32_t select_layer;       /* layer whose true Q/K give the scores (paper: 1) */
  int32_t n_recompute;        /* p = |Re| (a3_recompute_count) */
  int32_t score_source;       /* A3_SCORES_TRUE_KEYS (0, the paper's text) or A3_SCORES_CACHED_KEYS */
  int32_t selector;           /* A3_SELECT_ATTENTION (0, Eq. 3) or A3_SELECT_VALUE_DEVIATION */
  int32_t reserved;
  const void* x0;             /* dev [n][d_model]: embeddings of the whole input */
  void* k_fused;              /* dev [n_layers][n][Hkv][D], layer l at + l*layer_stride */
  void* v_fused;
  uint64_t layer_stride;      /* bytes */
  const int32_t* forced_re;   /* dev [n_recompute] ascending, or NULL: replaces the selection */
  int32_t* rows_out;          /* dev [n_recompute + n_question]: R = Re (ascending) then question slots */
  float* scores_out;          /* dev [n]: s(d_i) on candidates, 0 elsewhere */
  void* x_out;                /* dev [n_recompute + n_question][d_model]: final hidden rows of R */
  /* `ex` (Extension subsection), optional: with evict_capacity > 0 every layer's fused cache is also written in
   * compact form right after the layer has been recomputed, using that layer's question rows as the window
   * (a3_evict_layer).  C' = n_system + a3_evict_count(...) + n_question entries per layer. */
  int32_t evict_capacity;     /* C; 0: no eviction */
  int32_t evict_pool;         /* odd pooling width, 0 or 1: off */
  void* k_evicted;            /* dev [n_layers][C'][Hkv][D], layer l at + l*evicted_layer_stride */
  void* v_evicted;
  uint64_t evicted_layer_stride; /* bytes */
  int32_t* kept_out;          /* dev [n_layers][Hkv][C'] or NULL */
} a3_request;

/* Host buffers for a3_fuse_request_host (pinned memory recommended). */
typedef struct {
  const void* const* chunk_k; /* host array [n_chunks] of host pointers, each [n_layers][len][Hkv][D] */
  const void* const* chunk_v;
  const int32_t* chunk_len;   /* host [n_chunks] */
  const void* x0;             /* host [n][d_model] */
  int32_t* rows_out;          /* host [n_recompute + n_question] */
  void* x_out;                /* host [n_recompute + n_question][d_model] */
} a3_host_io;

/* Kernel-variant choices of a handle (a3_set_option).  Several steps exist in more than one kernel variant; by
 * default the launcher picks one from the shape.  These options pin a variant on ONE handle, for cross-checks
 * (every variant must meet the same tolerances; some pairs are bit-identical) and for measurements.  They are plain
 * fields of the handle: set them while no call on the handle is in flight. */
typedef enum {
  A3_OPT_ATTN_SPLIT = 0,        /* attention, one row tile per CTA: key segments per row tile; 0 = choose (default) */
  A3_OPT_ATTN_PAIR,             /* two-row-tile attention kernel: -1 choose (default), 0 never, 1 whenever supported */
  A3_OPT_ATTN_MAX_CTAS,         /* cap on the persistent attention grid; 0 = one CTA per SM (default) */
  A3_OPT_SWIGLU_NARROW,         /* one-CTA gate/up GEMM: 0 uniform tiles, 1 narrower last wave (default), 16..120 forced width */
  A3_OPT_SWIGLU_PAIR,           /* persistent CTA-pair gate/up GEMM: 0 never, 1 whenever the shape allows (default) */
  A3_OPT_RESIDUAL_T,            /* persistent CTA-pair C += A B^T: 0 never, 1 by shape (default), 2 whenever the shape allows */
  A3_OPT_GEMM_BN_RESIDUAL,      /* tile width of the tile GEMMs per epilogue; 0 = choose; 512 = the 256 x 256 CTA-pair tile */
  A3_OPT_GEMM_BN_SWIGLU,
  A3_OPT_GEMM_BN_QKV,
  A3_OPT_GEMM_STAGES_RESIDUAL,  /* pipeline depth that goes with the width above */
  A3_OPT_GEMM_STAGES_SWIGLU,
  A3_OPT_GEMM_STAGES_QKV,
  A3_OPT_SCORES_KERNEL,         /* relevance scores: 0 choose (default), 1 the tcgen05 kernel, 2 the warp-level MMA kernel */
  A3_OPT_QKV_T,                 /* persistent CTA-pair QKV projection (one head per CTA): 0 never, 1 whenever the shape allows (default) */
  A3_OPT_GEMM_TILING,           /* persistent CTA-pair GEMMs, token tiles: 0 widths that balance the pairs' loads (default), 1 even split */
  A3_OPT_COUNT
} a3_option;

/* ---- lifetime ---------------------------------------------------------------------- */

/* Creates a handle on the current device: checks the shape, borrows `layers` (host array
 * [n_layers] of dev pointers, copied), builds the fp32 cos/sin table [max_positions][D/2]
 * from float64 angles.  Allocates; not a hot call. */
int a3_create(a3_handle** out, const a3_model_desc* model, const a3_layer_weights* layers);
void a3_destroy(a3_handle* h);

/* Sets one a3_option of the handle.  A3_EINVAL for an unknown option; values outside an option's range fall back
 * to the default behaviour at the launch that reads them.  Host only; no device work. */
int a3_set_option(a3_handle* h, int option, int value);

/* Bytes of workspace a3_recompute_layer needs for max_rows rows (also enough for
 * a3_query_scores / a3_topk_select on caches up to max_rows slots). */
size_t a3_layer_workspace_bytes(const a3_handle* h, int max_rows);
/* Bytes of workspace a3_fuse_request needs for an input of n slots (chunks + question). */
size_t a3_request_workspace_bytes(const a3_handle* h, int n);
/* Additional device staging bytes a3_fuse_request_host needs. */
size_t a3_host_staging_bytes(const a3_handle* h, int n_ctx, int n);

/* Slots of the first m and last m tokens of every chunk, ascending, without slots below n_system (the comparison
 * method of the Baselines paragraph, LegoLink: m = 20).  chunk_len: host [n_chunks].  Writes at most `capacity`
 * slots to rows_out (host; may be NULL) and returns the full count.  Host only. */
int a3_chunk_edge_rows(const int32_t* chunk_len, int n_chunks, int m, int n_system, int32_t* rows_out, int capacity);

/* k distinct slots of [cand_begin, cand_end) drawn uniformly at random, ascending: the random selection the other
 * selectors are compared with (Attention Recovery subsection, discussion of Figure 3).  Counter-based and
 * reproducible: with n = cand_end - cand_begin candidates 0..n-1 in an array, step i = 0..k-1 swaps entry i with
 * entry i + (mix(seed + i) mod (n - i)), where mix is the SplitMix64 finaliser
 *   z = x + 0x9E3779B97F4A7C15; z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9; z = (z ^ (z >> 27)) * 0x94D049BB133111EB;
 *   mix = z ^ (z >> 31)                                            (64-bit unsigned arithmetic);
 * the first k entries, sorted, plus cand_begin are the result.  k is clamped to n.  Writes at most `capacity` slots
 * to rows_out (host; may be NULL) and returns the count.  Host only. */
int a3_random_rows(uint64_t seed, int cand_begin, int cand_end, int k, int32_t* rows_out, int capacity);

/* p = min(n_candidates, floor(ratio * n + 1e-9)): the size of Re (Eq. 3, p = r n). Host only. */
int a3_recompute_count(double ratio, int n, int n_candidates);

/* ---- the steps --------------------------------------------------------------------- */

/* Position recovery (Eq. 2): for layers [layer_begin, layer_end), every chunk c, token t:
 *   k_fused[l][dst_offset+t] = R(delta + token_step*t) k_src[l][t]   (rotation per head, fp32 arithmetic)
 *   v_fused[l][dst_offset+t] = v_src[l][t]
 * chunks: dev array; max_chunk_len >= every len (host copy of the largest length, sizes the grid).
 * Fused layer l lives at k_fused + l*layer_stride bytes and has kv_len slots (kv_len rows must fit in
 * layer_stride).  A chunk whose slots [dst_offset, dst_offset + len) do not lie inside [0, kv_len), whose len
 * exceeds max_chunk_len, or whose rotation leaves the RoPE table is skipped as a whole - nothing of it is written -
 * and A3_DEV_BAD_POSITION is set. */
int a3_rope_rerotate(const a3_handle* h, const a3_chunk_ref* chunks, int n_chunks, int max_chunk_len,
                     void* k_fused, void* v_fused, uint64_t layer_stride, int kv_len, int layer_begin, int layer_end,
                     a3_stream stream);

/* Relevance scores (Eq. 3): scores[i] = sum over question rows j and query heads h of
 * Softmax_row(q_{j,h} K^T / sqrt(D))[i] for i in [cand_begin, cand_end), 0 for other i < kv_len.
 * Each softmax row runs over slots 0..q_pos[j].  q_rows: dev [nq][Hq][D], already rotated;
 * q_pos: dev [nq], strictly ascending, each in [0, kv_len) (checked on the device: A3_DEV_UNSORTED_ROWS /
 * A3_DEV_BAD_POSITION).  k_layer: dev [kv_len][Hkv][D].  lse: dev [nq][Hq] natural-log row log-sum-exps of the
 * scaled logits (as a3_recompute_layer emits) or NULL, in which case a statistics pass runs first (ws then needs
 * a3_scores_workspace_bytes(h, nq) bytes).  The result is deterministic (fixed summation order). */
size_t a3_scores_workspace_bytes(const a3_handle* h, int nq);
int a3_query_scores(const a3_handle* h, const void* q_rows, const int32_t* q_pos, int nq, const void* k_layer,
                    int kv_len, int cand_begin, int cand_end, const float* lse, float* scores, void* ws,
                    size_t ws_bytes, a3_stream stream);

/* a3_query_scores without a workspace, for callers that cannot allocate device memory where they need the
 * scores (for example a serving engine that gave all free HBM to its KV-cache pool at start-up, or plug-in code
 * inside a framework that owns the allocator).  The paper has no counterpart: this is a packaging variant of the
 * call above, with the same arguments minus lse/ws and the same result, bit for bit.  The row log-sum-exps and
 * the partial statistics of the pass that computes them go to a fixed array inside the library image:
 * A3_STATIC_SCRATCH_BYTES (1 MiB: room for A3_STATIC_LSE_MAX log-sum-exps plus 768 KiB of partial statistics) that
 * every GPU which loads the library holds until the process exits.  nq * n_q_heads above A3_STATIC_LSE_MAX
 * returns A3_ETOOLARGE and launches nothing.
 * The call makes no allocation of any kind.  Its first call on a device looks up the array's device address
 * (once per device; that device must be current and must be the handle's) and should therefore be made before
 * any stream capture begins.  All calls share the array; it keeps the previous call's contents, and nothing in
 * it needs clearing because each call overwrites the entries it later reads.  Calls whose kernels may overlap
 * on the GPU race on it: order them. */
#define A3_STATIC_LSE_MAX 65536
#define A3_STATIC_SCRATCH_BYTES (A3_STATIC_LSE_MAX * 4 + 768 * 1024)
int a3_query_scores_static(const a3_handle* h, const void* q_rows, const int32_t* q_pos, int nq, const void* k_layer,
                           int kv_len, int cand_begin, int cand_end, float* scores, a3_stream stream);

/* Selection (Eq. 3, Re = top_p(s)): the k slots of [cand_begin, cand_end) with the largest score;
 * ties go to the lower slot; idx_out (dev [k]) is ascending.  k is clamped to the candidate count. */
int a3_topk_select(const a3_handle* h, const float* scores, int cand_begin, int cand_end, int k,
                   int32_t* idx_out, a3_stream stream);

/* One decoder layer for the carried rows (Eq. 5; Eq. 4 at the selection layer; the whole block
 * when the rows are all of 0..n-1): RMSNorm, QKV (+bias), RoPE of q and k at pos, k/v written to
 * cache rows pos BEFORE the attention, causal attention over slots 0..pos[m], output projection +
 * residual, RMSNorm, SwiGLU MLP + residual.  x_rows: dev [M][d_model], in/out.  pos: dev [M],
 * strictly ascending, < kv_len.  k_layer/v_layer: this layer's cache, dev [kv_len][Hkv][D].
 * lse_out: dev [M][Hq] or NULL. */
int a3_recompute_layer(const a3_handle* h, int layer, void* x_rows, const int32_t* pos, int M, void* k_layer,
                       void* v_layer, int kv_len, float* lse_out, void* ws, size_t ws_bytes, a3_stream stream);

/* Scatter (Eq. 5, K'_cat[Re,Q] <- ..., V_cat[Re,Q] <- ...): cache row slots[m] = row m.
 * k_rows/v_rows: dev [M][Hkv][D]; slots: dev [M], each in [0, kv_len). */
int a3_scatter_kv(const a3_handle* h, const void* k_rows, const void* v_rows, const int32_t* slots, int M,
                  void* k_layer, void* v_layer, int kv_len, a3_stream stream);

/* The gate/up half of the feed-forward network (the MLP inside H(.) of Eq. 5) of one layer alone:
 * out[M][d_ff] = silu(x Wg^T) * (x Wu^T) rounded to bf16, x: dev [M][d_model].  One launch; used to compare the
 * kernel variants of this GEMM with one another (a3_set_option) and with the oracle. */
int a3_swiglu_rows(const a3_handle* h, int layer, const void* x, void* out, int M, a3_stream stream);

/* Row gather X[R] (Eq. 4, Q_true[Re, Q]): dst[m] = src[rows[m]], rows of `width` bf16 elements. */
int a3_gather_rows(const a3_handle* h, const void* src, int n_src, const int32_t* rows, int M, int width,
                   void* dst, a3_stream stream);

/* The whole request (Method, "Attention-Aware Accurate Fusion"): position recovery of all layers,
 * the leading full blocks 0..select_layer-1 over all n rows, true K/V of all rows and question
 * queries at select_layer, scores, selection, then layers select_layer..L-1 on rows R only.
 * (Position recovery is queued for layers above select_layer only: the layers below it and the
 * selection layer itself get true K/V for every row, so recovered values there would never be read.)
 * Fills the fused cache in place, rows_out, scores_out, x_out. */
int a3_fuse_request(const a3_handle* h, const a3_request* req, void* ws, size_t ws_bytes, a3_stream stream);

/* The same request as a CUDA graph (the request allocates nothing and never synchronises, so it can be captured).
 * a3_graph_capture runs the request once on `stream` (first launches set kernel attributes, which a capture must not
 * see), then records it a second time into a graph and instantiates it; `stream` must not be the legacy default
 * stream and must have nothing else captured on it; profiling (a3_profile_enable) must be off.  The graph holds the
 * pointers of req, ws and the handle's weights: they must stay valid and unchanged in place until a3_graph_destroy;
 * their CONTENTS (chunk caches, x0) may change between launches.  a3_graph_launch replays every kernel of the request
 * on `stream` (asynchronous, no allocation); results land where a3_fuse_request would have put them.
 * Errors: A3_EINVAL (null argument, default stream, profiling on), the request's own status, A3_ECUDA. */
typedef struct a3_graph a3_graph;
int a3_graph_capture(const a3_handle* h, const a3_request* req, void* ws, size_t ws_bytes, a3_stream stream,
                     a3_graph** out);
int a3_graph_launch(const a3_graph* g, a3_stream stream);
/* Kernel launches one replay stands for (what a3_launch_count advances by per a3_graph_launch). */
int a3_graph_kernel_count(const a3_graph* g);
void a3_graph_destroy(a3_graph* g);

/* Precomputation (Eq. 1, K_i, V_i = LLM(i)): prefills one chunk alone at local positions 0..T-1, i.e. runs every
 * layer over all T rows, and leaves the chunk's per-layer caches in k_chunk / v_chunk (dev [n_layers][T][Hkv][D],
 * layer l at + l*layer_stride bytes).  x_chunk: dev [T][d_model], embeddings in, final hidden state out.
 * Called on the whole input X it is the full prefill without reuse.  ws >= a3_request_workspace_bytes(T). */
int a3_precompute_chunk(const a3_handle* h, void* x_chunk, int T, void* k_chunk, void* v_chunk, uint64_t layer_stride,
                        void* ws, size_t ws_bytes, a3_stream stream);

/* Several independent requests on one stream (batched serving). */
int a3_fuse_batch(const a3_handle* h, const a3_request* reqs, int n_requests, void* ws, size_t ws_bytes,
                  a3_stream stream);

/* a3_fuse_request with the chunk caches and embeddings in HOST memory (pinned memory lets the copies
 * overlap the compute): copies them to `staging` (dev, a3_host_staging_bytes) on a copy stream the
 * handle creates on first use, layer by layer, while `stream` computes; builds the chunk descriptors,
 * fuses, copies rows_out and x_out back to the host and waits for both streams - also when it returns an
 * error after the first copy was queued, so the host buffers and the staging area are free on return whatever
 * the status.  Chunk caches of layers up to select_layer are not copied: those layers are recomputed for every
 * row.  req->chunks, req->x0 are ignored (taken from io); the fused cache and scores stay on the device.
 * The handle keeps a host copy of the chunk descriptors, grown (realloc) only when a call has more chunks than
 * any before it. */
int a3_fuse_request_host(const a3_handle* h, const a3_request* req, const a3_host_io* io, void* staging,
                         size_t staging_bytes, void* ws, size_t ws_bytes, a3_stream stream);

/* ---- diagnostics -------------------------------------------------------------------- */

/* `ex`, the eviction extension (Extension subsection), for one layer: keep the system prompt slots [0, n_system)
 * and the question slots [n_ctx, kv_len) whole and, per KV head, the k = a3_evict_count(...) document slots with
 * the largest question-window attention
 *   e[g][i] = sum over question rows j and the query heads h of KV head g of Softmax_row(q_{j,h} K^T / sqrt(D))[i]
 * (SnapKV's vote; summed over g it is Eq. 3's s).  pool (odd, 1 = off) replaces e by its running maximum over
 * `pool` neighbouring candidates before the selection (SnapKV's clustering).  Ties go to the lower slot.
 *   q_window: dev [nq][Hq][D] rotated question queries of this layer; q_pos: dev [nq] their slots (n_ctx..);
 *   lse: dev [nq][Hq] natural-log row log-sum-exps (a3_recompute_layer's lse_out rows of the question);
 *   k_layer, v_layer: dev [kv_len][Hkv][D], kv_len = n_ctx + nq;
 *   k_out, v_out: dev [C'][Hkv][D], C' = n_system + k + nq: entry c of head g is source slot kept_out[g][c];
 *   kept_out: dev [Hkv][C'] int32 (ascending per head) or NULL.
 * ws: a3_evict_workspace_bytes(h, kv_len), borrowed.  Four launches, no allocation, no synchronisation. */
int a3_evict_count(int capacity, int n_system, int n_ctx, int n_question);
size_t a3_evict_workspace_bytes(const a3_handle* h, int kv_len);
int a3_evict_layer(const a3_handle* h, const void* q_window, const int32_t* q_pos, int nq, const float* lse,
                   const void* k_layer, const void* v_layer, int kv_len, int n_system, int n_ctx, int capacity, int pool,
                   void* k_out, void* v_out, int32_t* kept_out, void* ws, size_t ws_bytes, a3_stream stream);

/* First token after fusion (what the paper's time-to-first-token figures end with; Inference paragraph of the
 * Experiments): a = RMSNorm(x_row) * final_norm (rounded to bf16), logits = lm_head a, token = argmax (lowest id
 * on ties).  x_row: dev [d_model] bf16, normally the last row of a3_fuse_request's x_out; final_norm: dev
 * [d_model] bf16; lm_head: dev [vocab][d_model] bf16, 16-byte aligned; logits_out: dev [vocab] fp32 or NULL;
 * token_out: dev int32.  ws: dev, 256-byte aligned, a3_first_token_workspace_bytes(h) bytes, borrowed for the
 * call.  One kernel launch (plus a 4-byte memset), no allocation, no synchronisation.  Non-finite logits set
 * A3_DEV_NONFINITE_SCORE and never win. */
size_t a3_first_token_workspace_bytes(const a3_handle* h);
int a3_first_token(const a3_handle* h, const void* x_row, const void* final_norm, const void* lm_head, int vocab,
                   float* logits_out, int32_t* token_out, void* ws, size_t ws_bytes, a3_stream stream);

/* Waits for `stream`, reads and clears the device status word (A3_DEV_* bits). */
int a3_device_status(const a3_handle* h, uint32_t* bits_out, a3_stream stream);
const char* a3_status_string(int status);
/* cudaError_t of the last failed CUDA call made by this library on the calling thread. */
int a3_last_cuda_error(void);
/* Number of kernel launches this library has queued since the counter was last reset (host counter). */
uint64_t a3_launch_count(int reset);

/* Per-kernel-class device timing with CUDA events recorded on the launching stream around every launch.
 * a3_profile_enable(h, max_records > 0) allocates the event pool (not a hot call) and starts recording;
 * max_records = 0 stops and frees it.  When the pool is full further launches are not recorded.
 * a3_profile_read waits for `stream`, adds up the elapsed time per class and clears the records. */
typedef enum {
  A3_K_REROTATE = 0, A3_K_RMSNORM, A3_K_GEMM_QKV, A3_K_ATTENTION, A3_K_GEMM_RESIDUAL, A3_K_GEMM_SWIGLU,
  A3_K_SCORES, A3_K_TOPK, A3_K_ROWS /* gather, scatter, index kernels */, A3_K_FIRST_TOKEN, A3_K_CLASSES
} a3_kernel_class;
typedef struct { uint64_t launches; double ms; } a3_profile_entry;
int a3_profile_enable(a3_handle* h, int max_records);
int a3_profile_read(a3_handle* h, a3_profile_entry* out /* host [A3_K_CLASSES] */, a3_stream stream);
const char* a3_kernel_class_name(int cls);

#ifdef __cplusplus
}
#endif
#endif /* A3_H_ */

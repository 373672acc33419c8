// Internal declarations shared by the translation units of liba3.so (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "a3.h"

typedef __nv_bfloat16 bf16;

namespace a3 { struct Profiler; }

struct a3_handle {
  a3_model_desc m;
  a3_layer_weights* layers;  // host copy [n_layers]
  float2* rope_tab;          // dev [max_positions][D/2] (cos, sin)
  uint32_t* dev_status;      // dev, 1 word (+ padding)
  int device;
  int sm_count;
  void* tmaps;               // host-side tensor-map cache (a3_gemm.cu)
  a3::Profiler* prof;        // null unless a3_profile_enable is on
  void* host_pipe;           // copy stream + events of a3_fuse_request_host, created on first use
  int opt[A3_OPT_COUNT];     // kernel-variant choices (a3_set_option); defaults set by a3_create
};

namespace a3 {

extern thread_local int g_last_cuda_error;
extern unsigned long long g_launches;

inline int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return A3_ECUDA;
}
#define A3_CUDA(call)                                   \
  do {                                                  \
    cudaError_t e_ = (call);                            \
    if (e_ != cudaSuccess) return ::a3::cuda_fail(e_);  \
  } while (0)

// Call after every kernel launch: counts it and converts a launch error into a status.
inline int launched() {
  ++g_launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  return A3_OK;
}
#define A3_LAUNCHED()                 \
  do {                                \
    int s_ = ::a3::launched();        \
    if (s_ != A3_OK) return s_;       \
  } while (0)
#define A3_TRY(expr)                  \
  do {                                \
    int s_ = (expr);                  \
    if (s_ != A3_OK) return s_;       \
  } while (0)

// Event pair around one launch (only when profiling is enabled on the handle).
struct Profiler {
  cudaEvent_t* ev;
  int* cls;
  int capacity, used;  // in records (two events each)
};
struct ProfScope {
  Profiler* p;
  cudaStream_t st;
  ProfScope(const a3_handle* h, int k, cudaStream_t s) : p(h ? h->prof : nullptr), st(s) {
    if (p && p->used < p->capacity) {
      p->cls[p->used] = k;
      cudaEventRecord(p->ev[2 * p->used], st);
    } else {
      p = nullptr;
    }
  }
  ~ProfScope() {
    if (p) {
      cudaEventRecord(p->ev[2 * p->used + 1], st);
      ++p->used;
    }
  }
};

// Programmatic dependent launch: a kernel launched with launch_pdl may become resident while its predecessor in
// the stream is still running; it must execute pdl_wait() before its first global-memory access (everything before
// that - barrier and tensor-memory set-up, descriptor prefetch - overlaps the predecessor's tail) and it lets its own
// successor do the same with pdl_launch_dependents().  Both instructions are no-ops under an ordinary launch.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// The opt-in to more than 48 KiB of dynamic shared memory is a per-device attribute of a kernel: it is set once per
// device (the handle's, which is current during its calls), not once per process.
struct SmemAttrOnce {
  std::atomic<unsigned long long> devices{0};
};
template <typename F>
inline int smem_attr_once(SmemAttrOnce& once, int device, F func, int bytes) {
  const unsigned long long bit = 1ull << (device & 63);
  if (once.devices.load(std::memory_order_acquire) & bit) return A3_OK;
  A3_CUDA(cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  once.devices.fetch_or(bit, std::memory_order_release);
  return A3_OK;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int cdiv(long long a, long long b) { return (int)((a + b - 1) / b); }

// ---------------------------------------------------------------- internal step launchers

// out[m] = rmsnorm(x[m]) * gain, rows of width d.
int rmsnorm_rows(const a3_handle* h, const bf16* x, const bf16* gain, float eps, int M, int d, bf16* out, cudaStream_t st);

enum GemmEpilogue { EPI_RESIDUAL = 0, EPI_SWIGLU = 1, EPI_QKV = 2 };

struct GemmSegment {
  const bf16* B;     // [n][K] row-major
  const bf16* bias;  // [n] or null
  int n;             // columns of this segment (multiple of 128)
  int kind;          // 0 = q, 1 = k, 2 = v (EPI_QKV only)
};

struct GemmArgs {
  const bf16* A;  // [M][K] row-major
  int M, K;
  GemmSegment seg[3];
  int nseg;
  const bf16* B2;  // EPI_SWIGLU: the "up" matrix, same shape as seg[0].B (gate)
  bf16* C;         // EPI_RESIDUAL: [M][N] in/out (C += A B^T); EPI_SWIGLU: [M][N] out
  int ldc;
  // EPI_QKV
  bf16* q_out;      // [M][Hq*D]
  bf16* k_cache;    // [kv_len][Hkv*D]
  bf16* v_cache;
  const int32_t* pos;  // [M] cache slot = RoPE position of each row
  int kv_len;
};

// SwiGLU GEMM with the weights as the M-side operand of a CTA pair, persistent (a3_swiglu_pair.cu).
bool swiglu_pair_usable(const a3_handle* h, const GemmArgs& a);
int gemm_swiglu_pair(const a3_handle* h, const GemmArgs& a, cudaStream_t st);
// C += A B^T with the same kernel structure (weights on the M side, persistent CTA pairs).
bool residual_t_usable(const a3_handle* h, const GemmArgs& a);
int gemm_residual_t(const a3_handle* h, const GemmArgs& a, cudaStream_t st);
// QKV projection (bias, RoPE, scatter in the epilogue) with one head per CTA of a pair
bool qkv_t_usable(const a3_handle* h, const GemmArgs& a);
int gemm_qkv_t(const a3_handle* h, const GemmArgs& a, cudaStream_t st);

// C-tile GEMM with fused epilogue on the tensor cores; all operands K-major bf16, fp32 accumulate.
int gemm_bf16(const a3_handle* h, GemmEpilogue epi, const GemmArgs& a, cudaStream_t st);

// Causal attention of M rows (at cache slots pos[m]) over a [kv_len][Hkv][D] cache.
// q: [M][Hq][D]; o: [M][Hq][D] (may be null: statistics only); lse: [M][Hq] or null.
// part / part_bytes: optional scratch for partial results when the keys are split across CTAs (attention_part_bytes).
int attention_rows(const a3_handle* h, const bf16* q, const int32_t* pos, int M, const bf16* k, const bf16* v,
                   int kv_len, bf16* o, float* lse, void* part, size_t part_bytes, cudaStream_t st);
size_t attention_part_bytes(const a3_handle* h);
// Statistics-only calls (o == null) split the keys of the few question row tiles over the SMs; the partial row
// statistics of nq rows need at most this much of `part` (a fixed cap, so that every caller - whatever scratch it
// has - arrives at the same split and therefore at bit-identical log-sum-exps).
constexpr size_t STATS_PART_CAP = 768 * 1024;
size_t stats_part_bytes(const a3_handle* h, int nq);
int scores_with_stats(const a3_handle* h, const bf16* q, const int32_t* q_pos, int nq, const bf16* k, int kv_len, int cand_begin,
                      int cand_end, float* lse, void* part, size_t part_bytes, float* scores, cudaStream_t st);

int scores_pass(const a3_handle* h, const bf16* q, const int32_t* q_pos, int nq, const bf16* k, int kv_len,
                int cand_begin, int cand_end, const float* lse, float* scores, cudaStream_t st, float* per_head = nullptr);
// `batches` independent selections, one CTA each: scores + b*score_stride -> idx_out + b*idx_stride
int topk_batched(const a3_handle* h, const float* scores, size_t score_stride, int batches, int cand_begin, int cand_end,
                 int k, int32_t* idx_out, size_t idx_stride, cudaStream_t st);

// scores[slot] = |v_true[slot] - cached value of that slot|^2 for candidate slots covered by a chunk (others untouched)
int value_deviation(const a3_handle* h, const a3_chunk_ref* chunks, int n_chunks, int max_chunk_len, int layer, const bf16* v_true,
                    int cand_begin, int cand_end, float* scores, cudaStream_t st);
int iota_rows(const a3_handle* h, int32_t* out, int begin, int count, cudaStream_t st);
int check_rows(const a3_handle* h, const int32_t* pos, int M, int kv_len, cudaStream_t st);

}  // namespace a3

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__
namespace a3 {

__device__ __forceinline__ float bf2f(bf16 x) { return __bfloat162float(x); }

// 8 bf16 packed in a uint4 <-> 8 floats
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
  uint4 v;
  __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return v;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&t);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool pred) {
  int sz = pred ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

}  // namespace a3
#endif

// a3_query_scores_static: the relevance scores of Eq. 3 for callers that cannot provide a workspace.
//
// Some hosts of this library have no way to allocate device memory at the point where they need the scores: a
// serving engine that handed every free byte of HBM to its KV-cache pool at start-up and never calls the CUDA
// allocator again, or plug-in code running inside a framework that owns the allocator.  a3_query_scores needs
// scratch when the caller does not supply the rows' log-sum-exps: nq * Hq floats for them, and the partial row
// statistics of the pass that computes them with the keys split over the SMs; this variant keeps both in a fixed
// array that is part of the library image instead.
//
// The array lives in every CUDA context that loads the library (A3_STATIC_SCRATCH_BYTES = 1 MiB per GPU: 256 KiB for
// A3_STATIC_LSE_MAX log-sum-exps, 768 KiB for the partial statistics; held until the process exits).  All calls
// share it and it keeps whatever the previous call left there.  Nothing in it has to start at zero: the statistics
// pass overwrites every entry a call uses before the combine and score passes read it.  Two calls whose kernels overlap on the GPU (different streams, or different host threads) race on it;
// callers must order them.
#include <mutex>

#include "a3_internal.cuh"

namespace {

static_assert(A3_STATIC_SCRATCH_BYTES == A3_STATIC_LSE_MAX * 4 + a3::STATS_PART_CAP, "scratch layout");
static __device__ __align__(256) float g_lse_scratch[A3_STATIC_SCRATCH_BYTES / 4];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// In host code `g_lse_scratch` is only a handle for the runtime, not an address a kernel could use: the device
// address is looked up once per device, with that device current, and cached.
int scratch_on_current_device(float** out) {
  int dev = -1;
  A3_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return A3_EUNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    A3_CUDA(cudaGetSymbolAddress((void**)&p, g_lse_scratch));
    if (!p) return A3_ECUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return A3_OK;
}

}  // namespace

using namespace a3;

extern "C" int a3_query_scores_static(const a3_handle* h, const void* q_rows, const int32_t* q_pos, int nq,
                                      const void* k_layer, int kv_len, int cand_begin, int cand_end, float* scores,
                                      a3_stream stream) {
  if (!h || nq < 0 || kv_len < 0 || cand_begin < 0 || cand_end < cand_begin || cand_end > kv_len) return A3_EINVAL;
  if ((long long)nq * h->m.n_q_heads > (long long)A3_STATIC_LSE_MAX) return A3_ETOOLARGE;
  if (kv_len == 0) return A3_OK;
  if (!scores || !k_layer) return A3_EINVAL;
  if (nq > 0 && (!q_rows || !q_pos)) return A3_EINVAL;
  if (((uintptr_t)q_rows | (uintptr_t)k_layer) & 15) return A3_EINVAL;
  if (kv_len > h->m.max_positions) return A3_EINVAL;
  int dev = -1;
  A3_CUDA(cudaGetDevice(&dev));
  if (dev != h->device) return A3_EINVAL;  // the scratch address belongs to the current device
  float* lse = nullptr;
  A3_TRY(scratch_on_current_device(&lse));
  cudaStream_t st = (cudaStream_t)stream;
  A3_TRY(check_rows(h, q_pos, nq, kv_len, st));
  // same split of the statistics pass as a3_query_scores (it depends on the shape alone), hence the same bits
  return scores_with_stats(h, (const bf16*)q_rows, q_pos, nq, (const bf16*)k_layer, kv_len, cand_begin, cand_end, lse,
                           lse + A3_STATIC_LSE_MAX, STATS_PART_CAP, scores, st);
}

// HBM-streaming steps: RoPE table, position recovery (Eq. 2), scatter / gather of rows (Eq. 4, Eq. 5),
// RMSNorm, and the small index kernels.  All bf16 traffic moves as 16-byte vectors, coalesced.
#include "a3_internal.cuh"

namespace a3 {

thread_local int g_last_cuda_error = 0;
unsigned long long g_launches = 0;

// ------------------------------------------------------------------ RoPE table
// tab[p][i] = (cos(p*theta_i), sin(p*theta_i)), theta_i = base^(-2i/D); the angle is formed in float64
// (an fp32 product p*theta_i is off by 1e-3 rad at positions of a few 10^4).
__global__ void rope_table_kernel(float2* tab, int max_pos, int half, double base, int D) {
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)max_pos * half) return;
  int p = (int)(idx / half), i = (int)(idx % half);
  double theta = pow(base, -2.0 * (double)i / (double)D);
  double s, c;
  sincos((double)p * theta, &s, &c);
  tab[idx] = make_float2((float)c, (float)s);
}

int build_rope_table(float2* tab, int max_pos, int D, double base, cudaStream_t st) {
  long long total = (long long)max_pos * (D / 2);
  rope_table_kernel<<<cdiv(total, 256), 256, 0, st>>>(tab, max_pos, D / 2, base, D);
  A3_LAUNCHED();
  return A3_OK;
}

// ------------------------------------------------------------------ position recovery (Eq. 2)
// grid: (token tiles of the longest chunk, chunk, layer).  One CTA moves TOK consecutive tokens of one chunk
// and layer: the span is contiguous in the chunk cache and in the fused cache.
constexpr int RR_THREADS = 256;

template <int D, int LAYOUT>
__global__ void __launch_bounds__(RR_THREADS)
rerotate_kernel(const a3_chunk_ref* __restrict__ chunks, char* __restrict__ kf, char* __restrict__ vf,
                unsigned long long layer_stride, int kv_len, int max_chunk_len, int layer_begin, int row_elems, int tok_per_cta,
                const float2* __restrict__ tab, int max_pos, uint32_t* status) {
  const a3_chunk_ref ch = chunks[blockIdx.y];
  const int t0 = blockIdx.x * tok_per_cta;
  if (ch.len < 0 && blockIdx.x == 0 && threadIdx.x == 0) atomicOr(status, A3_DEV_BAD_POSITION);
  if (t0 >= ch.len) return;
  const int l = layer_begin + blockIdx.z;
  const int nt = min(tok_per_cta, ch.len - t0);
  int ad = ch.delta < 0 ? -ch.delta : ch.delta;
  // with a per-token step the rotation of token t is delta + token_step * t: both ends must be in the table
  const long long a_last = (long long)ch.delta + (long long)ch.token_step * (ch.len - 1);
  // the chunk's slots must lie inside the fused cache and its length inside what the grid was sized for: a chunk that
  // fails either check is skipped as a whole (every CTA of it takes this exit, so nothing of it is written)
  const bool bad = ad >= max_pos || (a_last < 0 ? -a_last : a_last) >= max_pos || ch.dst_offset < 0 ||
                   (long long)ch.dst_offset + ch.len > (long long)kv_len || ch.len > max_chunk_len ||
                   ((uintptr_t)ch.k_src & 15) || ((uintptr_t)ch.v_src & 15) || (ch.src_layer_stride & 15);
  if (bad) {
    if (threadIdx.x == 0) atomicOr(status, A3_DEV_BAD_POSITION);
    return;
  }
  const float sgn = ch.delta < 0 ? -1.f : 1.f;
  const size_t row_bytes = (size_t)row_elems * 2;
  const uint4* ksrc = reinterpret_cast<const uint4*>((const char*)ch.k_src + (size_t)l * ch.src_layer_stride + (size_t)t0 * row_bytes);
  const uint4* vsrc = reinterpret_cast<const uint4*>((const char*)ch.v_src + (size_t)l * ch.src_layer_stride + (size_t)t0 * row_bytes);
  uint4* kdst = reinterpret_cast<uint4*>(kf + (size_t)l * layer_stride + (size_t)(ch.dst_offset + t0) * row_bytes);
  uint4* vdst = reinterpret_cast<uint4*>(vf + (size_t)l * layer_stride + (size_t)(ch.dst_offset + t0) * row_bytes);
  const int nvec = nt * (row_elems / 8);
  const float2* trow = tab + (size_t)ad * (D / 2);

  if (ch.token_step != 0) {
    // Keys stored without positional embedding (or being converted to that form): every token has an angle of
    // its own, so cos/sin come from the table row of the token's rotation instead of living in registers.
    const int vec_per_tok = row_elems / 8;
    if (LAYOUT == 0) {
      constexpr int UPH = D / 16;
      const int nunit = nvec / 2;
      for (int u = threadIdx.x; u < nunit; u += RR_THREADS) {
        const int j = u % UPH;
        const int lo = (u / UPH) * (D / 8) + j;
        const int tok = lo / vec_per_tok;
        const int a = ch.delta + ch.token_step * (t0 + tok);
        const float sg = a < 0 ? -1.f : 1.f;
        const float4* tr = reinterpret_cast<const float4*>(tab + (size_t)(a < 0 ? -a : a) * (D / 2) + 8 * j);
        float fa[8], fb[8], ra[8], rb[8];
        unpack8(__ldcs(ksrc + lo), fa);
        unpack8(__ldcs(ksrc + lo + UPH), fb);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float4 t = __ldg(tr + e);  // (cos, sin) of frequencies 8j+2e and 8j+2e+1
          const float c0 = t.x, s0 = sg * t.y, c1 = t.z, s1 = sg * t.w;
          ra[2 * e] = fa[2 * e] * c0 - fb[2 * e] * s0;
          rb[2 * e] = fa[2 * e] * s0 + fb[2 * e] * c0;
          ra[2 * e + 1] = fa[2 * e + 1] * c1 - fb[2 * e + 1] * s1;
          rb[2 * e + 1] = fa[2 * e + 1] * s1 + fb[2 * e + 1] * c1;
        }
        __stcs(kdst + lo, pack8(ra));
        __stcs(kdst + lo + UPH, pack8(rb));
      }
    } else {
      constexpr int VPH = D / 8;
      for (int v = threadIdx.x; v < nvec; v += RR_THREADS) {
        const int c = v % VPH;
        const int tok = v / vec_per_tok;
        const int a = ch.delta + ch.token_step * (t0 + tok);
        const float sg = a < 0 ? -1.f : 1.f;
        const float4* tr = reinterpret_cast<const float4*>(tab + (size_t)(a < 0 ? -a : a) * (D / 2) + 4 * c);
        float f[8], r[8];
        unpack8(__ldcs(ksrc + v), f);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float4 t = __ldg(tr + e);
          const float c0 = t.x, s0 = sg * t.y, c1 = t.z, s1 = sg * t.w;
          r[4 * e] = f[4 * e] * c0 - f[4 * e + 1] * s0;
          r[4 * e + 1] = f[4 * e] * s0 + f[4 * e + 1] * c0;
          r[4 * e + 2] = f[4 * e + 2] * c1 - f[4 * e + 3] * s1;
          r[4 * e + 3] = f[4 * e + 2] * s1 + f[4 * e + 3] * c1;
        }
        __stcs(kdst + v, pack8(r));
      }
    }
  } else if (LAYOUT == 0) {
    // pairs (i, i + D/2): a unit is the two 16-byte vectors of one head that hold columns [8j,8j+8) and +D/2.
    constexpr int UPH = D / 16;  // units per head
    const int j = threadIdx.x % UPH;  // RR_THREADS is a multiple of UPH, so j is fixed per thread
    float cs[8], sn[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float2 t = __ldg(trow + 8 * j + e);
      cs[e] = t.x;
      sn[e] = sgn * t.y;
    }
    const int nunit = nvec / 2;
    for (int u0 = threadIdx.x; u0 < nunit; u0 += 2 * RR_THREADS) {
      // two units and two value vectors per trip: 6 independent 16-byte loads in flight per thread
      int u1 = u0 + RR_THREADS;
      bool has1 = u1 < nunit;
      int lo0 = (u0 / UPH) * (D / 8) + j, lo1 = (u1 / UPH) * (D / 8) + j;
      uint4 a0 = __ldcs(ksrc + lo0), b0 = __ldcs(ksrc + lo0 + UPH);
      uint4 a1 = make_uint4(0, 0, 0, 0), b1 = a1;
      if (has1) {
        a1 = __ldcs(ksrc + lo1);
        b1 = __ldcs(ksrc + lo1 + UPH);
      }
      float fa[8], fb[8], ra[8], rb[8];
      unpack8(a0, fa);
      unpack8(b0, fb);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        ra[e] = fa[e] * cs[e] - fb[e] * sn[e];
        rb[e] = fa[e] * sn[e] + fb[e] * cs[e];
      }
      __stcs(kdst + lo0, pack8(ra));
      __stcs(kdst + lo0 + UPH, pack8(rb));
      if (has1) {
        unpack8(a1, fa);
        unpack8(b1, fb);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          ra[e] = fa[e] * cs[e] - fb[e] * sn[e];
          rb[e] = fa[e] * sn[e] + fb[e] * cs[e];
        }
        __stcs(kdst + lo1, pack8(ra));
        __stcs(kdst + lo1 + UPH, pack8(rb));
      }
    }
  } else {
    // pairs (2i, 2i+1): one vector holds four pairs, frequencies 4c..4c+3 where c = vector index within the head.
    constexpr int VPH = D / 8;
    const int c = threadIdx.x % VPH;
    float cs[4], sn[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float2 t = __ldg(trow + 4 * c + e);
      cs[e] = t.x;
      sn[e] = sgn * t.y;
    }
    for (int v = threadIdx.x; v < nvec; v += RR_THREADS) {
      float f[8], r[8];
      unpack8(__ldcs(ksrc + v), f);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        r[2 * e] = f[2 * e] * cs[e] - f[2 * e + 1] * sn[e];
        r[2 * e + 1] = f[2 * e] * sn[e] + f[2 * e + 1] * cs[e];
      }
      __stcs(kdst + v, pack8(r));
    }
  }
  // V is copied unchanged.
  for (int v = threadIdx.x; v < nvec; v += 4 * RR_THREADS) {
    uint4 x[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (v + e * RR_THREADS < nvec) x[e] = __ldcs(vsrc + v + e * RR_THREADS);
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (v + e * RR_THREADS < nvec) __stcs(vdst + v + e * RR_THREADS, x[e]);
  }
}

}  // namespace a3

using namespace a3;

extern "C" int a3_rope_rerotate(const a3_handle* h, const a3_chunk_ref* chunks, int n_chunks, int max_chunk_len,
                                void* k_fused, void* v_fused, uint64_t layer_stride, int kv_len, int layer_begin, int layer_end,
                                a3_stream stream) {
  if (!h || !chunks || !k_fused || !v_fused) return A3_EINVAL;
  if (n_chunks < 0 || max_chunk_len < 0 || kv_len < 0 || layer_begin < 0 || layer_end > h->m.n_layers || layer_begin > layer_end) return A3_EINVAL;
  if (((uintptr_t)k_fused & 15) || ((uintptr_t)v_fused & 15) || (layer_stride & 15)) return A3_EINVAL;
  if ((uint64_t)kv_len * h->m.n_kv_heads * h->m.head_dim * 2 > layer_stride) return A3_EINVAL;  // kv_len rows must fit in a layer
  if (n_chunks == 0 || max_chunk_len == 0 || layer_begin == layer_end) return A3_OK;
  if (n_chunks > 65535 || layer_end - layer_begin > 65535) return A3_EUNSUPPORTED;
  const int row_elems = h->m.n_kv_heads * h->m.head_dim;
  // 16 KiB of K and 16 KiB of V per CTA
  int tok = (int)((16 * 1024) / (row_elems * 2));
  if (tok < 1) tok = 1;
  dim3 grid(cdiv(max_chunk_len, tok), n_chunks, layer_end - layer_begin);
  cudaStream_t st = (cudaStream_t)stream;
#define RR_LAUNCH(DD, LL)                                                                                             \
  rerotate_kernel<DD, LL><<<grid, RR_THREADS, 0, st>>>(chunks, (char*)k_fused, (char*)v_fused, layer_stride, kv_len,  \
                                                       max_chunk_len, layer_begin, row_elems, tok, h->rope_tab,      \
                                                       h->m.max_positions, h->dev_status)
  ProfScope prof(h, A3_K_REROTATE, st);
  if (h->m.head_dim == 128 && h->m.rope_layout == 0) RR_LAUNCH(128, 0);
  else if (h->m.head_dim == 128) RR_LAUNCH(128, 1);
  else if (h->m.head_dim == 64 && h->m.rope_layout == 0) RR_LAUNCH(64, 0);
  else RR_LAUNCH(64, 1);
#undef RR_LAUNCH
  A3_LAUNCHED();
  return A3_OK;
}

// ------------------------------------------------------------------ value deviation (comparison selector)
namespace a3 {

// scores[o_c + t] = sum over KV heads and channels of (v_true[o_c + t] - v_cached_c[t])^2 for candidate slots.
// grid: (token tiles of the longest chunk, chunk); one warp per token, 16-byte loads, fp32 accumulation in a
// fixed order (lane-strided partial sums, then a shuffle tree): deterministic.
__global__ void __launch_bounds__(256)
value_deviation_kernel(const a3_chunk_ref* __restrict__ chunks, int layer, const uint4* __restrict__ v_true, int row_vecs, int cand_begin,
                       int cand_end, float* __restrict__ scores) {
  const a3_chunk_ref ch = chunks[blockIdx.y];
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= ch.len) return;
  const int slot = ch.dst_offset + t;
  if (slot < cand_begin || slot >= cand_end) return;
  const int lane = threadIdx.x & 31;
  const uint4* a = v_true + (size_t)slot * row_vecs;
  const uint4* b = reinterpret_cast<const uint4*>((const char*)ch.v_src + (size_t)layer * ch.src_layer_stride) + (size_t)t * row_vecs;
  float acc = 0.f;
  for (int v = lane; v < row_vecs; v += 32) {
    float fa[8], fb[8];
    unpack8(__ldg(a + v), fa);
    unpack8(__ldcs(b + v), fb);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float d = fa[e] - fb[e];
      acc = fmaf(d, d, acc);
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) scores[slot] = acc;
}

int value_deviation(const a3_handle* h, const a3_chunk_ref* chunks, int n_chunks, int max_chunk_len, int layer, const bf16* v_true,
                    int cand_begin, int cand_end, float* scores, cudaStream_t st) {
  if (n_chunks <= 0 || max_chunk_len <= 0) return A3_OK;
  if (n_chunks > 65535) return A3_EUNSUPPORTED;
  ProfScope prof(h, A3_K_SCORES, st);
  value_deviation_kernel<<<dim3(cdiv(max_chunk_len, 8), n_chunks), 256, 0, st>>>(chunks, layer, (const uint4*)v_true,
                                                                                 h->m.n_kv_heads * h->m.head_dim / 8, cand_begin, cand_end, scores);
  A3_LAUNCHED();
  return A3_OK;
}

}  // namespace a3

// ------------------------------------------------------------------ scatter / gather
namespace a3 {

__global__ void __launch_bounds__(256)
scatter_kv_kernel(const uint4* __restrict__ k_rows, const uint4* __restrict__ v_rows, const int32_t* __restrict__ slots,
                  int M, int row_vecs, uint4* __restrict__ kc, uint4* __restrict__ vc, int kv_len, uint32_t* status) {
  // one warp-group of row_vecs lanes per row; several rows per CTA
  const int rows_per_cta = max(1, 256 / row_vecs);
  const int lane_vecs = min(row_vecs, 256);
  const int r = blockIdx.x * rows_per_cta + threadIdx.x / lane_vecs;
  if (threadIdx.x / lane_vecs >= rows_per_cta || r >= M) return;
  const int slot = slots[r];
  if (slot < 0 || slot >= kv_len) {
    if (threadIdx.x % lane_vecs == 0) atomicOr(status, A3_DEV_BAD_POSITION);
    return;
  }
  for (int v = threadIdx.x % lane_vecs; v < row_vecs; v += lane_vecs) {
    uint4 a = __ldcs(k_rows + (size_t)r * row_vecs + v);
    uint4 b = __ldcs(v_rows + (size_t)r * row_vecs + v);
    kc[(size_t)slot * row_vecs + v] = a;
    vc[(size_t)slot * row_vecs + v] = b;
  }
}

__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ src, int n_src, const int32_t* __restrict__ rows, int M, int row_vecs,
                   uint4* __restrict__ dst, uint32_t* status) {
  const int r = blockIdx.x;
  const int s = rows[r];
  if (s < 0 || s >= n_src) {
    if (threadIdx.x == 0) atomicOr(status, A3_DEV_BAD_POSITION);
    return;
  }
  for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) dst[(size_t)r * row_vecs + v] = __ldg(src + (size_t)s * row_vecs + v);
}

__global__ void iota_kernel(int32_t* out, int begin, int count) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) out[i] = begin + i;
}

__global__ void check_rows_kernel(const int32_t* pos, int M, int kv_len, uint32_t* status) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  int p = pos[i];
  if (p < 0 || p >= kv_len) atomicOr(status, A3_DEV_BAD_POSITION);
  if (i > 0 && pos[i - 1] >= p) atomicOr(status, A3_DEV_UNSORTED_ROWS);
}

int iota_rows(const a3_handle* h, int32_t* out, int begin, int count, cudaStream_t st) {
  if (count <= 0) return A3_OK;
  ProfScope prof(h, A3_K_ROWS, st);
  iota_kernel<<<cdiv(count, 256), 256, 0, st>>>(out, begin, count);
  A3_LAUNCHED();
  return A3_OK;
}

int check_rows(const a3_handle* h, const int32_t* pos, int M, int kv_len, cudaStream_t st) {
  if (M <= 0) return A3_OK;
  ProfScope prof(h, A3_K_ROWS, st);
  check_rows_kernel<<<cdiv(M, 256), 256, 0, st>>>(pos, M, kv_len, h->dev_status);
  A3_LAUNCHED();
  return A3_OK;
}

// ------------------------------------------------------------------ RMSNorm
// One CTA per row; the row is read once into registers (16-byte vectors), fp32 sum of squares by shuffles and one
// shared-memory exchange, out = x * rsqrt(mean(x^2) + eps) * gain rounded once to bf16.  Rows wider than
// RN_THREADS * RN_VPT vectors fall back to a second read of the tail.
constexpr int RN_THREADS = 128, RN_VPT = 4;
__global__ void __launch_bounds__(RN_THREADS)
rmsnorm_kernel(const uint4* __restrict__ x, const uint4* __restrict__ gain, float eps, int row_vecs, uint4* __restrict__ out) {
  pdl_wait();
  pdl_launch_dependents();
  const uint4* xr = x + (size_t)blockIdx.x * row_vecs;
  uint4 v[RN_VPT];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < RN_VPT; ++i) {
    const int idx = threadIdx.x + i * RN_THREADS;
    v[i] = idx < row_vecs ? __ldg(xr + idx) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int i = 0; i < RN_VPT; ++i) {
    float f[8];
    unpack8(v[i], f);
#pragma unroll
    for (int e = 0; e < 8; ++e) ss += f[e] * f[e];
  }
  for (int idx = threadIdx.x + RN_VPT * RN_THREADS; idx < row_vecs; idx += RN_THREADS) {
    float f[8];
    unpack8(__ldg(xr + idx), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) ss += f[e] * f[e];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  __shared__ float part[RN_THREADS / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < RN_THREADS / 32; ++w) tot += part[w];
  const float inv = rsqrtf(tot / (float)(row_vecs * 8) + eps);
  uint4* orow = out + (size_t)blockIdx.x * row_vecs;
#pragma unroll
  for (int i = 0; i < RN_VPT; ++i) {
    const int idx = threadIdx.x + i * RN_THREADS;
    if (idx < row_vecs) {
      float f[8], g[8], r[8];
      unpack8(v[i], f);
      unpack8(__ldg(gain + idx), g);
#pragma unroll
      for (int e = 0; e < 8; ++e) r[e] = f[e] * inv * g[e];
      orow[idx] = pack8(r);
    }
  }
  for (int idx = threadIdx.x + RN_VPT * RN_THREADS; idx < row_vecs; idx += RN_THREADS) {
    float f[8], g[8], r[8];
    unpack8(__ldg(xr + idx), f);
    unpack8(__ldg(gain + idx), g);
#pragma unroll
    for (int e = 0; e < 8; ++e) r[e] = f[e] * inv * g[e];
    orow[idx] = pack8(r);
  }
}

int rmsnorm_rows(const a3_handle* h, const bf16* x, const bf16* gain, float eps, int M, int d, bf16* out, cudaStream_t st) {
  if (M <= 0) return A3_OK;
  ProfScope prof(h, A3_K_RMSNORM, st);
  A3_CUDA(launch_pdl(rmsnorm_kernel, dim3(M), dim3(RN_THREADS), 0, st, (const uint4*)x, (const uint4*)gain, eps, d / 8, (uint4*)out));
  A3_LAUNCHED();
  return A3_OK;
}

}  // namespace a3

extern "C" int a3_scatter_kv(const a3_handle* h, const void* k_rows, const void* v_rows, const int32_t* slots, int M,
                             void* k_layer, void* v_layer, int kv_len, a3_stream stream) {
  if (!h || M < 0 || kv_len < 0) return A3_EINVAL;
  if (M == 0) return A3_OK;
  if (!k_rows || !v_rows || !slots || !k_layer || !v_layer) return A3_EINVAL;
  if (((uintptr_t)k_rows | (uintptr_t)v_rows | (uintptr_t)k_layer | (uintptr_t)v_layer) & 15) return A3_EINVAL;
  const int row_vecs = h->m.n_kv_heads * h->m.head_dim / 8;
  const int rows_per_cta = row_vecs >= 256 ? 1 : 256 / row_vecs;
  ProfScope prof(h, A3_K_ROWS, (cudaStream_t)stream);
  scatter_kv_kernel<<<cdiv(M, rows_per_cta), 256, 0, (cudaStream_t)stream>>>(
      (const uint4*)k_rows, (const uint4*)v_rows, slots, M, row_vecs, (uint4*)k_layer, (uint4*)v_layer, kv_len, h->dev_status);
  A3_LAUNCHED();
  return A3_OK;
}

extern "C" int a3_gather_rows(const a3_handle* h, const void* src, int n_src, const int32_t* rows, int M, int width,
                              void* dst, a3_stream stream) {
  if (!h || M < 0 || n_src < 0 || width <= 0 || (width % 8)) return A3_EINVAL;
  if (M == 0) return A3_OK;
  if (!src || !rows || !dst) return A3_EINVAL;
  if (((uintptr_t)src | (uintptr_t)dst) & 15) return A3_EINVAL;
  ProfScope prof(h, A3_K_ROWS, (cudaStream_t)stream);
  gather_rows_kernel<<<M, 256, 0, (cudaStream_t)stream>>>((const uint4*)src, n_src, rows, M, width / 8, (uint4*)dst, h->dev_status);
  A3_LAUNCHED();
  return A3_OK;
}

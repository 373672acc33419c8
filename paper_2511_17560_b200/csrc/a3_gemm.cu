// Projection / MLP GEMMs of the recompute path (Eq. 5: Q_l = X_l W^q, K <- X_l W^k, V <- X_l W^v; H(.)):
//   C[M][N] = A[M][K] * B[N][K]^T, bf16 operands (both K-major), fp32 accumulation, fused epilogues:
//   EPI_RESIDUAL  C <- C + A B^T                       (output projection and MLP down projection)
//   EPI_SWIGLU    C <- silu(A Bg^T) * (A Bu^T)         (gate and up in one pass, 64 + 64 columns per tile)
//   EPI_QKV       +bias, RoPE of q/k at pos[m], q -> q_out, k/v -> cache rows pos[m] (the scatter of Eq. 5)
// This translation unit is the mma.sync (warp-level tensor core) implementation: 128x128x64 tiles,
// 3-stage cp.async pipeline, ldmatrix from 128-byte-swizzled shared memory.
#include "a3_internal.cuh"

namespace a3 {

constexpr int BM = 128, BN = 128, BK = 64, STAGES = 3, GEMM_THREADS = 256;
constexpr int STAGE_BYTES = (BM + BN) * BK * 2;        // 32 KiB
constexpr int CT_LD = BN + 4;                          // fp32 staging tile leading dimension
constexpr int GEMM_SMEM = STAGES * STAGE_BYTES;        // 96 KiB >= 128*132*4 = 66 KiB staging

struct GemmDev {
  const bf16* A;
  int M, K;
  const bf16* B[3];
  const bf16* bias[3];
  int seg_tiles_end[3];  // exclusive tile index where each segment ends (tiles of 128 columns)
  int kind[3];
  const bf16* B2;
  bf16* C;
  int ldc;
  bf16* q_out;
  bf16* k_cache;
  bf16* v_cache;
  const int32_t* pos;
  int kv_len;
  int Hq, Hkv, D, layout, max_pos;
  const float2* tab;
  uint32_t* status;
};

// byte offset of 16-byte chunk `c` of row `r` in a [rows][64] bf16 tile with the 128-byte XOR swizzle
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS)
gemm_mma_kernel(const GemmDev p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp >> 2, wn = warp & 3;  // 2 x 4 warps, warp tile 64 x 32
  const int m0 = blockIdx.x * BM;
  const int nt = blockIdx.y;

  // which B rows feed this tile
  int seg = 0, seg_tile0 = 0;
  if (EPI == EPI_QKV) {
    while (seg < 2 && nt >= p.seg_tiles_end[seg]) {
      seg_tile0 = p.seg_tiles_end[seg];
      ++seg;
    }
  }
  const bf16* Bbase = p.B[seg];
  const int nb0 = (EPI == EPI_SWIGLU) ? nt * 64 : (nt - seg_tile0) * BN;  // first B row (column of the segment)

  const uint32_t smem_base = smem_u32(smem);
  const int KT = p.K / BK;

  auto load_stage = [&](int stage, int kt) {
    const uint32_t sa = smem_base + stage * STAGE_BYTES;
    const uint32_t sb = sa + BM * BK * 2;
    const int k0 = kt * BK;
#pragma unroll
    for (int i = 0; i < (BM * 8) / GEMM_THREADS; ++i) {
      int idx = tid + i * GEMM_THREADS;
      int r = idx >> 3, c = idx & 7;
      int gr = m0 + r;
      bool ok = gr < p.M;
      const bf16* src = p.A + (size_t)(ok ? gr : 0) * p.K + k0 + c * 8;
      cp_async16(sa + swz(r, c), src, ok);
    }
#pragma unroll
    for (int i = 0; i < (BN * 8) / GEMM_THREADS; ++i) {
      int idx = tid + i * GEMM_THREADS;
      int r = idx >> 3, c = idx & 7;
      const bf16* src;
      if (EPI == EPI_SWIGLU)
        src = (r < 64 ? Bbase + (size_t)(nb0 + r) * p.K : p.B2 + (size_t)(nb0 + r - 64) * p.K) + k0 + c * 8;
      else
        src = Bbase + (size_t)(nb0 + r) * p.K + k0 + c * 8;
      cp_async16(sb + swz(r, c), src, true);
    }
  };

  float acc[4][4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < KT) load_stage(s, s);
    cp_async_commit();
  }

  for (int kt = 0; kt < KT; ++kt) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    {
      int nk = kt + STAGES - 1;
      if (nk < KT) load_stage(nk % STAGES, nk);
      cp_async_commit();
    }
    const uint32_t sa = smem_base + (kt % STAGES) * STAGE_BYTES;
    const uint32_t sb = sa + BM * BK * 2;
#pragma unroll
    for (int ks = 0; ks < BK / 16; ++ks) {
      uint32_t af[4][4], bfr[4][2];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int r = wm * 64 + i * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        int c = ks * 2 + (lane >> 4);
        ldmatrix_x4(sa + swz(r, c), af[i][0], af[i][1], af[i][2], af[i][3]);
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        int r = wn * 32 + j * 16 + (lane & 7) + (lane >> 4) * 8;
        int c = ks * 2 + ((lane >> 3) & 1);
        ldmatrix_x4(sb + swz(r, c), bfr[2 * j][0], bfr[2 * j][1], bfr[2 * j + 1][0], bfr[2 * j + 1][1]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) mma_bf16(acc[i][j], af[i], bfr[j][0], bfr[j][1]);
    }
  }
  cp_async_wait<0>();
  __syncthreads();

  // ---- stage the fp32 tile in shared memory
  float* ct = reinterpret_cast<float*>(smem);
  {
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int r = wm * 64 + i * 16 + g, c = wn * 32 + j * 8 + 2 * t;
        *reinterpret_cast<float2*>(&ct[r * CT_LD + c]) = make_float2(acc[i][j][0], acc[i][j][1]);
        *reinterpret_cast<float2*>(&ct[(r + 8) * CT_LD + c]) = make_float2(acc[i][j][2], acc[i][j][3]);
      }
  }
  __syncthreads();

  if (EPI == EPI_RESIDUAL) {
    const int n0 = nt * BN;
    for (int idx = tid; idx < BM * 16; idx += GEMM_THREADS) {
      int r = idx >> 4, v = idx & 15;
      int gr = m0 + r;
      if (gr >= p.M) continue;
      uint4* cp = reinterpret_cast<uint4*>(p.C + (size_t)gr * p.ldc + n0 + v * 8);
      float f[8];
      unpack8(*cp, f);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] += ct[r * CT_LD + v * 8 + e];
      *cp = pack8(f);
    }
  } else if (EPI == EPI_SWIGLU) {
    const int n0 = nt * 64;
    for (int idx = tid; idx < BM * 8; idx += GEMM_THREADS) {
      int r = idx >> 3, v = idx & 7;
      int gr = m0 + r;
      if (gr >= p.M) continue;
      float f[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float gte = ct[r * CT_LD + v * 8 + e], up = ct[r * CT_LD + 64 + v * 8 + e];
        f[e] = gte / (1.f + __expf(-gte)) * up;
      }
      *reinterpret_cast<uint4*>(p.C + (size_t)gr * p.ldc + n0 + v * 8) = pack8(f);
    }
  } else {
    const int kind = p.kind[seg];
    const int D = p.D, half = D / 2;
    const bf16* bias = p.bias[seg];
    for (int idx = tid; idx < BM * 8; idx += GEMM_THREADS) {
      int r = idx >> 3, j = idx & 7;
      int gr = m0 + r;
      if (gr >= p.M) continue;
      const int ps = p.pos[gr];
      if (ps < 0 || ps >= p.kv_len || ps >= p.max_pos) {
        if (j == 0) atomicOr(p.status, A3_DEV_BAD_POSITION);
        continue;
      }
      const int upd = D / 16;                          // units per head
      const int lo = (j / upd) * D + (j % upd) * 8;    // tile column of the low vector
      const int hi = lo + half;
      float a[8], b[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        a[e] = ct[r * CT_LD + lo + e];
        b[e] = ct[r * CT_LD + hi + e];
      }
      if (bias) {
        float ba[8], bb[8];
        unpack8(*reinterpret_cast<const uint4*>(bias + nb0 + lo), ba);
        unpack8(*reinterpret_cast<const uint4*>(bias + nb0 + hi), bb);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          a[e] += ba[e];
          b[e] += bb[e];
        }
      }
      if (kind != 2) {
        const float2* trow = p.tab + (size_t)ps * half;
        if (p.layout == 0) {
          const int f0 = lo % D;  // frequency index of element e is f0 + e
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            float2 cs = __ldg(trow + f0 + e);
            float x = a[e], y = b[e];
            a[e] = x * cs.x - y * cs.y;
            b[e] = x * cs.y + y * cs.x;
          }
        } else {
          const int fa = (lo % D) / 2, fb = (hi % D) / 2;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float2 cs = __ldg(trow + fa + e);
            float x = a[2 * e], y = a[2 * e + 1];
            a[2 * e] = x * cs.x - y * cs.y;
            a[2 * e + 1] = x * cs.y + y * cs.x;
            cs = __ldg(trow + fb + e);
            x = b[2 * e];
            y = b[2 * e + 1];
            b[2 * e] = x * cs.x - y * cs.y;
            b[2 * e + 1] = x * cs.y + y * cs.x;
          }
        }
      }
      bf16* dst;
      if (kind == 0) dst = p.q_out + (size_t)gr * (p.Hq * D) + nb0;
      else if (kind == 1) dst = p.k_cache + (size_t)ps * (p.Hkv * D) + nb0;
      else dst = p.v_cache + (size_t)ps * (p.Hkv * D) + nb0;
      *reinterpret_cast<uint4*>(dst + lo) = pack8(a);
      *reinterpret_cast<uint4*>(dst + hi) = pack8(b);
    }
  }
}

static int gemm_bf16_mma(const a3_handle* h, GemmEpilogue epi, const GemmArgs& a, cudaStream_t st) {
  if (a.M <= 0) return A3_OK;
  if (a.K % BK) return A3_EUNSUPPORTED;
  GemmDev p{};
  p.A = a.A;
  p.M = a.M;
  p.K = a.K;
  int tiles = 0;
  for (int s = 0; s < 3; ++s) {
    if (s < a.nseg) {
      if (a.seg[s].n % (epi == EPI_SWIGLU ? 64 : BN)) return A3_EUNSUPPORTED;
      p.B[s] = a.seg[s].B;
      p.bias[s] = a.seg[s].bias;
      p.kind[s] = a.seg[s].kind;
      tiles += a.seg[s].n / (epi == EPI_SWIGLU ? 64 : BN);
    }
    p.seg_tiles_end[s] = tiles;
  }
  p.B2 = a.B2;
  p.C = a.C;
  p.ldc = a.ldc;
  p.q_out = a.q_out;
  p.k_cache = a.k_cache;
  p.v_cache = a.v_cache;
  p.pos = a.pos;
  p.kv_len = a.kv_len;
  p.Hq = h->m.n_q_heads;
  p.Hkv = h->m.n_kv_heads;
  p.D = h->m.head_dim;
  p.layout = h->m.rope_layout;
  p.max_pos = h->m.max_positions;
  p.tab = h->rope_tab;
  p.status = h->dev_status;
  dim3 grid(cdiv(a.M, BM), tiles);
  static bool attr_set = false;
  if (!attr_set) {
    A3_CUDA(cudaFuncSetAttribute(gemm_mma_kernel<EPI_RESIDUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
    A3_CUDA(cudaFuncSetAttribute(gemm_mma_kernel<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
    A3_CUDA(cudaFuncSetAttribute(gemm_mma_kernel<EPI_QKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
    attr_set = true;
  }
  ProfScope prof(h, epi == EPI_RESIDUAL ? A3_K_GEMM_RESIDUAL : epi == EPI_SWIGLU ? A3_K_GEMM_SWIGLU : A3_K_GEMM_QKV, st);
  if (epi == EPI_RESIDUAL) gemm_mma_kernel<EPI_RESIDUAL><<<grid, GEMM_THREADS, GEMM_SMEM, st>>>(p);
  else if (epi == EPI_SWIGLU) gemm_mma_kernel<EPI_SWIGLU><<<grid, GEMM_THREADS, GEMM_SMEM, st>>>(p);
  else gemm_mma_kernel<EPI_QKV><<<grid, GEMM_THREADS, GEMM_SMEM, st>>>(p);
  A3_LAUNCHED();
  return A3_OK;
}

int gemm_bf16_tc(const a3_handle* h, GemmEpilogue epi, const GemmArgs& a, cudaStream_t st);

// 0: tcgen05 kernel (a3_gemm_tc.cu); 1: the warp-level mma.sync kernel above, kept as a cross-check for bring-up
int g_gemm_impl = 0;

int gemm_bf16(const a3_handle* h, GemmEpilogue epi, const GemmArgs& a, cudaStream_t st) {
  return g_gemm_impl == 1 ? gemm_bf16_mma(h, epi, a, st) : gemm_bf16_tc(h, epi, a, st);
}

}  // namespace a3

extern "C" void a3_internal_set_gemm_impl(int impl) { a3::g_gemm_impl = impl; }

// Shared pieces of the tcgen05 attention kernels: tile constants and PTX wrappers (mbarrier with bounded waits, TMA,
// tcgen05 MMA / tensor-memory loads and stores, shared-memory descriptors).
#pragma once
#include <cuda.h>

#include "a3_internal.cuh"

namespace a3 {

constexpr int ATC_BM = 128, ATC_BN = 128;
constexpr unsigned long long ATC_WAIT_NS = 500000000ull;
constexpr float ATC_LOG2E = 1.4426950408889634f, ATC_LN2 = 0.6931471805599453f;

namespace atc {
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > ATC_WAIT_NS) {
      *abort_flag = 1;
      atomicOr(status, A3_DEV_WAIT_EXHAUSTED);
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// same, A operand read from tensor memory (128 lanes x k, two bf16 per 32-bit column)
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void st32(uint32_t taddr, const float* v) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// K-major [rows][64] bf16 sub-tile, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t desc_k_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// MN-major operand stored as [k rows][64 mn elements] sub-tiles (one 128-byte row per k), 128-byte swizzle:
// 8-k-row groups are 1024 bytes apart (SBO), successive 64-element mn atoms `lbo` bytes apart (LBO)
__device__ __forceinline__ uint64_t desc_mn_sw128(uint32_t saddr, uint32_t lbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) | ((uint64_t)(1024u >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// bf16 x bf16 -> fp32, M = 128, A K-major; b_mn = 1 when B is MN-major
__host__ __device__ constexpr uint32_t idesc(int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(ATC_BM >> 4) << 24);
}
// byte offset of element chunk (16 bytes) j of row r inside a [rows][64] bf16 sub-tile with the 128-byte swizzle
__device__ __forceinline__ uint32_t swz(int r, int j) { return (uint32_t)(r * 128 + ((j ^ (r & 7)) << 4)); }
}  // namespace atc

// 2^v for a pair on the FMA pipe: v = n + f with n integer and |f| <= 1/2 (magic-number rounding), 2^f by a cubic
// (2e-4 relative, a tenth of the bf16 step of P), 2^n by an add into the exponent field.  Inputs are clamped to
// [-125, 126]: below, the result is 2^-125, i.e. nothing; above, it is 2^126, which the row sum's overflow guard
// catches like the +inf of ex2.approx (an unclamped exponent would wrap around and could go unnoticed); -inf must
// not be passed (masked logits take ex2.approx).
// The two-row-tile kernel sends every ATC_POLY_EVERY-th pair of exponentials of an unmasked tile this way: with both
// row tiles' softmax running all the time the exponential unit (16 results per clock and SM) paces it (+3 %).  In
// the one-tile kernel the gain was inside the noise of the measurement and the path is not used.
constexpr int ATC_POLY_EVERY = 4;
__device__ __forceinline__ float2 exp2_poly2(float2 v) {
  const float2 vc = make_float2(fminf(fmaxf(v.x, -125.f), 126.f), fminf(fmaxf(v.y, -125.f), 126.f));
  const float2 tt = __fadd2_rn(vc, make_float2(12582912.f, 12582912.f));
  const float2 rr = __fadd2_rn(tt, make_float2(-12582912.f, -12582912.f));
  const float2 ff = __fadd2_rn(vc, make_float2(-rr.x, -rr.y));
  float2 pp = __ffma2_rn(make_float2(0.054848004f, 0.054848004f), ff, make_float2(0.24180661f, 0.24180661f));
  pp = __ffma2_rn(pp, ff, make_float2(0.69324821f, 0.69324821f));
  pp = __ffma2_rn(pp, ff, make_float2(0.99998868f, 0.99998868f));
  return make_float2(__int_as_float(__float_as_int(pp.x) + (__float_as_int(tt.x) << 23)),
                     __int_as_float(__float_as_int(pp.y) + (__float_as_int(tt.y) << 23)));
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// a3_attention_pair.cu: two row tiles per CTA (launches with many row tiles, head dimension 128, output wanted)
int attention_rows_pair(const a3_handle* h, const CUtensorMap& tK, const CUtensorMap& tV, const bf16* q, const int32_t* pos, int M,
                        int kv_len, bf16* o, float* lse, cudaStream_t st);

}  // namespace a3

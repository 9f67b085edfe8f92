// Small device helpers used by every libqknorm kernel: bf16 <-> fp32 on packed
// words, streaming 128-bit loads/stores.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace qknorm {

// A packed word holds two bf16: element 2i in the low half, 2i+1 in the high half.
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// One rounding, to nearest even (cvt.rn.bf16x2.f32); `a` lands in the low half.
__device__ __forceinline__ uint32_t bf_pack(float a, float b) {
  __nv_bfloat162 r = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&r);
}

// Mixed-precision FMA of sm_100 (PTX fma.rn.f32.bf16): d = a*b + c with a, b the
// bf16 halves of packed words and c, d fp32.  The product of two bf16 values is
// exact in fp32, so this rounds exactly like widening first and using an fp32
// FMA, without the two widening instructions per word.
__device__ __forceinline__ void fma_bf16x2_sq(uint32_t x, float& acc_lo, float& acc_hi) {
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "mov.b32 {lo, hi}, %2;\n\t"
      "fma.rn.f32.bf16 %0, lo, lo, %0;\n\t"
      "fma.rn.f32.bf16 %1, hi, hi, %1;\n\t}"
      : "+f"(acc_lo), "+f"(acc_hi)
      : "r"(x));
}
// (x_lo * g_lo, x_hi * g_hi) in fp32, exact; the addend is -0 so that a product of -0 keeps its sign.
__device__ __forceinline__ float2 mul_bf16x2(uint32_t x, uint32_t g) {
  float2 p;
  asm("{\n\t.reg .b16 xl, xh, gl, gh;\n\t"
      "mov.b32 {xl, xh}, %2;\n\t"
      "mov.b32 {gl, gh}, %3;\n\t"
      "fma.rn.f32.bf16 %0, xl, gl, 0f80000000;\n\t"
      "fma.rn.f32.bf16 %1, xh, gh, 0f80000000;\n\t}"
      : "=f"(p.x), "=f"(p.y)
      : "r"(x), "r"(g));
  return p;
}

// Activations are touched once: stream them past the caches.  These are plain
// coherent accesses (never the read-only path), so an output may alias its input.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) { __stcs(p, v); }

// RMS^-1 of Algorithm 1 from the global sum of squares; IEEE divide and sqrt.
__device__ __forceinline__ float rstd_from_sumsq(float sumsq, int h_total, float eps) {
  return 1.0f / sqrtf(sumsq / (float)h_total + eps);
}

}  // namespace qknorm

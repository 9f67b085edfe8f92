// Device helpers used by every libqknorm kernel: the two storage formats of the
// activations (bf16 and FP8-E4M3) as traits, streaming 128-bit loads/stores.
//
// All arithmetic is fp32 (Section IV-C: sums of squares are accumulated in fp32 for
// both storage formats).  Widening is exact for both formats; the result
// (x * gamma) * RMS^-1 is rounded ONCE to the storage format, to nearest even
// (FP8: saturating at +-448).  gamma is bf16 for both.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace qknorm {

// A packed word holds two bf16: element 2i in the low half, 2i+1 in the high half.
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float2 bf_unpack2(uint32_t u) { return make_float2(bf_lo(u), bf_hi(u)); }

// One rounding, to nearest even (cvt.rn.bf16x2.f32); `a` lands in the low half.
__device__ __forceinline__ uint32_t bf_pack(float a, float b) {
  __nv_bfloat162 r = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&r);
}

// Mixed-precision FMA of sm_100 (PTX fma.rn.f32.bf16 / .f16): d = a*b + c with a, b
// 16-bit halves of packed words and c, d fp32.  The product of two bf16 (or two
// fp16 values that came from FP8) is exact in fp32, so this rounds exactly like
// widening first and using an fp32 FMA, without the widening instructions.
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

// Four E4M3 bytes of a word -> two fp16 pairs (exact: every E4M3 value is an fp16 value).
__device__ __forceinline__ void e4m3x4_to_f16x2(uint32_t w, uint32_t& f01, uint32_t& f23) {
  asm("{\n\t.reg .b16 p01, p23;\n\t"
      "mov.b32 {p01, p23}, %2;\n\t"
      "cvt.rn.f16x2.e4m3x2 %0, p01;\n\t"
      "cvt.rn.f16x2.e4m3x2 %1, p23;\n\t}"
      : "=r"(f01), "=r"(f23)
      : "r"(w));
}
__device__ __forceinline__ void fma_f16x2_sq(uint32_t h, float& acc_lo, float& acc_hi) {
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "mov.b32 {lo, hi}, %2;\n\t"
      "fma.rn.f32.f16 %0, lo, lo, %0;\n\t"
      "fma.rn.f32.f16 %1, hi, hi, %1;\n\t}"
      : "+f"(acc_lo), "+f"(acc_hi)
      : "r"(h));
}
// Two fp32 -> two E4M3 bytes in a 16-bit word (`lo` in the low byte); nearest even, saturating.
__device__ __forceinline__ uint32_t e4m3_pack2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return (uint32_t)r;
}

// ---- storage formats --------------------------------------------------------------------------

struct IoBf16 {
  static constexpr int kBytes = 2;       // bytes per element
  static constexpr int kGammaVecs = 1;   // 16-byte bf16 gamma vectors per 16-byte activation chunk
  static constexpr bool kF16Gamma = false;  // no fp16 copy of gamma: bf16 * bf16 has its own mixed FMA
  // adds the squares of the word's elements to two accumulators
  static __device__ __forceinline__ void sumsq_word(uint32_t w, float& a, float& b) { fma_bf16x2_sq(w, a, b); }
  // (x * gamma) * r for one 16-byte chunk; g1 is unused
  static __device__ __forceinline__ uint4 scale_chunk(const uint4& x, const uint4& g0, const uint4&, float2 r2) {
    uint4 o;
    float2 p = __fmul2_rn(mul_bf16x2(x.x, g0.x), r2);
    o.x = bf_pack(p.x, p.y);
    p = __fmul2_rn(mul_bf16x2(x.y, g0.y), r2);
    o.y = bf_pack(p.x, p.y);
    p = __fmul2_rn(mul_bf16x2(x.z, g0.z), r2);
    o.z = bf_pack(p.x, p.y);
    p = __fmul2_rn(mul_bf16x2(x.w, g0.w), r2);
    o.w = bf_pack(p.x, p.y);
    return o;
  }
  static __device__ __forceinline__ uint4 scale_chunk_g16(const uint4& x, const uint4& g0, const uint4& g1, float2 r2) {
    return scale_chunk(x, g0, g1, r2);  // never selected (kF16Gamma is false)
  }
  static __device__ __forceinline__ float load(const void* base, long long i) {
    return __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t*>(base)[i]) << 16);
  }
  static __device__ __forceinline__ void store(void* base, long long i, float v) {
    const __nv_bfloat16 o = __float2bfloat16_rn(v);
    reinterpret_cast<uint16_t*>(base)[i] = *reinterpret_cast<const uint16_t*>(&o);
  }
};

// (x_lo * g_lo, x_hi * g_hi) in fp32 for fp16 pairs; exact when x came from E4M3 (4 significant
// bits) and g from bf16 (8 significant bits).  The addend is -0 so that a product of -0 keeps its sign.
__device__ __forceinline__ float2 mul_f16x2(uint32_t x, uint32_t g) {
  float2 p;
  asm("{\n\t.reg .b16 xl, xh, gl, gh;\n\t"
      "mov.b32 {xl, xh}, %2;\n\t"
      "mov.b32 {gl, gh}, %3;\n\t"
      "fma.rn.f32.f16 %0, xl, gl, 0f80000000;\n\t"
      "fma.rn.f32.f16 %1, xh, gh, 0f80000000;\n\t}"
      : "=f"(p.x), "=f"(p.y)
      : "r"(x), "r"(g));
  return p;
}

// Is this bf16 value exactly an fp16 value?  Zero, or a normal bf16 with exponent in [-17, 15]
// (below -14 it lands on fp16 subnormals, whose spacing 2^-24 still holds 8 significant bits down
// to 2^-17).  Infinities, NaNs and anything else answer no.
__device__ __forceinline__ bool bf16_fits_f16(uint32_t b16) {
  const uint32_t e = (b16 >> 7) & 0xffu, m = b16 & 0x7fu;
  return (e == 0u && m == 0u) || (e >= 127u - 17u && e <= 127u + 15u);
}
__device__ __forceinline__ bool bf16x2_fits_f16(uint32_t w) { return bf16_fits_f16(w & 0xffffu) && bf16_fits_f16(w >> 16); }
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {  // exact when bf16x2_fits_f16(w)
  const __half2 h = __floats2half2_rn(bf_lo(w), bf_hi(w));
  return *reinterpret_cast<const uint32_t*>(&h);
}

struct IoE4m3 {
  static constexpr int kBytes = 1;
  static constexpr int kGammaVecs = 2;   // 16 elements per chunk need 32 bytes of bf16 gamma
  // When every gamma value is also an fp16 value (any realistic norm weight), the kernel keeps an
  // fp16 copy of gamma and forms x * gamma with the fp16 mixed FMA: the product is exact either
  // way, so the result is bit-identical to the bf16-gamma path, at fewer instructions.
  static constexpr bool kF16Gamma = true;
  static __device__ __forceinline__ uint32_t scale_word_g16(uint32_t x, uint32_t g01, uint32_t g23, float2 r2) {
    uint32_t f01, f23;
    e4m3x4_to_f16x2(x, f01, f23);
    const float2 o01 = __fmul2_rn(mul_f16x2(f01, g01), r2);
    const float2 o23 = __fmul2_rn(mul_f16x2(f23, g23), r2);
    return e4m3_pack2(o01.x, o01.y) | (e4m3_pack2(o23.x, o23.y) << 16);
  }
  static __device__ __forceinline__ uint4 scale_chunk_g16(const uint4& x, const uint4& g0, const uint4& g1, float2 r2) {
    uint4 o;
    o.x = scale_word_g16(x.x, g0.x, g0.y, r2);
    o.y = scale_word_g16(x.y, g0.z, g0.w, r2);
    o.z = scale_word_g16(x.z, g1.x, g1.y, r2);
    o.w = scale_word_g16(x.w, g1.z, g1.w, r2);
    return o;
  }
  static __device__ __forceinline__ void sumsq_word(uint32_t w, float& a, float& b) {
    uint32_t f01, f23;
    e4m3x4_to_f16x2(w, f01, f23);
    fma_f16x2_sq(f01, a, b);
    fma_f16x2_sq(f23, a, b);
  }
  // one word of 4 elements with its two gamma words (elements 0,1 and 2,3)
  static __device__ __forceinline__ uint32_t scale_word(uint32_t x, uint32_t g01, uint32_t g23, float2 r2) {
    uint32_t f01, f23;
    e4m3x4_to_f16x2(x, f01, f23);
    const float2 x01 = __half22float2(*reinterpret_cast<const __half2*>(&f01));
    const float2 x23 = __half22float2(*reinterpret_cast<const __half2*>(&f23));
    const float2 o01 = __fmul2_rn(__fmul2_rn(x01, bf_unpack2(g01)), r2);
    const float2 o23 = __fmul2_rn(__fmul2_rn(x23, bf_unpack2(g23)), r2);
    return e4m3_pack2(o01.x, o01.y) | (e4m3_pack2(o23.x, o23.y) << 16);
  }
  static __device__ __forceinline__ uint4 scale_chunk(const uint4& x, const uint4& g0, const uint4& g1, float2 r2) {
    uint4 o;
    o.x = scale_word(x.x, g0.x, g0.y, r2);
    o.y = scale_word(x.y, g0.z, g0.w, r2);
    o.z = scale_word(x.z, g1.x, g1.y, r2);
    o.w = scale_word(x.w, g1.z, g1.w, r2);
    return o;
  }
  static __device__ __forceinline__ float load(const void* base, long long i) {
    const uint32_t b = reinterpret_cast<const uint8_t*>(base)[i];
    uint32_t f01, f23;
    e4m3x4_to_f16x2(b, f01, f23);
    return __half2float(__ushort_as_half((unsigned short)(f01 & 0xffffu)));
  }
  static __device__ __forceinline__ void store(void* base, long long i, float v) {
    reinterpret_cast<uint8_t*>(base)[i] = (uint8_t)(e4m3_pack2(v, 0.f) & 0xffu);
  }
};

// Activations are touched once: stream them past the caches.  These are plain
// coherent accesses (never the read-only path), so an output may alias its input.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) { __stcs(p, v); }

// RMS^-1 of Algorithm 1 from the global sum of squares.
__device__ __forceinline__ float rstd_of(float sumsq, float inv_h_total, float eps) {
  return rsqrtf(fmaf(sumsq, inv_h_total, eps));
}

}  // namespace qknorm

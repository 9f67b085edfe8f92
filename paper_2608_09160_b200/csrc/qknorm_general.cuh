// General kernel: any width, any 2-byte alignment, any slice count.  One CTA
// per (token, tensor) row, element-wise 16-bit accesses, the row is read a
// second time for the scaling pass (from L1/L2).  It is the path for shapes the
// vectorised kernels do not take; it follows Algorithm 1 literally: one block
// reduction per slice (Phase A), the slices' scalars added in ascending order,
// RMS^-1, then (x * gamma) * RMS^-1.
#pragma once
#include "qknorm_device.cuh"
#include "qknorm_params.h"

namespace qknorm {

constexpr int kGeneralThreads = 256;

// Sum over the CTA, returned to every thread; fixed order, no atomics.
__device__ __forceinline__ float block_sum_256(float v, float* red) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < kGeneralThreads / 32; ++w) tot += red[w];
  __syncthreads();  // red is reused by the next call
  return tot;
}

template <class IO>
__global__ void __launch_bounds__(kGeneralThreads) general_kernel(const __grid_constant__ Params P) {
  __shared__ float red[kGeneralThreads / 32];
  const long long items = 2 * P.T;
  for (long long item = blockIdx.x; item < items; item += gridDim.x) {
    const long long t = item >> 1;
    const TensorArgs& A = (item & 1) ? P.k : P.q;
    if (A.d == 0) continue;  // uniform over the CTA
    const int w = A.w;
    // Phase A per slice, combined in ascending slice order
    float total = 0.f;
    for (int s = 0; s < P.S; ++s) {
      const long long row = t * A.ldx;
      float acc = 0.f;
      for (int j = threadIdx.x; j < w; j += kGeneralThreads) {
        const float v = IO::load(A.x[s], row + j);
        acc = fmaf(v, v, acc);
      }
      const float part = block_sum_256(acc, red);
      if (A.partials != nullptr && threadIdx.x == 0) A.partials[(long long)s * P.T + t] = part;
      total += part;
    }
    const float r = rstd_of(total, A.inv_d, P.eps);
    if (A.rstd != nullptr && threadIdx.x == 0) A.rstd[t] = r;
    // Phases B/C
    for (int s = 0; s < P.S; ++s) {
      const long long row = t * A.ldx, orow = t * A.ldy;
      const uint16_t* gm = A.gamma[s];
      for (int j = threadIdx.x; j < w; j += kGeneralThreads) {
        const float v = IO::load(A.x[s], row + j);
        const float gv = __uint_as_float(((uint32_t)gm[j]) << 16);
        IO::store(A.y[s], orow + j, (v * gv) * r);
      }
    }
  }
}

// Vectorised form of the same two passes for rows that satisfy the 16-byte rules but are too wide
// for the register-resident kernels (one tensor beyond 32768 elements): a CTA of 1024 threads per
// (token, tensor) row, 16-byte chunks, the second pass re-reads the row from L2 (a row is at most
// 128 KB and a few hundred CTAs are resident, so the rows in work fit L2 many times over).
constexpr int kWideThreads = 1024;

// The 32 warps are dealt to the slices, 32 / S warps each, so that all slices are summed (and later
// scaled) side by side with one block barrier per row; a slice's scalar is the sum of its warps'
// scalars in warp order, the slices' scalars are added in ascending slice order.
template <class IO>
__global__ void __launch_bounds__(kWideThreads) wide_kernel(const __grid_constant__ Params P) {
  constexpr int GV = IO::kGammaVecs;
  __shared__ float red[kWideThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wps = 32 / P.S;               // warps per slice (S <= 16: at least 2)
  const int s = warp / wps;                // this warp's slice; warps beyond S * wps idle
  const bool active = s < P.S;
  const int first = (warp - s * wps) * 32 + lane;
  const int stride = wps * 32;
  const long long items = 2 * P.T;
  for (long long item = blockIdx.x; item < items; item += gridDim.x) {
    const long long t = item >> 1;
    const TensorArgs& A = (item & 1) ? P.k : P.q;
    if (A.d == 0) continue;  // uniform over the CTA
    const int cw = (A.w * IO::kBytes) >> 4;  // 16-byte chunks per slice row
    const uint4* row = nullptr;
    float a = 0.f, b = 0.f;
    if (active) {
      row = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(A.x[s]) +
                                           (unsigned long long)t * A.ldx * IO::kBytes);
      for (int c = first; c < cw; c += stride) {
        const uint4 v = row[c];  // a plain load: the line should stay in L2 for the second pass
        IO::sumsq_word(v.x, a, b);
        IO::sumsq_word(v.y, a, b);
        IO::sumsq_word(v.z, a, b);
        IO::sumsq_word(v.w, a, b);
      }
    }
    float ws = a + b;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, off);
    if (lane == 0) red[warp] = ws;
    __syncthreads();
    float total = 0.f;
    for (int s2 = 0; s2 < P.S; ++s2) {
      float part = 0.f;
      for (int j = 0; j < wps; ++j) part += red[s2 * wps + j];
      if (A.partials != nullptr && threadIdx.x == 0) A.partials[(long long)s2 * P.T + t] = part;
      total += part;
    }
    __syncthreads();  // red is reused by the next row
    const float r = rstd_of(total, A.inv_d, P.eps);
    if (A.rstd != nullptr && threadIdx.x == 0) A.rstd[t] = r;
    if (active) {
      const float2 r2 = make_float2(r, r);
      uint4* out = reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(A.y[s]) +
                                            (unsigned long long)t * A.ldy * IO::kBytes);
      const uint4* gm = reinterpret_cast<const uint4*>(A.gamma[s]);
      for (int c = first; c < cw; c += stride) {
        const uint4 v = row[c];
        const uint4 ga = __ldg(gm + (size_t)c * GV), gb = __ldg(gm + (size_t)c * GV + GV - 1);
        st_stream(out + c, IO::scale_chunk(v, ga, gb, r2));
      }
    }
  }
}

}  // namespace qknorm

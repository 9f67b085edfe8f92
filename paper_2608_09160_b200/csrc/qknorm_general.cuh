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

}  // namespace qknorm

// One-GPU stand-ins for the two ways of doing tensor-parallel QK-Norm that the
// paper compares against (Sections II-C and IV-A), so that the fused kernels can
// be quoted in the paper's own terms (bytes moved, launches).  They compute the
// same result as qknorm_fwd_sharded and are checked against the same oracle.
//
//  * gather, then norm  -- the standard path: every rank first obtains the FULL
//    Q/K vector (All-Gather), then normalises it.  Here: one kernel copies the S
//    slice buffers side by side into a scratch buffer of full rows, then the
//    ordinary kernels run with that scratch as their input.  Every activation
//    crosses HBM four times instead of twice.
//  * statistic pass, then scale pass -- scalar aggregation without fusion: one
//    kernel writes each slice's sum of squares to a scratch array (the scalars a
//    rank would send), a second kernel adds them in ascending slice order and
//    scales.  Every activation is read twice and written once.
#pragma once
#include "qknorm_device.cuh"
#include "qknorm_params.h"

namespace qknorm {

constexpr int kBaselineThreads = 256;

// ---- gather: slice buffers -> full rows ----------------------------------------------------
// dst row t = [Q slice 0 .. S-1][K slice 0 .. S-1] (row pitch = (dq + dk) * elem bytes).
// VEC: 16-byte copies (slice rows and pointers 16-byte aligned); else byte copies.
template <bool VEC>
__global__ void __launch_bounds__(kBaselineThreads) gather_kernel(const __grid_constant__ Params P, unsigned char* dst) {
  const long long row_bytes = ((long long)P.q.d + P.k.d) * P.elem_bytes;
  const long long unit = VEC ? 16 : 1;
  const long long units_per_row = row_bytes / unit;
  const long long total = P.T * units_per_row;
  const long long q_bytes = (long long)P.q.d * P.elem_bytes;
  for (long long i = (long long)blockIdx.x * kBaselineThreads + threadIdx.x; i < total;
       i += (long long)gridDim.x * kBaselineThreads) {
    const long long t = i / units_per_row;
    long long off = (i - t * units_per_row) * unit;  // byte offset inside the full row
    const bool is_k = off >= q_bytes;
    const TensorArgs& A = is_k ? P.k : P.q;
    if (is_k) off -= q_bytes;
    const long long slice_bytes = (long long)A.w * P.elem_bytes;
    const int s = (int)(off / slice_bytes);
    const long long in_slice = off - (long long)s * slice_bytes;
    const unsigned char* src = reinterpret_cast<const unsigned char*>(A.x[s]) + t * A.ldx * P.elem_bytes + in_slice;
    unsigned char* d = dst + t * row_bytes + (is_k ? q_bytes : 0) + off;
    if (VEC) *reinterpret_cast<uint4*>(d) = ld_stream(reinterpret_cast<const uint4*>(src));
    else *d = *src;
  }
}

// ---- pass 1: every slice's own sum of squares to global memory (Phase A only) ----------------
// One warp per (token, tensor, slice).  scratch layout: [tensor][slice][token] fp32.
template <class IO, bool VEC>
__global__ void __launch_bounds__(kBaselineThreads) stat_kernel(const __grid_constant__ Params P, float* scratch) {
  const int lane = threadIdx.x & 31;
  const long long items = P.T * 2 * P.S;
  const long long warps = (long long)gridDim.x * (kBaselineThreads / 32);
  for (long long it = (long long)blockIdx.x * (kBaselineThreads / 32) + (threadIdx.x >> 5); it < items; it += warps) {
    const long long t = it / (2 * P.S);
    const int r = (int)(it - t * 2 * P.S);
    const int tensor = r / P.S, s = r - tensor * P.S;
    const TensorArgs& A = tensor ? P.k : P.q;
    if (A.d == 0) continue;
    float a = 0.f, b = 0.f;
    if (VEC) {
      const uint4* x = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(A.x[s]) +
                                                      t * A.ldx * IO::kBytes);
      const int chunks = (A.w * IO::kBytes) >> 4;
      for (int c = lane; c < chunks; c += 32) {
        const uint4 v = ld_stream(x + c);
        IO::sumsq_word(v.x, a, b);
        IO::sumsq_word(v.y, a, b);
        IO::sumsq_word(v.z, a, b);
        IO::sumsq_word(v.w, a, b);
      }
    } else {
      for (int j = lane; j < A.w; j += 32) {
        const float v = IO::load(A.x[s], t * A.ldx + j);
        a = fmaf(v, v, a);
      }
    }
    float ss = a + b;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    if (lane == 0) scratch[((long long)tensor * P.S + s) * P.T + t] = ss;
  }
}

// ---- pass 2: add the slices' scalars in ascending order, scale, store (Phases B/C) -------------
template <class IO, bool VEC>
__global__ void __launch_bounds__(kBaselineThreads) scale_kernel(const __grid_constant__ Params P, const float* scratch) {
  const int lane = threadIdx.x & 31;
  const long long items = P.T * 2 * P.S;
  const long long warps = (long long)gridDim.x * (kBaselineThreads / 32);
  for (long long it = (long long)blockIdx.x * (kBaselineThreads / 32) + (threadIdx.x >> 5); it < items; it += warps) {
    const long long t = it / (2 * P.S);
    const int r = (int)(it - t * 2 * P.S);
    const int tensor = r / P.S, s = r - tensor * P.S;
    const TensorArgs& A = tensor ? P.k : P.q;
    if (A.d == 0) continue;
    float total = 0.f;
    for (int s2 = 0; s2 < P.S; ++s2) total += scratch[((long long)tensor * P.S + s2) * P.T + t];
    const float rs = rstd_of(total, A.inv_d, P.eps);
    if (s == 0 && lane == 0 && A.rstd != nullptr) A.rstd[t] = rs;
    if (lane == 0 && A.partials != nullptr) A.partials[(long long)s * P.T + t] = scratch[((long long)tensor * P.S + s) * P.T + t];
    if (VEC) {
      const uint4* x = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(A.x[s]) +
                                                      t * A.ldx * IO::kBytes);
      uint4* y = reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(A.y[s]) + t * A.ldy * IO::kBytes);
      const uint4* g = reinterpret_cast<const uint4*>(A.gamma[s]);
      const int chunks = (A.w * IO::kBytes) >> 4;
      const float2 r2 = make_float2(rs, rs);
      for (int c = lane; c < chunks; c += 32) {
        const uint4 v = ld_stream(x + c);
        const uint4 g0 = __ldg(g + (size_t)c * IO::kGammaVecs);
        const uint4 g1 = __ldg(g + (size_t)c * IO::kGammaVecs + IO::kGammaVecs - 1);
        st_stream(y + c, IO::scale_chunk(v, g0, g1, r2));
      }
    } else {
      for (int j = lane; j < A.w; j += 32) {
        const float v = IO::load(A.x[s], t * A.ldx + j);
        const float gv = __uint_as_float(((uint32_t)A.gamma[s][j]) << 16);
        IO::store(A.y[s], t * A.ldy + j, (v * gv) * rs);
      }
    }
  }
}

}  // namespace qknorm

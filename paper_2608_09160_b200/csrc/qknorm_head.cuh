// Headwise QK-Norm (Section II-A: every attention head has a normalisation factor of its own).
//
// Every head (head_dim consecutive columns of a row) is normalised on its own:
// mean over head_dim, the gamma entries of those columns.  Heads are small
// (head_dim = 128 is 256 bytes), so a head is served by a group of `lph` lanes
// (the power of two >= head_dim/8, one 16-byte chunk per lane) and a warp step
// covers 32/lph consecutive heads: 512 contiguous bytes when head_dim is a power
// of two.  A warp owns a token and walks over its Q heads, then its K heads, U
// steps at a time so that U independent loads per lane are in flight.  The head
// scalar is a log2(lph)-step shuffle tree; there is nothing to combine across
// tensor-parallel shards because a head never straddles a shard.
#pragma once
#include "qknorm_device.cuh"

namespace qknorm {

struct HeadSide {
  const void* x;          // [T, nh*head_dim] bf16, rows ldx bytes apart
  const uint16_t* gamma;  // [nh*head_dim] bf16
  void* y;
  float* rstd;            // optional [T, nh]
  long long ldx, ldy;     // BYTES between consecutive rows
  int nh;                 // heads per row (0 = tensor absent)
};

struct HeadParams {
  HeadSide q, k;
  long long T;
  int head_dim;
  int hc;        // 16-byte chunks per head (vector kernel)
  int log_lph;   // log2 of the lanes per head
  float inv_hd;  // 1 / head_dim
  float eps;
};

constexpr int kHeadThreads = 256;

template <int U>
__global__ void __launch_bounds__(kHeadThreads) head_kernel(const __grid_constant__ HeadParams H) {
  const int lane = threadIdx.x & 31;
  const int lph = 1 << H.log_lph;
  const int hpw = 32 >> H.log_lph;  // heads per warp step
  const int sub = lane >> H.log_lph;
  const int c = lane & (lph - 1);
  const bool cvalid = c < H.hc;
  const long long warps = (long long)gridDim.x * (kHeadThreads / 32);
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  for (long long t = (long long)blockIdx.x * (kHeadThreads / 32) + (threadIdx.x >> 5); t < H.T; t += warps) {
#pragma unroll
    for (int side = 0; side < 2; ++side) {
      const HeadSide& A = side ? H.k : H.q;
      if (A.nh == 0) continue;
      const unsigned char* xrow = reinterpret_cast<const unsigned char*>(A.x) + t * A.ldx;
      unsigned char* yrow = reinterpret_cast<unsigned char*>(A.y) + t * A.ldy;
      const uint4* gam = reinterpret_cast<const uint4*>(A.gamma);
      for (int h0 = 0; h0 < A.nh; h0 += hpw * U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int h = h0 + u * hpw + sub;
          v[u] = (cvalid && h < A.nh) ? ld_stream(reinterpret_cast<const uint4*>(xrow) + (size_t)h * H.hc + c) : zero;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int h = h0 + u * hpw + sub;
          float a = 0.f, b = 0.f;
          IoBf16::sumsq_word(v[u].x, a, b);
          IoBf16::sumsq_word(v[u].y, a, b);
          IoBf16::sumsq_word(v[u].z, a, b);
          IoBf16::sumsq_word(v[u].w, a, b);
          float ss = a + b;
          for (int off = lph >> 1; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
          const float r = rstd_of(ss, H.inv_hd, H.eps);
          if (h < A.nh) {
            if (A.rstd != nullptr && c == 0) A.rstd[t * A.nh + h] = r;
            if (cvalid) {
              const uint4 g = __ldg(gam + (size_t)h * H.hc + c);
              st_stream(reinterpret_cast<uint4*>(yrow) + (size_t)h * H.hc + c,
                        IoBf16::scale_chunk(v[u], g, g, make_float2(r, r)));
            }
          }
        }
      }
    }
  }
}

// Any head_dim, any 2-byte alignment: one warp per head, element-wise, two passes.
__global__ void __launch_bounds__(kHeadThreads) head_general_kernel(const __grid_constant__ HeadParams H) {
  const int lane = threadIdx.x & 31;
  const int nht = H.q.nh + H.k.nh;
  const long long items = H.T * nht;
  const long long warps = (long long)gridDim.x * (kHeadThreads / 32);
  for (long long it = (long long)blockIdx.x * (kHeadThreads / 32) + (threadIdx.x >> 5); it < items; it += warps) {
    const long long t = it / nht;
    const int hh = (int)(it - t * nht);
    const bool is_k = hh >= H.q.nh;
    const HeadSide& A = is_k ? H.k : H.q;
    const int h = is_k ? hh - H.q.nh : hh;
    const uint16_t* x = reinterpret_cast<const uint16_t*>(reinterpret_cast<const unsigned char*>(A.x) + t * A.ldx) +
                        (size_t)h * H.head_dim;
    uint16_t* y = reinterpret_cast<uint16_t*>(reinterpret_cast<unsigned char*>(A.y) + t * A.ldy) + (size_t)h * H.head_dim;
    const uint16_t* gm = A.gamma + (size_t)h * H.head_dim;
    float acc = 0.f;
    for (int j = lane; j < H.head_dim; j += 32) {
      const float v = IoBf16::load(x, j);
      acc = fmaf(v, v, acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    const float r = rstd_of(acc, H.inv_hd, H.eps);
    if (A.rstd != nullptr && lane == 0) A.rstd[t * A.nh + h] = r;
    for (int j = lane; j < H.head_dim; j += 32)
      IoBf16::store(y, j, (IoBf16::load(x, j) * IoBf16::load(gm, j)) * r);
  }
}

}  // namespace qknorm

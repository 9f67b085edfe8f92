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
//
// Column slices: a tensor may come as S slice buffers of nh heads each (what S
// tensor-parallel ranks hold).  The warp then walks the S * nh heads of the token
// as one list and picks the slice's pointers per head, so narrow slices (a K slice
// of one head) still fill whole warp steps.  Both storage formats: a 16-byte chunk
// is 8 bf16 or 16 FP8-E4M3 elements.
#pragma once
#include "qknorm_device.cuh"
#include "qknorm_params.h"

namespace qknorm {

struct HeadSide {
  const void* x[kMaxShards];          // slice s: [T, nh*head_dim] bf16 or FP8-E4M3, rows ldx bytes apart
  const uint16_t* gamma[kMaxShards];  // slice s: [nh*head_dim] bf16
  void* y[kMaxShards];
  float* rstd;            // optional [T, S*nh]: head h of slice s at column s*nh + h
  long long ldx, ldy;     // BYTES between consecutive rows
  int nh;                 // heads per slice row (0 = tensor absent)
  int heads;              // S * nh
  float inv_nh;           // 1 / nh
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

// head index over all slices -> (slice, head inside the slice); exact for the head counts a row can have
__device__ __forceinline__ void head_locate(const HeadSide& A, int h, int& s, int& hl) {
  s = __float2int_rz(((float)h + 0.5f) * A.inv_nh);
  hl = h - s * A.nh;
}

template <int U, class IO>
__global__ void __launch_bounds__(kHeadThreads) head_kernel(const __grid_constant__ HeadParams H) {
  constexpr int GV = IO::kGammaVecs;
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
      if (A.heads == 0) continue;
      for (int h0 = 0; h0 < A.heads; h0 += hpw * U) {
        uint4 v[U];
        int sl[U], hl[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int h = h0 + u * hpw + sub;
          sl[u] = 0;
          hl[u] = h;
          v[u] = zero;
          if (h < A.heads) {
            if (A.heads != A.nh) head_locate(A, h, sl[u], hl[u]);
            if (cvalid) {
              const unsigned char* xrow = reinterpret_cast<const unsigned char*>(A.x[sl[u]]) + t * A.ldx;
              v[u] = ld_stream(reinterpret_cast<const uint4*>(xrow) + (size_t)hl[u] * H.hc + c);
            }
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int h = h0 + u * hpw + sub;
          float a = 0.f, b = 0.f;
          IO::sumsq_word(v[u].x, a, b);
          IO::sumsq_word(v[u].y, a, b);
          IO::sumsq_word(v[u].z, a, b);
          IO::sumsq_word(v[u].w, a, b);
          float ss = a + b;
          for (int off = lph >> 1; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
          const float r = rstd_of(ss, H.inv_hd, H.eps);
          if (h < A.heads) {
            if (A.rstd != nullptr && c == 0) A.rstd[t * A.heads + h] = r;
            if (cvalid) {
              const uint4* gam = reinterpret_cast<const uint4*>(A.gamma[sl[u]]) + ((size_t)hl[u] * H.hc + c) * GV;
              const uint4 g0 = __ldg(gam);
              const uint4 g1 = GV > 1 ? __ldg(gam + 1) : g0;
              unsigned char* yrow = reinterpret_cast<unsigned char*>(A.y[sl[u]]) + t * A.ldy;
              st_stream(reinterpret_cast<uint4*>(yrow) + (size_t)hl[u] * H.hc + c,
                        IO::scale_chunk(v[u], g0, g1, make_float2(r, r)));
            }
          }
        }
      }
    }
  }
}

// Any head_dim, any element alignment: one warp per head, element-wise, two passes.
template <class IO>
__global__ void __launch_bounds__(kHeadThreads) head_general_kernel(const __grid_constant__ HeadParams H) {
  const int lane = threadIdx.x & 31;
  const int nht = H.q.heads + H.k.heads;
  const long long items = H.T * nht;
  const long long warps = (long long)gridDim.x * (kHeadThreads / 32);
  for (long long it = (long long)blockIdx.x * (kHeadThreads / 32) + (threadIdx.x >> 5); it < items; it += warps) {
    const long long t = it / nht;
    const int hh = (int)(it - t * nht);
    const bool is_k = hh >= H.q.heads;
    const HeadSide& A = is_k ? H.k : H.q;
    const int h = is_k ? hh - H.q.heads : hh;
    const int s = h / A.nh, hl = h - s * A.nh;
    const unsigned char* x = reinterpret_cast<const unsigned char*>(A.x[s]) + t * A.ldx + (size_t)hl * H.head_dim * IO::kBytes;
    unsigned char* y = reinterpret_cast<unsigned char*>(A.y[s]) + t * A.ldy + (size_t)hl * H.head_dim * IO::kBytes;
    const uint16_t* gm = A.gamma[s] + (size_t)hl * H.head_dim;
    float acc = 0.f;
    for (int j = lane; j < H.head_dim; j += 32) {
      const float v = IO::load(x, j);
      acc = fmaf(v, v, acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    const float r = rstd_of(acc, H.inv_hd, H.eps);
    if (A.rstd != nullptr && lane == 0) A.rstd[t * A.heads + h] = r;
    for (int j = lane; j < H.head_dim; j += 32) IO::store(y, j, (IO::load(x, j) * IoBf16::load(gm, j)) * r);
  }
}

}  // namespace qknorm

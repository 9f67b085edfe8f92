// Thread layout and per-token arithmetic shared by the vectorised kernels.
//
// Layout.  A CTA serves one token at a time.  Its threads are cut into 2*S
// groups, one per (tensor, slice): first the S slices of Q, G_q threads each,
// then the S slices of K, G_k threads each ("rank" s of Algorithm 1 is the
// pair of groups with slice index s).  Thread g of a group owns the 16-byte
// chunks g, g+G, ..., g+(N-1)G of its slice row (those that exist).  So:
//   * a warp touches consecutive 16-byte chunks of one slice row (coalesced,
//     and conflict-free when the row sits in shared memory),
//   * everything a thread holds belongs to ONE slice of ONE tensor, so its
//     running sum of squares is a piece of that slice's Phase-A scalar S_local,
//   * the thread's gamma chunks are loaded once and kept in registers over the
//     token loop (the W_local multiply of Phase B costs no memory traffic),
//   * narrow K rows (GQA) get proportionally fewer threads instead of idle lanes.
// G_q, G_k are multiples of `sub` (16 or 32 lanes): a lane group never
// straddles two slices, so the slice scalar is a shuffle tree inside the lane
// group plus one shared-memory slot per lane group.
//
// Arithmetic (Algorithm 1): fp32 throughout, two elements per instruction with
// the packed FFMA2/FMUL2 of sm_100; partial sums are combined slot by slot,
// slice by slice in ascending order; RMS^-1 = rsqrt(S_global / H_total + eps);
// y = (x * gamma) * RMS^-1 rounded once to bf16.
//
// The kernels are instruction-issue sensitive (about 1.6e12 elements/s have to
// pass through 148 SMs), so the per-chunk code is kept to a handful of
// instructions: loop-invariant offsets, no per-chunk bounds tests on the loads.
#pragma once
#include "qknorm_device.cuh"
#include "qknorm_params.h"

namespace qknorm {

// Largest CTA the kernels with N chunks per thread are compiled for, and how
// many such CTAs the register budget is shaped for.
__host__ __device__ constexpr int max_threads_for(int n) { return n <= 2 ? 1024 : 512; }
__host__ __device__ constexpr int min_blocks_for(int) { return 1; }

struct LaneMap {
  bool active;        // this thread serves a slice
  bool leader;        // first lane of its lane group (writes the group's slot)
  bool first;         // first thread of its tensor (writes rstd)
  int slice;          // s
  int g;              // index inside the slice's group
  int nvalid;         // how many of the N chunk positions exist for this thread
  float inv_d;        // 1 / H_total of this thread's tensor
  int slot;           // this lane group's slot
  int slot0;          // first slot of this thread's tensor
  int sps;            // slots per slice
  const unsigned char* x;  // slice base pointers
  const uint4* gamma;
  unsigned char* y;
  float* rstd;
  float* partials;
  unsigned long long in_pitch;   // bytes between consecutive rows of the slice's input
  unsigned long long out_pitch;  // and of its output
  uint32_t chunk_off;  // g * 16: byte offset of this thread's first chunk inside its slice row
  uint32_t stride;     // G * 16: byte distance between a thread's consecutive chunks
  uint32_t stage_off;  // byte offset of the first chunk inside a gathered row (Q slices, then K slices)
};

template <class IO>
__device__ __forceinline__ LaneMap make_lane(const Params& P, int tid, int n_chunks_per_thread) {
  LaneMap m;
  const bool is_k = P.k.d != 0 && tid >= P.k.first_thread;
  const TensorArgs& A = is_k ? P.k : P.q;
  const int rel = tid - A.first_thread;
  const int G = A.G > 0 ? A.G : 1;
  const int s = rel / G;
  m.active = A.d != 0 && s < P.S;
  m.slice = m.active ? s : 0;
  m.g = rel - s * G;
  const int chunks = (A.w * IO::kBytes) >> 4;  // 16-byte chunks per slice row
  int nv = m.active && m.g < chunks ? (chunks - m.g + G - 1) / G : 0;
  m.nvalid = nv < n_chunks_per_thread ? nv : n_chunks_per_thread;
  m.inv_d = A.inv_d;
  m.slot = tid >> P.log_sub;
  m.leader = (tid & ((1 << P.log_sub) - 1)) == 0;
  m.first = rel == 0;
  m.slot0 = A.first_thread >> P.log_sub;
  m.sps = G >> P.log_sub;
  m.x = reinterpret_cast<const unsigned char*>(A.x[m.slice]);
  m.gamma = reinterpret_cast<const uint4*>(A.gamma[m.slice]);
  m.y = reinterpret_cast<unsigned char*>(A.y[m.slice]);
  m.rstd = A.rstd;
  m.partials = A.partials;
  m.in_pitch = (unsigned long long)A.ldx * IO::kBytes;
  m.out_pitch = (unsigned long long)A.ldy * IO::kBytes;
  m.chunk_off = (uint32_t)m.g * 16u;
  m.stride = (uint32_t)G * 16u;
  m.stage_off = (is_k ? (uint32_t)P.q.d * IO::kBytes : 0u) + (uint32_t)m.slice * (uint32_t)A.w * IO::kBytes + m.chunk_off;
  return m;
}

// Sum of squares of N chunks (zeros where a chunk is absent): independent accumulators per chunk pair.
template <class IO, int N>
__device__ __forceinline__ float sumsq_chunks(const uint4 (&v)[N]) {
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
  for (int i = 0; i < N; ++i) {
    IO::sumsq_word(v[i].x, a0, a1);
    IO::sumsq_word(v[i].y, a2, a3);
    IO::sumsq_word(v[i].z, a0, a1);
    IO::sumsq_word(v[i].w, a2, a3);
  }
  return (a0 + a2) + (a1 + a3);
}

// Lane-group sum: every lane of a 16- or 32-lane group gets the group's total.
__device__ __forceinline__ float lane_group_sum(float a, int log_sub) {
  if (log_sub == 5) a += __shfl_xor_sync(0xffffffffu, a, 16);
  a += __shfl_xor_sync(0xffffffffu, a, 8);
  a += __shfl_xor_sync(0xffffffffu, a, 4);
  a += __shfl_xor_sync(0xffffffffu, a, 2);
  a += __shfl_xor_sync(0xffffffffu, a, 1);
  return a;
}

// Adds the slots of this thread's tensor: slot by slot inside a slice, then the
// slices' scalars in ascending slice order (the P2P-reduction line of Algorithm 1).
__device__ __forceinline__ float combine_slices(const float* slots, const LaneMap& m, int S) {
  const float* p = slots + m.slot0;
  float total = 0.f;
  if (m.sps == 1) {  // one lane group per slice: the slots ARE the slices' scalars
    for (int s2 = 0; s2 < S; ++s2) total += p[s2];
    return total;
  }
  for (int s2 = 0; s2 < S; ++s2) {
    float part = 0.f;
    for (int j = 0; j < m.sps; ++j) part += p[s2 * m.sps + j];
    total += part;
  }
  return total;
}

// The scalar of the thread's own slice (only needed when the caller asked for partials).
__device__ __forceinline__ float own_slice_scalar(const float* slots, const LaneMap& m) {
  const float* p = slots + m.slot0 + m.slice * m.sps;
  float part = 0.f;
  for (int j = 0; j < m.sps; ++j) part += p[j];
  return part;
}

// Everything after the row is in registers and the slots are visible: combine,
// RMS^-1, the optional statistics, scale and store.  `t` is the token.
template <class IO, int N>
__device__ __forceinline__ void finish_token(const Params& P, const LaneMap& m, const float* slots,
                                             const uint4 (&v)[N], const uint4 (&gm)[N * IO::kGammaVecs], long long t) {
  const float total = combine_slices(slots, m, P.S);
  const float r = rstd_of(total, m.inv_d, P.eps);
  if (!m.active) return;
  if (m.rstd != nullptr && m.first) m.rstd[t] = r;
  if (m.partials != nullptr && m.g == 0) m.partials[(long long)m.slice * P.T + t] = own_slice_scalar(slots, m);
  const float2 r2 = make_float2(r, r);
  unsigned char* out = m.y + (unsigned long long)t * m.out_pitch + m.chunk_off;
#pragma unroll
  for (int i = 0; i < N; ++i) {
    if (i < m.nvalid)
      st_stream(reinterpret_cast<uint4*>(out + (size_t)i * m.stride),
                IO::scale_chunk(v[i], gm[i * IO::kGammaVecs], gm[i * IO::kGammaVecs + IO::kGammaVecs - 1], r2));
  }
}

// gamma for the thread's chunks: kGammaVecs 16-byte bf16 vectors per activation chunk.
template <class IO, int N>
__device__ __forceinline__ void load_gamma(const LaneMap& m, uint4 (&gm)[N * IO::kGammaVecs]) {
#pragma unroll
  for (int i = 0; i < N; ++i) {
    const int c = m.g + i * (int)(m.stride >> 4);  // the thread's i-th activation chunk inside its slice row
#pragma unroll
    for (int v = 0; v < IO::kGammaVecs; ++v)
      gm[i * IO::kGammaVecs + v] = i < m.nvalid ? __ldg(m.gamma + c * IO::kGammaVecs + v) : make_uint4(0u, 0u, 0u, 0u);
  }
}

}  // namespace qknorm

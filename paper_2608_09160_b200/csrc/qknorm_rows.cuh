// Register-resident row kernel: the whole Q row and K row of one token live in
// the registers of one CTA between the single read and the single write
// (Section III-C: only the final result goes to HBM).
//
// Thread layout.  The CTA is cut into S groups of G threads, one group per
// column slice ("rank" of Algorithm 1).  Thread g of group s owns the 16-byte
// chunks g, g+G, g+2G, ... of slice s, for Q and for K, so
//   * a warp reads consecutive 16-byte chunks of one slice row (coalesced),
//   * every value a thread holds belongs to ONE slice: its running sum of
//     squares is a piece of that slice's Phase-A scalar S_local,
//   * gamma for those chunks is loaded once and stays in registers over the
//     token loop (the W_local multiply of Phase B needs no memory traffic).
// The group's scalar is formed by a shuffle tree (and, for G > 32, one shared
// memory slot per warp); after ONE barrier every thread adds the slices'
// scalars in ascending slice order (the "P2P reduction" line of Algorithm 1),
// forms RMS^-1, scales and stores.  Shared-memory slots are double buffered by
// token parity so the loop needs no second barrier.
//
// Token schedule (Section III-D): a bounded grid of co-resident CTAs, CTA b
// takes tokens b, b+grid, b+2*grid, ...
#pragma once
#include "qknorm_device.cuh"
#include "qknorm_params.h"

namespace qknorm {

template <int NQ, int NK, int MAXT>
__global__ void __launch_bounds__(MAXT) rows_kernel(const __grid_constant__ Params P) {
  __shared__ float slots[2][2][32];

  const int tid = threadIdx.x;
  const int G = P.G;
  const int s = tid >> P.logG;
  const int g = tid & (G - 1);
  const bool live = s < P.S;
  const int ss = live ? s : 0;
  const int logsub = P.logG < 5 ? P.logG : 5;   // lanes that reduce by shuffle: min(G, 32)
  const int sps = G >> logsub;                  // shared-memory slots per slice
  const int slot = tid >> logsub;
  const bool slot_leader = (tid & ((1 << logsub) - 1)) == 0;

  const int cq = P.q.w >> 3;  // 16-byte chunks per slice row
  const int ck = P.k.w >> 3;

  const uint4* xq = NQ ? reinterpret_cast<const uint4*>(P.q.x[ss]) : nullptr;
  const uint4* xk = NK ? reinterpret_cast<const uint4*>(P.k.x[ss]) : nullptr;
  uint4* yq = NQ ? reinterpret_cast<uint4*>(P.q.y[ss]) : nullptr;
  uint4* yk = NK ? reinterpret_cast<uint4*>(P.k.y[ss]) : nullptr;

  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  uint4 gq[NQ > 0 ? NQ : 1], gk[NK > 0 ? NK : 1];
#pragma unroll
  for (int i = 0; i < NQ; ++i) {
    const int c = g + i * G;
    gq[i] = (live && c < cq) ? __ldg(reinterpret_cast<const uint4*>(P.q.gamma[ss]) + c) : zero;
  }
#pragma unroll
  for (int i = 0; i < NK; ++i) {
    const int c = g + i * G;
    gk[i] = (live && c < ck) ? __ldg(reinterpret_cast<const uint4*>(P.k.gamma[ss]) + c) : zero;
  }

  int par = 0;
  for (long long t = blockIdx.x; t < P.T; t += gridDim.x, par ^= 1) {
    uint4 vq[NQ > 0 ? NQ : 1], vk[NK > 0 ? NK : 1];
    const uint4* rq = xq + t * cq;
    const uint4* rk = xk + t * ck;
    // ---- the one read of the row -------------------------------------------------
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const int c = g + i * G;
      vq[i] = (live && c < cq) ? ld_stream(rq + c) : zero;
    }
#pragma unroll
    for (int i = 0; i < NK; ++i) {
      const int c = g + i * G;
      vk[i] = (live && c < ck) ? ld_stream(rk + c) : zero;
    }
    // ---- Phase A: this slice's sum of squares -------------------------------------
    float aq = 0.f, ak = 0.f;
#pragma unroll
    for (int i = 0; i < NQ; ++i) aq = chunk_sumsq(vq[i], aq);
#pragma unroll
    for (int i = 0; i < NK; ++i) ak = chunk_sumsq(vk[i], ak);
    if (logsub == 5) {
      if (NQ) aq += __shfl_xor_sync(0xffffffffu, aq, 16);
      if (NK) ak += __shfl_xor_sync(0xffffffffu, ak, 16);
    }
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) {
      if (NQ) aq += __shfl_xor_sync(0xffffffffu, aq, off);
      if (NK) ak += __shfl_xor_sync(0xffffffffu, ak, off);
    }
    if (slot_leader) {
      if (NQ) slots[par][0][slot] = aq;
      if (NK) slots[par][1][slot] = ak;
    }
    __syncthreads();
    // ---- combine the slices' scalars in ascending slice order ----------------------
    float totq = 0.f, totk = 0.f, myq = 0.f, myk = 0.f;
    for (int s2 = 0; s2 < P.S; ++s2) {
      float pq = 0.f, pk = 0.f;
      for (int j = 0; j < sps; ++j) {
        if (NQ) pq += slots[par][0][s2 * sps + j];
        if (NK) pk += slots[par][1][s2 * sps + j];
      }
      totq += pq;
      totk += pk;
      if (s2 == tid) { myq = pq; myk = pk; }
    }
    // ---- RMS^-1, the gamma multiply, the final scaling, the one write ---------------
    if (NQ) {
      const float r = rstd_from_sumsq(totq, P.q.d, P.eps);
      if (P.q.rstd != nullptr && tid == 0) P.q.rstd[t] = r;
      if (P.q.partials != nullptr && tid < P.S) P.q.partials[(long long)tid * P.T + t] = myq;
      uint4* oq = yq + t * cq;
#pragma unroll
      for (int i = 0; i < NQ; ++i) {
        const int c = g + i * G;
        if (live && c < cq) st_stream(oq + c, scale_chunk(vq[i], gq[i], r));
      }
    }
    if (NK) {
      const float r = rstd_from_sumsq(totk, P.k.d, P.eps);
      if (P.k.rstd != nullptr && tid == 0) P.k.rstd[t] = r;
      if (P.k.partials != nullptr && tid < P.S) P.k.partials[(long long)tid * P.T + t] = myk;
      uint4* ok = yk + t * ck;
#pragma unroll
      for (int i = 0; i < NK; ++i) {
        const int c = g + i * G;
        if (live && c < ck) st_stream(ok + c, scale_chunk(vk[i], gk[i], r));
      }
    }
  }
}

using RowsKernel = void (*)(const Params);

// Instantiated in qknorm_rows_inst.cu, one translation unit per NQ.
// Returns nullptr when (nq, nk) is outside the instantiated set.
RowsKernel rows_kernel_throughput(int nq, int nk);  // CTAs of <= 256 threads
RowsKernel rows_kernel_latency(int nq, int nk);     // CTAs of <= 512 threads

// The chunk counts per thread that are instantiated; a request is rounded up to
// the next one (the surplus iterations are predicated off).
__host__ inline int rows_round_up_n(int n, bool latency) {
  const int tp[] = {0, 1, 2, 3, 4, 5, 6, 8};
  const int lat[] = {0, 1, 2, 4};
  if (latency) {
    for (int v : lat)
      if (n <= v) return v;
  } else {
    for (int v : tp)
      if (n <= v) return v;
  }
  return -1;
}

}  // namespace qknorm

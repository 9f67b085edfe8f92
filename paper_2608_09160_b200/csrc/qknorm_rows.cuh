// Register-resident row kernel: the whole Q row and K row of one token live in
// the registers of one CTA between the single read and the single write
// (Section III-C: only the final result goes to HBM).  Loads are plain 128-bit
// streaming loads, so this variant is the one for few tokens (decode sizes: one
// load round trip per row, no shared-memory staging) and the fallback of the
// TMA ring kernel.  Thread layout and arithmetic: qknorm_rowmap.cuh.
//
// One __syncthreads per token; the shared-memory slots are double buffered by
// token parity so that the loop needs no second barrier.
//
// Token schedule (Section III-D): a bounded grid of co-resident CTAs, CTA b
// takes tokens b, b+grid, b+2*grid, ...
#pragma once
#include "qknorm_rowmap.cuh"

namespace qknorm {

template <int N, class IO>
__global__ void __launch_bounds__(max_threads_for(N), min_blocks_for(N)) rows_kernel(const __grid_constant__ Params P) {
  __shared__ __align__(16) float slots[2][kMaxSlots];
  // Programmatic dependent launch (both instructions are no-ops without the launch attribute): let
  // the next kernel of the stream begin its own launch now, work out this thread's place in the row,
  // and only then wait: no memory is touched before everything earlier in the stream has completed
  // and is visible.  Back-to-back decode calls overlap their launch latencies this way.
  asm volatile("griddepcontrol.launch_dependents;");
  const LaneMap m = make_lane<IO>(P, threadIdx.x, N);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  uint4 gm[N * IO::kGammaVecs];
  load_gamma<IO, N>(m, gm);

  int par = 0;
  for (long long t = blockIdx.x; t < P.T; t += gridDim.x, par ^= 1) {
    uint4 v[N];
    const unsigned char* row = m.x + (unsigned long long)t * m.in_pitch + m.chunk_off;
#pragma unroll
    for (int i = 0; i < N; ++i)
      v[i] = i < m.nvalid ? ld_stream(reinterpret_cast<const uint4*>(row + (size_t)i * m.stride))
                          : make_uint4(0u, 0u, 0u, 0u);
    const float a = lane_group_sum(sumsq_chunks<IO, N>(v), P.log_sub);  // Phase A
    if (m.leader) slots[par][m.slot] = a;
    __syncthreads();
    finish_token<IO, N>(P, m, slots[par], v, gm, t);
  }
}

using RowsKernel = void (*)(const Params);
RowsKernel rows_kernel_for(int n, int elem_bytes);  // nullptr outside the instantiated set

}  // namespace qknorm

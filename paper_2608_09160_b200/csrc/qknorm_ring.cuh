// Prefill kernel: a persistent CTA streams its tokens through a ring of shared
// memory stages filled by the TMA unit (cp.async.bulk, completion on an
// mbarrier), so the bytes in flight per SM are set by the ring depth and not by
// how many registers the resident threads can spare.
//
// One stage holds one token: its Q row and its K row, every slice, laid out as
// the gathered row (Q slice 0..S-1, then K slice 0..S-1).  A stage is filled by
// 2*S bulk copies (one per slice row) issued by the first lanes of warp 0.
//
// Per token (Algorithm 1, phases A-C):
//   wait for the stage  ->  each thread pulls its 16-byte chunks into registers
//   -> per-slice sum of squares (shuffle tree + one shared-memory slot per lane group)
//   -> ONE __syncthreads: the slots are visible AND every thread is done with the
//      stage, so warp 0 immediately refills it with the token NST iterations ahead
//   -> slices' scalars added in ascending slice order, RMS^-1, (x*gamma)*RMS^-1,
//      one streaming 16-byte store per chunk straight from registers.
// Thread layout and arithmetic: qknorm_rowmap.cuh.  In-place calls are safe: a
// row is completely inside the ring before any of it is overwritten, and no
// other row is ever written by this CTA.
//
// Every wait on an mbarrier is bounded (about one second); a wait that runs
// out records an error word and the whole CTA leaves together, after one more
// bounded wait for the copies that are still on their way into its stages.
#pragma once
#include "qknorm_rowmap.cuh"

namespace qknorm {

namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false if the phase did not complete within ~1 s.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  while (!mbar_try_wait(bar, parity)) {
    if (globaltimer_ns() - t0 > 1000000000ull) return false;
  }
  return true;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
// global -> shared bulk copy; bytes % 16 == 0, both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                          uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}

}  // namespace ptx

constexpr int kRingMaxStages = 16;

// Dynamic shared memory: nst stages of stage_bytes each.  A stage is the gathered
// row followed by 16 bytes of zeros (stage_bytes >= row bytes + 16): a chunk
// position a thread does not have is read from the zeros, so the loads need no
// bounds test and contribute nothing to the sum of squares.
template <int N>
__global__ void __launch_bounds__(max_threads_for(N), min_blocks_for(N))
ring_kernel(const __grid_constant__ Params P, const int nst, const int stage_bytes, int* error_word) {
  extern __shared__ __align__(128) unsigned char ring_smem[];
  __shared__ __align__(16) float slots[2][kMaxSlots];
  __shared__ __align__(8) unsigned long long bars[kRingMaxStages];

  const int tid = threadIdx.x;
  const LaneMap m = make_lane<IoBf16>(P, tid, N);
  const uint32_t smem0 = ptx::smem_u32(ring_smem);
  const uint32_t bar0 = ptx::smem_u32(bars);
  const uint32_t row_bytes = ((uint32_t)P.q.d + (uint32_t)P.k.d) * 2u;

  if (tid == 0) {
    for (int i = 0; i < nst; ++i) ptx::mbar_init(bar0 + 8u * i, 1u);
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (tid < nst) *reinterpret_cast<uint4*>(ring_smem + (size_t)tid * stage_bytes + row_bytes) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();

  // tokens of this CTA: blockIdx.x + i * gridDim.x, i = 0 .. n_my-1
  const long long T = P.T;
  const long long first = blockIdx.x;
  const long long n_my = first < T ? (T - first + gridDim.x - 1) / gridDim.x : 0;

  // warp 0, lane l < 2S issues the copy of slice row l (Q slices first, then K slices)
  const bool issue_q = tid < P.S;
  const int is = issue_q ? tid : tid - P.S;
  uint32_t my_bytes = 0, my_dst = 0;
  unsigned long long my_pitch = 0;  // bytes between consecutive rows of the source
  const unsigned char* my_src = nullptr;
  if (tid < 2 * P.S) {
    const TensorArgs& A = issue_q ? P.q : P.k;
    if (A.d != 0) {
      my_bytes = (uint32_t)A.w * 2u;
      my_pitch = (unsigned long long)A.ldx * 2ull;
      my_src = reinterpret_cast<const unsigned char*>(A.x[is]);
      my_dst = (issue_q ? 0u : (uint32_t)P.q.d * 2u) + (uint32_t)is * my_bytes;
    }
  }
  const uint64_t policy = ptx::policy_evict_first();

  auto issue = [&](long long i, int st) {  // called by all of warp 0
    const long long t = first + i * gridDim.x;
    if (tid == 0) ptx::mbar_arrive_expect_tx(bar0 + 8u * st, row_bytes);
    __syncwarp();
    if (my_bytes)
      ptx::bulk_load(smem0 + (uint32_t)st * (uint32_t)stage_bytes + my_dst, my_src + (unsigned long long)t * my_pitch,
                     my_bytes, bar0 + 8u * st, policy);
  };

  if (tid < 32) {
    const int pre = n_my < nst ? (int)n_my : nst;
    for (int i = 0; i < pre; ++i) issue(i, i);
  }

  uint4 gm[N];
  load_gamma<IoBf16, N>(m, gm);
  // loop-invariant offsets inside a stage: the chunk, or the zeros behind the row
  uint32_t soff[N];
#pragma unroll
  for (int j = 0; j < N; ++j) soff[j] = j < m.nvalid ? m.stage_off + (uint32_t)j * m.stride : row_bytes;

  int par = 0, st = 0;
  uint32_t phase = 0;
  for (long long i = 0; i < n_my; ++i, par ^= 1) {
    const long long t = first + i * gridDim.x;
    const bool arrived = ptx::mbar_wait_bounded(bar0 + 8u * st, phase);
    const uint32_t base = smem0 + (uint32_t)st * (uint32_t)stage_bytes;
    uint4 v[N];
#pragma unroll
    for (int j = 0; j < N; ++j) v[j] = ptx::lds128(base + soff[j]);
    const float a = lane_group_sum(sumsq_chunks<IoBf16, N>(v), P.log_sub);  // Phase A
    if (m.leader) slots[par][m.slot] = a;
    // slots visible; the stage has been read by everyone.  The same barrier makes the time-out
    // decision one for the whole CTA: a thread whose wait ran out has only read a stage that may
    // be incomplete, nothing has been stored yet, and now everybody leaves together.
    if (__syncthreads_or(arrived ? 0 : 1)) {
      if (tid == 0) atomicCAS(error_word, 0, 1);  // 1 = a stage never arrived
      // Before the CTA retires (and its shared memory can go to another CTA) give every copy that
      // is still on its way one more bounded wait: stage j holds iteration i + ((j - st) mod nst).
      if (tid < nst) {
        const long long i2 = i + ((tid - st + nst) % nst);
        if (i2 < n_my) ptx::mbar_wait_bounded(bar0 + 8u * tid, (uint32_t)((i2 / nst) & 1));
      }
      __syncthreads();
      return;
    }
    if (tid < 32 && i + nst < n_my) issue(i + nst, st);
    finish_token<IoBf16, N>(P, m, slots[par], v, gm, t);
    if (++st == nst) { st = 0; phase ^= 1u; }
  }
}

using RingKernel = void (*)(const Params, int, int, int*);
RingKernel ring_kernel_for(int n);  // nullptr outside the instantiated set

}  // namespace qknorm

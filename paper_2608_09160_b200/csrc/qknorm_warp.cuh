// Prefill kernel: one warp per token, fed by the TMA unit.
//
// Every warp owns ONE shared-memory stage and one mbarrier.  The stage holds the
// warp's current token as the gathered row (Q slices, then K slices).  Per token:
//
//   wait for the stage  ->  drain it into registers (every lane pulls its 16-byte
//   chunks, up to L of them)  ->  per-slice sums of squares with shuffles only
//   ->  as soon as that reduction is done every lane has consumed the stage, so
//   the warp re-arms it with its NEXT token (2*S bulk copies, one per slice row)
//   ->  slices' scalars added in ascending slice order, RMS^-1, (x*gamma)*RMS^-1,
//   streaming 16-byte stores straight from registers.
//
// So each warp always has its next row in flight while it works on the current
// one (about 18-20 KB per warp, 8 warps per SM), there is no block-level barrier
// in the token loop, and the instructions per token that are not per-chunk work
// (shuffles, rsqrt, barrier wait, TMA issue) are spread over the whole row instead
// of a few chunks per thread.  That matters: this op has to push ~1.6e12
// elements/s through 148 SMs, so the instruction issue rate bounds it as much as
// DRAM does.
//
// Lane layout.  The 32 lanes are cut into S groups of g lanes (g = largest power
// of two <= 32/S); group s serves slice s ("rank" s of Algorithm 1) of both
// tensors.  Lane l of a group owns chunks l, l+g, l+2g, ... of its Q slice row
// (chunk slots 0 .. nq-1) and of its K slice row (slots nq4 .. nq4+nk-1, nq4 = nq
// rounded up to a multiple of 4).  Because the row arrives through shared memory,
// global traffic is whole slice rows whatever S is.  The slice scalar S_local is
// the lane's own sum plus a log2(g)-step shuffle tree (Phase A); the scalars are
// added in ascending slice order with S broadcasts (the P2P-reduction line of
// Phase B); RMS^-1 = rsqrt(S_global / H_total + eps); y = (x*gamma)*RMS^-1,
// rounded once (Phases B/C).
//
// Shared memory.  Slice s of a tensor starts at s * (slice bytes + skew) inside
// the stage; the skew (g*16 bytes when g < 8) puts the lane groups that read in
// the same quarter-warp on different banks.  16 bytes of zeros close the stage: a
// chunk slot a lane does not have is read from there, so loads need no bounds
// test and add nothing to the sums.  gamma is staged once per CTA as
// [chunk slot][lane], conflict-free for every warp.
//
// In-place calls are safe: a row is completely in registers before any of it is
// overwritten, and the only other row the warp touches is its next one.
// Every mbarrier wait is bounded (about one second); a wait that runs out records
// an error word and the warp leaves as a whole, after one more bounded wait for the
// copy that may still be on its way into its stage.
//
// Short unsharded rows (tokens_per_warp = R > 1).  The same kernel with the lane groups
// serving R consecutive TOKENS instead of S slices of one token: the stage holds a tile
// of R rows, every group keeps its own sums of squares (nothing is combined across
// groups), and the warp walks over tiles.  The per-token work of a warp (barrier wait,
// copy issue, shuffle tree, rsqrt, queue) is then done once per R tokens, which is what
// rows of a few hundred bytes need.
//
// Token schedule: a bounded persistent grid (Section III-D).  The first two waves of
// tokens are dealt round-robin; after that a warp takes its next token from a counter
// of the launch (one atomic add per token, issued a token ahead), so warps that run
// slower simply take fewer tokens.  Start-up: the warps of a CTA ask for their first
// rows a few hundred nanoseconds apart, and the kernel may be launched while the
// previous kernel of the stream is still running (programmatic dependent launch).
#pragma once
#include <type_traits>

#include "qknorm_ring.cuh"
#include "qknorm_rowmap.cuh"

namespace qknorm {

constexpr int kWarpMaxCtaWarps = 4;  // the CTA size is a launch parameter: 1..4 warps
// Registers are shaped for this many resident CTAs of 4 warps (80 / 128 / 168 / 255 registers
// per thread).  FP8 rows are instruction-bound and gain from a third CTA at 17..24 slots; bf16
// rows are faster with the registers than with the extra warps.
__host__ __device__ constexpr int warp_min_blocks(int l, int elem_bytes) {
  return l <= 8 ? 6 : (l <= 16 ? 4 : ((l <= 24 && elem_bytes == 1) ? 3 : 2));
}

struct WarpArgs {
  int log_g;            // log2 of the lanes per slice
  int nq, nk;           // chunk slots in use per lane for the Q part / the K part
  int nq4;              // first K slot (nq rounded up to a multiple of 4)
  int stage_bytes;      // bytes of one warp's stage (multiple of 128)
  int q_slice_stride;   // bytes between consecutive Q slices inside a stage (slice bytes + skew)
  int k_slice_stride;
  int k_base;           // byte offset of the K part inside a stage
  int zero_off;         // byte offset of the 16 zero bytes
  int* error_word;
  // Token queue of this launch, or nullptr for the fixed round-robin schedule.  Word 0: tokens
  // handed out beyond the first wave; word 1: warps that have left.  Both are zero when the
  // kernel starts and the last warp to leave puts them back to zero.
  unsigned long long* queue;
  int stagger_cycles;   // SM clock cycles between the first row requests of consecutive warps of a CTA
  // Short unsharded rows (S == 1): R > 1 tokens side by side per warp.  The lane groups then serve R
  // consecutive tokens instead of S slices of one token (stage rows = tokens, nothing is combined
  // across groups), and the kernel walks over tiles of R tokens instead of tokens.
  int tokens_per_warp;
};

// EXACT: every lane has all nq / nk chunk slots (S*g == 32 and the slice rows are
// whole multiples of g chunks), so the stores need no per-lane test either.
template <int L, bool EXACT, class IO>
__global__ void __launch_bounds__(kWarpMaxCtaWarps * 32, warp_min_blocks(L, IO::kBytes))
warp_kernel(const __grid_constant__ Params P, const __grid_constant__ WarpArgs wa) {
  constexpr int GV = IO::kGammaVecs;                            // 16-byte gamma vectors per chunk slot
  extern __shared__ __align__(128) unsigned char warp_smem[];  // one stage per warp
  __shared__ uint4 gsm[L * GV][32];
  __shared__ __align__(8) unsigned long long bars[kWarpMaxCtaWarps];

  // Programmatic dependent launch (no-ops without the launch attribute): the next kernel of the
  // stream may start its own launch now; this one sets up its barriers and addresses and then
  // waits, so no global memory is touched before everything earlier in the stream is complete.
  // (The host sizes this kernel's shared memory so that no SM can take more CTAs than the grid
  // gives it: a CTA of the next launch finds room only where a CTA of this one has left.)
  asm volatile("griddepcontrol.launch_dependents;");
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int g = 1 << wa.log_g;
  const int s = lane >> wa.log_g;
  const int l = lane & (g - 1);
  const int R = wa.tokens_per_warp;            // 1: lane groups are slices; > 1: lane groups are tokens
  const int groups = R > 1 ? R : P.S;
  const bool active = s < groups;
  const int srow = active ? s : 0;             // which row of the stage the lane's group reads
  const int ss = R > 1 ? 0 : srow;             // which slice's buffers the lane's group uses
  const int cq = (P.q.w * IO::kBytes) >> 4, ck = (P.k.w * IO::kBytes) >> 4;  // 16-byte chunks per slice row
  const int nvq = EXACT ? wa.nq : ((active && l < cq) ? (cq - l + g - 1) / g : 0);
  const int nvk = EXACT ? wa.nk : ((active && l < ck) ? (ck - l + g - 1) / g : 0);
  const int n_slots = wa.nq4 + wa.nk;  // uniform

  unsigned char* stage = warp_smem + (size_t)warp * wa.stage_bytes;
  const uint32_t stage_u32 = ptx::smem_u32(stage);
  const uint32_t bar = ptx::smem_u32(&bars[warp]);
  if (lane == 0) {
    ptx::mbar_init(bar, 1u);
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    *reinterpret_cast<uint4*>(stage + wa.zero_off) = make_uint4(0u, 0u, 0u, 0u);
  }
  // ---- who issues which bulk copy: lane i < groups the Q row i of the stage, lane groups+i the K row i ----
  const bool issue_q = lane < groups;
  const int is = issue_q ? lane : lane - groups;
  const int my_tok = R > 1 ? is : 0;           // token of the tile this lane's copy fetches
  uint32_t my_bytes = 0, my_dst = 0;
  unsigned long long my_pitch = 0;  // bytes between consecutive rows of the source
  const unsigned char* my_src = nullptr;
  if (lane < 2 * groups) {
    const TensorArgs& A = issue_q ? P.q : P.k;
    if (A.d != 0) {
      my_bytes = (uint32_t)A.w * IO::kBytes;
      my_pitch = (unsigned long long)A.ldx * IO::kBytes;
      my_src = reinterpret_cast<const unsigned char*>(A.x[R > 1 ? 0 : is]);
      my_dst = issue_q ? (uint32_t)is * (uint32_t)wa.q_slice_stride
                       : (uint32_t)wa.k_base + (uint32_t)is * (uint32_t)wa.k_slice_stride;
    }
  }
  const uint32_t row_bytes = ((uint32_t)P.q.d + (uint32_t)P.k.d) * IO::kBytes;
  const uint64_t policy = ptx::policy_evict_first();
  const long long units = R > 1 ? (P.T + R - 1) / R : P.T;  // what the warps walk over: tokens, or tiles of R tokens
  auto arm = [&](long long u) {  // whole warp: unit u into the stage
    const long long tok = u * R + my_tok;
    if (lane == 0) {
      const long long left = P.T - u * R;
      ptx::mbar_arrive_expect_tx(bar, row_bytes * (uint32_t)(left < R ? left : R));
    }
    __syncwarp();
    if (my_bytes && tok < P.T)
      ptx::bulk_load(stage_u32 + my_dst, my_src + (unsigned long long)tok * my_pitch, my_bytes, bar, policy);
  };

  const int cta_warps = blockDim.x >> 5;
  const long long first = (long long)blockIdx.x * cta_warps + warp;
  const long long step = (long long)gridDim.x * cta_warps;
  __syncwarp();  // the warp's mbarrier is initialised (lane 0 did it above)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // Staggered start: warp w of a CTA asks for its first row w * stagger_cycles after warp 0 does.
  // If all warps of the grid asked at once, all first rows would arrive together, late (the
  // requests are served side by side), and nothing would be written until then; spread over
  // about one token time, the warps start in the rhythm they settle into anyway and the first
  // stores go out after a third of the time.
  const long long c_entry = wa.stagger_cycles ? clock64() : 0ll;
  const long long my_delay = (long long)wa.stagger_cycles * warp;
  if (my_delay == 0 && first < units) arm(first);

  // gamma, once per CTA: slot j of lane `lane` holds the GV bf16 vectors that go with the lane's
  // j-th chunk; slots dealt round-robin to the warps.
  bool gamma_f16 = false;
  {
    const uint4* gq = reinterpret_cast<const uint4*>(P.q.gamma[ss]) + (size_t)l * GV;
    const uint4* gk = reinterpret_cast<const uint4*>(P.k.gamma[ss]) + (size_t)l * GV;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    bool fits = true;
    // B slots per batch: all loads of a batch are issued before the first one is used, so staging
    // costs one or two memory round trips instead of one per slot
    constexpr int B = (L <= 8 ? 4 : 10) / GV;  // the small-L kernels are held to 64 registers
    for (int j0 = warp; j0 < L; j0 += B * cta_warps) {
      uint4 gv[B][GV];
#pragma unroll
      for (int b = 0; b < B; ++b) {
        const int j = j0 + b * cta_warps;
#pragma unroll
        for (int v = 0; v < GV; ++v) {
          gv[b][v] = zero;
          if (j < nvq) gv[b][v] = __ldg(gq + (size_t)j * g * GV + v);
          else if (j >= wa.nq4 && j - wa.nq4 < nvk) gv[b][v] = __ldg(gk + (size_t)(j - wa.nq4) * g * GV + v);
        }
      }
#pragma unroll
      for (int b = 0; b < B; ++b) {
        const int j = j0 + b * cta_warps;
        if (j < L) {
#pragma unroll
          for (int v = 0; v < GV; ++v) {
            gsm[j * GV + v][lane] = gv[b][v];
            if (IO::kF16Gamma)
              fits = fits && bf16x2_fits_f16(gv[b][v].x) && bf16x2_fits_f16(gv[b][v].y) && bf16x2_fits_f16(gv[b][v].z) &&
                     bf16x2_fits_f16(gv[b][v].w);
          }
        }
      }
    }
    if (IO::kF16Gamma) {
      // every gamma value of the CTA is also an fp16 value: keep gamma as fp16 (each thread
      // converts the entries it wrote) and multiply with the fp16 mixed FMA
      gamma_f16 = __syncthreads_and(fits ? 1 : 0) != 0;
      if (gamma_f16) {
        for (int j = warp; j < L; j += cta_warps) {
#pragma unroll
          for (int v = 0; v < GV; ++v) {
            uint4 gv = gsm[j * GV + v][lane];
            gv.x = bf16x2_to_f16x2(gv.x);
            gv.y = bf16x2_to_f16x2(gv.y);
            gv.z = bf16x2_to_f16x2(gv.z);
            gv.w = bf16x2_to_f16x2(gv.w);
            gsm[j * GV + v][lane] = gv;
          }
        }
      }
    }
  }
  __syncthreads();  // the last block-level barrier
  if (my_delay != 0) {
    while (clock64() - c_entry < my_delay) __nanosleep(64);
    if (first < units) arm(first);
  }


  // ---- loop-invariant per-lane offsets ------------------------------------------------------------
  // inside a stage: chunk l of the lane's Q slice / K slice
  const uint32_t sq0 = stage_u32 + (uint32_t)srow * (uint32_t)wa.q_slice_stride + (uint32_t)l * 16u;
  const uint32_t sk0 = stage_u32 + (uint32_t)wa.k_base + (uint32_t)srow * (uint32_t)wa.k_slice_stride + (uint32_t)l * 16u;
  const uint32_t szero = stage_u32 + (uint32_t)wa.zero_off;
  const uint32_t sstride = (uint32_t)g * 16u;
  unsigned char* yq = reinterpret_cast<unsigned char*>(P.q.y[ss]) + (size_t)l * 16u;
  unsigned char* yk = reinterpret_cast<unsigned char*>(P.k.y[ss]) + (size_t)l * 16u;
  const unsigned long long q_row = (unsigned long long)P.q.ldy * IO::kBytes, k_row = (unsigned long long)P.k.ldy * IO::kBytes;

  // Which token a warp takes next.  Without a queue warp i takes tokens i, i + step, i + 2*step, ...
  // With a queue only the first two waves are fixed and every further token comes from the launch's
  // counter, one atomic add per token, so a warp on a slow SM simply takes fewer tokens and all warps
  // finish within a token or two of each other.  The add for the token after next is issued when the
  // next one is armed and its result is read a whole token later, so its round trip to L2 (about a
  // microsecond under load) never holds the warp up.
  unsigned long long ticket = 0;
  const bool queued = wa.queue != nullptr;
  auto claim_issue = [&]() {
    if (lane == 0) ticket = atomicAdd(wa.queue, 1ull);
  };
  auto claim_result = [&]() -> long long { return 2 * step + (long long)__shfl_sync(0xffffffffu, ticket, 0); };
  long long t = first, t_next = first + step;
  if (queued && t_next < units) claim_issue();

  uint32_t phase = 0;
  bool timed_out = false;
  while (t < units) {
    // one decision for the whole warp: lanes that saw the phase complete must not go on alone
    if (__any_sync(0xffffffffu, !ptx::mbar_wait_bounded(bar, phase))) {
      timed_out = true;
      break;
    }
    phase ^= 1u;
    // ---- drain the stage into registers --------------------------------------------------------
    uint4 v[L];
#pragma unroll
    for (int jb = 0; jb < L; jb += 4) {
      if (jb >= n_slots) break;
      const bool kpart = jb >= wa.nq4;  // uniform: a block of 4 slots is all Q or all K
      const uint32_t base = kpart ? sk0 + (uint32_t)(jb - wa.nq4) * sstride : sq0 + (uint32_t)jb * sstride;
      const int nv = kpart ? nvk - (jb - wa.nq4) : nvq - jb;  // slots of this block the lane has
#pragma unroll
      for (int i = 0; i < 4; ++i) v[jb + i] = ptx::lds128((EXACT || i < nv) ? base + (uint32_t)i * sstride : szero);
    }
    // ---- Phase A: sums of squares of the lane's Q chunks and K chunks ---------------------------------
    float2 aq = make_float2(0.f, 0.f), ak = make_float2(0.f, 0.f);
#pragma unroll
    for (int jb = 0; jb < L; jb += 4) {
      if (jb >= n_slots) break;
      // four independent chains (one per chunk slot), two accumulators each
      float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f, c4 = 0.f, c5 = 0.f, c6 = 0.f, c7 = 0.f;
      IO::sumsq_word(v[jb].x, c0, c1);
      IO::sumsq_word(v[jb + 1].x, c2, c3);
      IO::sumsq_word(v[jb + 2].x, c4, c5);
      IO::sumsq_word(v[jb + 3].x, c6, c7);
      IO::sumsq_word(v[jb].y, c0, c1);
      IO::sumsq_word(v[jb + 1].y, c2, c3);
      IO::sumsq_word(v[jb + 2].y, c4, c5);
      IO::sumsq_word(v[jb + 3].y, c6, c7);
      IO::sumsq_word(v[jb].z, c0, c1);
      IO::sumsq_word(v[jb + 1].z, c2, c3);
      IO::sumsq_word(v[jb + 2].z, c4, c5);
      IO::sumsq_word(v[jb + 3].z, c6, c7);
      IO::sumsq_word(v[jb].w, c0, c1);
      IO::sumsq_word(v[jb + 1].w, c2, c3);
      IO::sumsq_word(v[jb + 2].w, c4, c5);
      IO::sumsq_word(v[jb + 3].w, c6, c7);
      const float2 b = __fadd2_rn(__fadd2_rn(make_float2(c0, c1), make_float2(c2, c3)),
                                  __fadd2_rn(make_float2(c4, c5), make_float2(c6, c7)));
      if (jb >= wa.nq4) ak = __fadd2_rn(ak, b);
      else aq = __fadd2_rn(aq, b);
    }
    float pq = aq.x + aq.y, pk = ak.x + ak.y;
    if (g > 16) { pq += __shfl_xor_sync(0xffffffffu, pq, 16); pk += __shfl_xor_sync(0xffffffffu, pk, 16); }
    if (g > 8) { pq += __shfl_xor_sync(0xffffffffu, pq, 8); pk += __shfl_xor_sync(0xffffffffu, pk, 8); }
    if (g > 4) { pq += __shfl_xor_sync(0xffffffffu, pq, 4); pk += __shfl_xor_sync(0xffffffffu, pk, 4); }
    if (g > 2) { pq += __shfl_xor_sync(0xffffffffu, pq, 2); pk += __shfl_xor_sync(0xffffffffu, pk, 2); }
    if (g > 1) { pq += __shfl_xor_sync(0xffffffffu, pq, 1); pk += __shfl_xor_sync(0xffffffffu, pk, 1); }
    // ---- the slices' scalars in ascending slice order -------------------------------------------------
    float totq = pq, totk = pk;  // (R > 1: every lane group keeps its own token's sums)
    if (R > 1) {
      __syncwarp();  // every lane has consumed the stage
    } else if (P.S > 1) {
      totq = 0.f;
      totk = 0.f;
      for (int s2 = 0; s2 < P.S; ++s2) {
        totq += __shfl_sync(0xffffffffu, pq, s2 << wa.log_g);
        totk += __shfl_sync(0xffffffffu, pk, s2 << wa.log_g);
      }
    } else {
      totq = __shfl_sync(0xffffffffu, pq, 0);  // also the point where every lane has consumed the stage
      totk = __shfl_sync(0xffffffffu, pk, 0);
    }
    // every lane's chunks are in registers and have been used: refill the stage with the next token
    long long t_after = units;
    if (t_next < units) {
      arm(t_next);
      if (!queued) {
        t_after = t_next + step;
      } else {
        t_after = claim_result();          // asked for one token ago
        if (t_after < units) claim_issue();  // the one after that
      }
    }
    const long long tg = R > 1 ? t * R + s : t;   // the token this lane's group works on
    const bool live = R > 1 ? (active && tg < P.T) : true;

    const float rq = rstd_of(totq, P.q.inv_d, P.eps);
    const float rk = rstd_of(totk, P.k.inv_d, P.eps);
    if (R > 1 ? (live && l == 0) : lane == 0) {
      if (P.q.rstd != nullptr) P.q.rstd[tg] = rq;
      if (P.k.rstd != nullptr) P.k.rstd[tg] = rk;
    }
    if (active && l == 0 && live) {
      if (P.q.partials != nullptr) P.q.partials[(long long)ss * P.T + tg] = pq;
      if (P.k.partials != nullptr) P.k.partials[(long long)ss * P.T + tg] = pk;
    }
    // ---- Phases B/C: (x * gamma) * RMS^-1, the one write ------------------------------------------------
    unsigned char* dq_ = yq + (unsigned long long)tg * q_row;
    unsigned char* dk_ = yk + (unsigned long long)tg * k_row;
    auto store_pass = [&](auto f16_gamma) {  // the branch on the gamma format stays outside the slot loops
#pragma unroll
      for (int jb = 0; jb < L; jb += 4) {
        if (jb >= n_slots) break;
        const bool kpart = jb >= wa.nq4;
        const float r = kpart ? rk : rq;
        const float2 r2 = make_float2(r, r);
        unsigned char* dst = kpart ? dk_ + (size_t)(jb - wa.nq4) * sstride : dq_ + (size_t)jb * sstride;
        const int nv = !live ? 0 : (kpart ? (EXACT ? wa.nk : nvk) - (jb - wa.nq4) : (EXACT ? wa.nq : nvq) - jb);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 ga = gsm[(jb + i) * GV][lane], gb = gsm[(jb + i) * GV + GV - 1][lane];
          uint4 o;
          if constexpr (decltype(f16_gamma)::value) o = IO::scale_chunk_g16(v[jb + i], ga, gb, r2);
          else o = IO::scale_chunk(v[jb + i], ga, gb, r2);
          if (i < nv) st_stream(reinterpret_cast<uint4*>(dst + (size_t)i * sstride), o);
        }
      }
    };
    if (IO::kF16Gamma && gamma_f16) store_pass(std::true_type{});
    else store_pass(std::false_type{});
    t = t_next;
    t_next = t_after;
  }
  if (timed_out) {
    // The row this warp waited for never arrived in time.  Record it, then give the copy one more
    // bounded wait: the CTA must not retire (and hand its shared memory to another CTA) while a
    // bulk copy into that memory may still land.
    if (lane == 0) atomicCAS(wa.error_word, 0, 2);  // 2 = a warp's stage never arrived
    __any_sync(0xffffffffu, !ptx::mbar_wait_bounded(bar, phase));
  }
  if (wa.queue != nullptr) {
    // leave the queue as this launch found it: the last warp out (of all warps of the grid,
    // with or without tokens, timed out or not) puts both words back to zero
    __syncwarp();
    if (lane == 0) {
      __threadfence();
      const unsigned long long gone = atomicAdd(wa.queue + 1, 1ull);
      if (gone + 1ull == (unsigned long long)step) {
        atomicExch(wa.queue, 0ull);
        atomicExch(wa.queue + 1, 0ull);
      }
    }
  }
}

using WarpKernel = void (*)(const Params, const WarpArgs);
WarpKernel warp_kernel_for(int l, bool exact, int elem_bytes);  // nullptr outside the instantiated set
int warp_round_up_l(int n);                      // next instantiated L >= n, or -1

}  // namespace qknorm

// Column-sharded (tensor-parallel) QK-RMSNorm with the scalar exchange of Algorithm 1,
// Phase B: every rank holds one column slice of Q and of K, forms its own sums of
// squares (Phase A), PUSHES the two scalars into every peer's inbox, waits until the
// peers' scalars have landed in its own inbox, adds all N scalars in ascending rank
// order and scales its slice (Phase C).  Per token and tensor 8 bytes cross the link to
// each peer instead of the slice itself (Section III-A).
//
// How it differs from the flag protocol of Algorithm 1 (kept: push into the consumer's
// memory, wait on local memory only, fp32 scalars, rank-order sum, bounded grid):
//  * value and flag are ONE 8-byte word {epoch tag, fp32 bits} written with a single
//    64-bit store.  A naturally aligned 64-bit store is never torn, so the consumer
//    either sees the old word or the whole new one: no fence between data and flag, no
//    second write.
//  * nothing is cleared between calls.  The tag is the call's epoch (the caller counts
//    calls); a slot counts as filled when its tag equals the current epoch.  Inboxes are
//    double-buffered by epoch parity: a rank can run at most one call ahead of a peer
//    (it needs the peer's scalars of call c+1 to finish c+1), so what it writes for c+2
//    lands in the half the peer finished with c.
//  * no warp is set aside for communication.  The kernel keeps the warp-level design of
//    the single-GPU path: a warp has its NEXT tile of rows in flight (TMA bulk copies into
//    its own shared-memory stage) while it waits for the scalars of the current one, and
//    the other warps of the SM cover the link latency.
//  * a warp works on several tokens side by side (see tp_kernel), and one lane per
//    (token, peer) pair carries the exchange: all pushes of a tile are one store
//    instruction, all polls one loop.
//
// The launch is cooperative, so the driver itself refuses a grid whose CTAs are not all
// resident (the bounded grid of Section III-D).  Every warp works through its tokens in
// ascending order and pushes before it waits, so with all CTAs of all ranks resident
// the smallest unfinished token can always complete: no deadlock, whatever grid each
// rank chose.
//
// One launch can serve several ranks whose buffers live on the same GPU (CTA b serves
// rank b mod n_local).  That is how the protocol is exercised on a single GPU: all
// ranks' CTAs are co-resident in one cooperative launch, "peer" inboxes are just other
// allocations.  With one process per GPU n_local is 1 and the peers' inboxes are peer
// mappings of their memory.
//
// Every wait is bounded.  A poll that runs out (or sees that another warp's did) records
// {code, token, missing rank} in the header of the rank's inbox, waits for the warp's own
// bulk copy in flight and leaves; outputs of unfinished tokens are then undefined.
#pragma once
#include <type_traits>

#include "qknorm_warp.cuh"

namespace qknorm {

constexpr int kTpRounds = 4;        // exchange rounds of 32 (token, rank) pairs: tile * N <= 128
constexpr int kTpHeaderWords = 32;  // 256-byte header in front of the slots (64-bit words)

// status codes in word 0 of the inbox header
constexpr int kTpOk = 0;
constexpr int kTpPeerTimeout = 1;   // a peer's scalar did not arrive in time
constexpr int kTpStageTimeout = 2;  // the warp's own bulk copy did not arrive in time

struct TpRank {
  const void* xq;            // X_local of Q: [T, wq]
  const void* xk;            // X_local of K: [T, wk]
  const uint16_t* gq;        // W_local of Q: [wq] bf16
  const uint16_t* gk;
  void* yq;                  // Y_local (may equal xq)
  void* yk;
  float* rstd_q;             // optional [T]: RMS^-1 as this rank computed it
  float* rstd_k;
  float* partial_q;          // optional [T]: this rank's own S_local
  float* partial_k;
  unsigned long long* inbox;                   // this rank's inbox (header + slots)
  unsigned long long* peer_inbox[kMaxShards];  // rank p's inbox as this GPU addresses it
  int rank;
  int pad_;
};

struct TpParams {
  TpRank r[kMaxShards];   // the n_local ranks this launch serves
  int n_local;
  int N;                  // ranks in all (the TP degree)
  long long T;
  long long cap;          // token capacity the inboxes were sized for
  int wq, wk;             // slice widths (elements); 0 = tensor absent
  long long ldxq, ldxk, ldyq, ldyk;  // row pitches (elements)
  float inv_dq, inv_dk;   // 1 / H_total = 1 / (N * w)
  float eps;
  uint32_t epoch;         // != 0
  unsigned long long wait_ns;
  int log_g;              // log2 of the lanes that serve one token (32 >> log_g tokens per warp tile)
  int nq, nk, nq4;        // chunk slots per lane: Q part, K part, first K slot
  int stage_bytes;        // one warp's stage: the tile's Q rows, its K rows, 16 zero bytes
  int q_row_stride;       // bytes between consecutive tokens' Q rows inside a stage (row + bank skew)
  int k_row_stride;
  int k_base, zero_off;
};

namespace ptx {
__device__ __forceinline__ void st_relaxed_sys_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_sys_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_relaxed_gpu_s32(const int* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
}  // namespace ptx

// Resident CTAs of 4 warps the registers are shaped for.  The exchange keeps four slot
// pointers, the tag and the peer bookkeeping alive across the token loop, so a slice row
// gets a few registers more per thread than the single-GPU kernel gives it.
__host__ __device__ constexpr int tp_min_blocks(int l, int elem_bytes) {
  return l <= 8 ? 6 : (l <= 16 ? 3 : 2);
}

__host__ __device__ inline long long tp_slot_index(int parity, int tensor, int src_rank, int N, long long cap) {
  return (long long)kTpHeaderWords + ((long long)((parity * 2 + tensor) * N + src_rank)) * cap;
}

// Waits until both slots carry the epoch's tag (a null slot counts as filled).  False when
// the wait ran out or another warp of this rank already gave up.
__device__ __forceinline__ bool tp_poll2(const unsigned long long* sq, const unsigned long long* sk, uint32_t epoch,
                                         unsigned long long wait_ns, const int* status, float& vq, float& vk) {
  unsigned long long a = sq ? ptx::ld_relaxed_sys_u64(sq) : 0ull;
  unsigned long long b = sk ? ptx::ld_relaxed_sys_u64(sk) : 0ull;
  bool ha = !sq || (uint32_t)(a >> 32) == epoch;
  bool hb = !sk || (uint32_t)(b >> 32) == epoch;
  if (!(ha && hb)) {
    const unsigned long long t0 = ptx::globaltimer_ns();
    unsigned spins = 0;
    while (true) {
      if (!ha) {
        a = ptx::ld_relaxed_sys_u64(sq);
        ha = (uint32_t)(a >> 32) == epoch;
      }
      if (!hb) {
        b = ptx::ld_relaxed_sys_u64(sk);
        hb = (uint32_t)(b >> 32) == epoch;
      }
      if (ha && hb) break;
      if ((++spins & 31u) == 0u) {
        if (ptx::globaltimer_ns() - t0 > wait_ns) return false;
        if (ptx::ld_relaxed_gpu_s32(status) != kTpOk) return false;
      }
    }
  }
  vq = __uint_as_float((uint32_t)a);
  vk = __uint_as_float((uint32_t)b);
  return true;
}

// A warp works on a TILE of R = 32 >> log_g consecutive tokens at a time: lane group s
// (g = 32 / R lanes) serves token t0 + s, lane l of the group owns chunks l, l+g, ... of
// that token's Q slice row and K slice row.  Slice rows are short (a few KB), so one token
// per warp would spend most of its instructions on per-token work (barrier wait, copy
// issue, shuffles, push, poll); with R tokens side by side that work is done once per tile:
// one log2(g)-step shuffle tree gives all R scalars, ONE store instruction pushes R x (N-1)
// scalars (lane p*R + r: token r to rank p), one poll loop collects them, N broadcasts per
// tensor form all R sums.  When R * N exceeds 32 the pairs take up to kTpRounds rounds.
template <int L, class IO>
__global__ void __launch_bounds__(kWarpMaxCtaWarps * 32, tp_min_blocks(L, IO::kBytes))
tp_kernel(const __grid_constant__ TpParams P) {
  constexpr int GV = IO::kGammaVecs;
  extern __shared__ __align__(128) unsigned char tp_smem[];  // one stage per warp
  __shared__ uint4 gsm[L * GV][32];
  __shared__ __align__(8) unsigned long long bars[kWarpMaxCtaWarps];

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int lr = (int)(blockIdx.x % (unsigned)P.n_local);
  const TpRank& R = P.r[lr];
  const long long cta = blockIdx.x / (unsigned)P.n_local;
  const long long ctas = gridDim.x / (unsigned)P.n_local;
  int* const status = reinterpret_cast<int*>(R.inbox);

  const int g = 1 << P.log_g;
  const int tile = 32 >> P.log_g;  // tokens per tile
  const int s = lane >> P.log_g;   // which token of the tile this lane serves
  const int l = lane & (g - 1);
  const int cq = (P.wq * IO::kBytes) >> 4, ck = (P.wk * IO::kBytes) >> 4;  // 16-byte chunks per slice row
  const int nvq = l < cq ? (cq - l + g - 1) >> P.log_g : 0;
  const int nvk = l < ck ? (ck - l + g - 1) >> P.log_g : 0;
  const int n_slots = P.nq4 + P.nk;

  unsigned char* stage = tp_smem + (size_t)warp * P.stage_bytes;
  const uint32_t stage_u32 = ptx::smem_u32(stage);
  const uint32_t bar = ptx::smem_u32(&bars[warp]);
  if (lane == 0) {
    ptx::mbar_init(bar, 1u);
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    *reinterpret_cast<uint4*>(stage + P.zero_off) = make_uint4(0u, 0u, 0u, 0u);
  }
  // lane i < tile fetches the Q slice row of token i of the tile, lane tile + i its K slice row
  const bool issue_q = lane < tile;
  const int is = issue_q ? lane : lane - tile;
  uint32_t my_bytes = 0, my_dst = 0;
  unsigned long long my_pitch = 0;
  const unsigned char* my_src = nullptr;
  if (lane < 2 * tile) {
    if (issue_q && cq) {
      my_bytes = (uint32_t)P.wq * IO::kBytes;
      my_pitch = (unsigned long long)P.ldxq * IO::kBytes;
      my_src = reinterpret_cast<const unsigned char*>(R.xq);
      my_dst = (uint32_t)is * (uint32_t)P.q_row_stride;
    } else if (!issue_q && ck) {
      my_bytes = (uint32_t)P.wk * IO::kBytes;
      my_pitch = (unsigned long long)P.ldxk * IO::kBytes;
      my_src = reinterpret_cast<const unsigned char*>(R.xk);
      my_dst = (uint32_t)P.k_base + (uint32_t)is * (uint32_t)P.k_row_stride;
    }
  }
  const uint32_t row_bytes = ((uint32_t)P.wq + (uint32_t)P.wk) * IO::kBytes;
  const uint64_t policy = ptx::policy_evict_first();
  auto arm = [&](long long t0) {  // whole warp; t0 = first token of the tile
    const long long left = P.T - t0;
    const int n = left < tile ? (int)left : tile;
    if (lane == 0) ptx::mbar_arrive_expect_tx(bar, (uint32_t)n * row_bytes);
    __syncwarp();
    if (my_bytes && is < n) ptx::bulk_load(stage_u32 + my_dst, my_src + (unsigned long long)(t0 + is) * my_pitch, my_bytes, bar, policy);
  };

  const int cta_warps = blockDim.x >> 5;
  const long long first = (cta * cta_warps + warp) * tile;
  const long long step = ctas * cta_warps * tile;
  __syncwarp();
  if (first < P.T) arm(first);

  // gamma of the slice, once per CTA, as [chunk slot][lane] (the same values in every lane group)
  bool gamma_f16 = false;
  {
    const uint4* gq = reinterpret_cast<const uint4*>(R.gq) + (size_t)l * GV;
    const uint4* gk = reinterpret_cast<const uint4*>(R.gk) + (size_t)l * GV;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    bool fits = true;
    for (int j = warp; j < L; j += cta_warps) {
#pragma unroll
      for (int v = 0; v < GV; ++v) {
        uint4 gv = zero;
        if (j < nvq) gv = __ldg(gq + (size_t)j * g * GV + v);
        else if (j >= P.nq4 && j - P.nq4 < nvk) gv = __ldg(gk + (size_t)(j - P.nq4) * g * GV + v);
        gsm[j * GV + v][lane] = gv;
        if (IO::kF16Gamma)
          fits = fits && bf16x2_fits_f16(gv.x) && bf16x2_fits_f16(gv.y) && bf16x2_fits_f16(gv.z) && bf16x2_fits_f16(gv.w);
      }
    }
    if (IO::kF16Gamma) {
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

  // ---- the exchange: pair number (rd * 32 + lane) = p * tile + r carries token r of the tile to and
  // from rank p; kTpRounds rounds of 32 pairs cover tile * N <= 128 pairs ---------------------------
  const int parity = (int)(P.epoch & 1u);
  const int xr = lane & (tile - 1);         // token of the tile this lane exchanges (the same in every round)
  const int xp0 = lane >> (5 - P.log_g);    // rank this lane talks to in round 0; round rd: xp0 + rd * g
  const long long slot_q_out = tp_slot_index(parity, 0, R.rank, P.N, P.cap) + xr;  // in a peer's inbox
  const long long slot_k_out = tp_slot_index(parity, 1, R.rank, P.N, P.cap) + xr;
  const int rounds = (tile * P.N + 31) >> 5;
  const unsigned long long tag = (unsigned long long)P.epoch << 32;

  const uint32_t sq0 = stage_u32 + (uint32_t)s * (uint32_t)P.q_row_stride + (uint32_t)l * 16u;
  const uint32_t sk0 = stage_u32 + (uint32_t)P.k_base + (uint32_t)s * (uint32_t)P.k_row_stride + (uint32_t)l * 16u;
  const uint32_t szero = stage_u32 + (uint32_t)P.zero_off;
  const uint32_t sstride = (uint32_t)g * 16u;
  unsigned char* yq = reinterpret_cast<unsigned char*>(R.yq) + (size_t)l * 16u;
  unsigned char* yk = reinterpret_cast<unsigned char*>(R.yk) + (size_t)l * 16u;
  const unsigned long long q_row = (unsigned long long)P.ldyq * IO::kBytes, k_row = (unsigned long long)P.ldyk * IO::kBytes;

  uint32_t phase = 0;
  for (long long t0 = first; t0 < P.T; t0 += step) {
    if (!ptx::mbar_wait_bounded(bar, phase)) {
      if (lane == 0 && atomicCAS(status, kTpOk, kTpStageTimeout) == kTpOk) {
        status[1] = (int)(t0 & 0x7fffffff);
        status[2] = -1;
      }
      return;
    }
    phase ^= 1u;
    const long long t = t0 + s;       // this lane group's token
    const bool live = t < P.T;        // the last tile may be short: its stage rows are stale, never published
    // ---- drain the stage into registers --------------------------------------------------------
    uint4 v[L];
#pragma unroll
    for (int jb = 0; jb < L; jb += 4) {
      if (jb >= n_slots) break;
      const bool kpart = jb >= P.nq4;
      const uint32_t base = kpart ? sk0 + (uint32_t)(jb - P.nq4) * sstride : sq0 + (uint32_t)jb * sstride;
      const int nv = kpart ? nvk - (jb - P.nq4) : nvq - jb;
#pragma unroll
      for (int i = 0; i < 4; ++i) v[jb + i] = ptx::lds128(i < nv ? base + (uint32_t)i * sstride : szero);
    }
    // ---- Phase A: S_local of the Q slice and of the K slice, one token per lane group --------------
    float2 aq = make_float2(0.f, 0.f), ak = make_float2(0.f, 0.f);
#pragma unroll
    for (int jb = 0; jb < L; jb += 4) {
      if (jb >= n_slots) break;
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
      if (jb >= P.nq4) ak = __fadd2_rn(ak, b);
      else aq = __fadd2_rn(aq, b);
    }
    float pq = aq.x + aq.y, pk = ak.x + ak.y;
    // the same tree in every lane of a group: all g lanes end with the same bits
    if (g > 16) { pq += __shfl_xor_sync(0xffffffffu, pq, 16); pk += __shfl_xor_sync(0xffffffffu, pk, 16); }
    if (g > 8) { pq += __shfl_xor_sync(0xffffffffu, pq, 8); pk += __shfl_xor_sync(0xffffffffu, pk, 8); }
    if (g > 4) { pq += __shfl_xor_sync(0xffffffffu, pq, 4); pk += __shfl_xor_sync(0xffffffffu, pk, 4); }
    if (g > 2) { pq += __shfl_xor_sync(0xffffffffu, pq, 2); pk += __shfl_xor_sync(0xffffffffu, pk, 2); }
    if (g > 1) { pq += __shfl_xor_sync(0xffffffffu, pq, 1); pk += __shfl_xor_sync(0xffffffffu, pk, 1); }
    // ---- Phase B, communication path: token xr's scalars to every rank ------------------------------
    const float mine_q = __shfl_sync(0xffffffffu, pq, xr << P.log_g);  // also: every lane has consumed the stage
    const float mine_k = __shfl_sync(0xffffffffu, pk, xr << P.log_g);
    const bool xlive = t0 + xr < P.T;
#pragma unroll
    for (int rd = 0; rd < kTpRounds; ++rd) {
      if (rd >= rounds) break;
      const int xp = xp0 + (rd << P.log_g);
      if (xlive && xp < P.N && xp != R.rank) {
        unsigned long long* peer = R.peer_inbox[xp];
        if (cq) ptx::st_relaxed_sys_u64(peer + slot_q_out + t0, tag | (unsigned long long)__float_as_uint(mine_q));
        if (ck) ptx::st_relaxed_sys_u64(peer + slot_k_out + t0, tag | (unsigned long long)__float_as_uint(mine_k));
      }
    }
    const bool armed = t0 + step < P.T;
    if (armed) arm(t0 + step);  // the next tile is on its way while this one waits for its peers
    if (live && l == 0) {
      if (R.partial_q != nullptr) R.partial_q[t] = pq;
      if (R.partial_k != nullptr) R.partial_k[t] = pk;
    }
    // ---- wait for the peers' scalars in this rank's own inbox ---------------------------------------
    float inq[kTpRounds], ink[kTpRounds];  // pair (rd, lane): rank xp's scalars of token xr (its own for xp == rank)
    unsigned missing = 0u;
    int missing_round = 0;
#pragma unroll
    for (int rd = 0; rd < kTpRounds; ++rd) {
      inq[rd] = mine_q;
      ink[rd] = mine_k;
      if (rd >= rounds) continue;
      const int xp = xp0 + (rd << P.log_g);
      bool got = true;
      if (xlive && xp < P.N && xp != R.rank) {
        const unsigned long long* src_q = cq ? R.inbox + tp_slot_index(parity, 0, xp, P.N, P.cap) + xr + t0 : nullptr;
        const unsigned long long* src_k = ck ? R.inbox + tp_slot_index(parity, 1, xp, P.N, P.cap) + xr + t0 : nullptr;
        got = tp_poll2(src_q, src_k, P.epoch, P.wait_ns, status, inq[rd], ink[rd]);
      }
      const unsigned m = __ballot_sync(0xffffffffu, !got);
      if (m != 0u && missing == 0u) {
        missing = m;
        missing_round = rd;
      }
    }
    if (missing != 0u) {
      if (lane == 0 && atomicCAS(status, kTpOk, kTpPeerTimeout) == kTpOk) {
        const int bad = __ffs((int)missing) - 1;
        status[1] = (int)((t0 + (bad & (tile - 1))) & 0x7fffffff);
        status[2] = (bad >> (5 - P.log_g)) + (missing_round << P.log_g);
      }
      if (armed) ptx::mbar_wait_bounded(bar, phase);  // the warp's own copy in flight
      return;
    }
    // ---- S_global: all N scalars in ascending rank order, the same on every rank ----------------------
    float totq = 0.f, totk = 0.f;
#pragma unroll
    for (int rd = 0; rd < kTpRounds; ++rd) {
      for (int pp = 0; pp < g; ++pp) {  // rank rd * g + pp sits in lane pp * tile + s of round rd
        if ((rd << P.log_g) + pp >= P.N) break;
        totq += __shfl_sync(0xffffffffu, inq[rd], pp * tile + s);
        totk += __shfl_sync(0xffffffffu, ink[rd], pp * tile + s);
      }
    }
    const float rq = rstd_of(totq, P.inv_dq, P.eps);
    const float rk = rstd_of(totk, P.inv_dk, P.eps);
    if (live && l == 0) {
      if (R.rstd_q != nullptr) R.rstd_q[t] = rq;
      if (R.rstd_k != nullptr) R.rstd_k[t] = rk;
    }
    // ---- Phase B compute path and Phase C: (x * gamma) * RMS^-1, the one write ------------------------
    unsigned char* dq_ = yq + (unsigned long long)t * q_row;
    unsigned char* dk_ = yk + (unsigned long long)t * k_row;
    auto store_pass = [&](auto f16_gamma) {
#pragma unroll
      for (int jb = 0; jb < L; jb += 4) {
        if (jb >= n_slots) break;
        const bool kpart = jb >= P.nq4;
        const float r = kpart ? rk : rq;
        const float2 r2 = make_float2(r, r);
        unsigned char* dst = kpart ? dk_ + (size_t)(jb - P.nq4) * sstride : dq_ + (size_t)jb * sstride;
        const int nv = live ? (kpart ? nvk - (jb - P.nq4) : nvq - jb) : 0;
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
  }
}

using TpKernel = void (*)(const TpParams);
TpKernel tp_kernel_for(int l, int elem_bytes);  // nullptr outside the instantiated set

}  // namespace qknorm

// Column-sharded (tensor-parallel) QK-RMSNorm with the scalar exchange of Algorithm 1,
// Phase B: every rank holds one column slice of Q and of K, forms its own sums of
// squares (Phase A), PUSHES the two scalars into every peer's inbox, waits until the
// peers' scalars have landed in its own inbox, adds all N scalars in one fixed order
// (the same on every rank) and scales its slice (Phase C).  Per token and tensor 8 bytes cross the link to
// each peer instead of the slice itself (Section III-A).
//
// How it differs from the flag protocol of Algorithm 1 (kept: push into the consumer's
// memory, wait on local memory only, fp32 scalars, the same sum on every rank, bounded grid):
//  * value and flag are ONE 8-byte word {epoch tag, fp32 bits} written with a single
//    64-bit store.  A naturally aligned 64-bit store is never torn, so the consumer
//    either sees the old word or the whole new one: no fence between data and flag, no
//    second write.
//  * nothing is cleared between calls.  The tag is the call's epoch (the caller counts
//    calls); a slot counts as filled when its tag equals the current epoch.  Inboxes are
//    double-buffered by epoch parity: a rank can run at most one call ahead of a peer
//    (it needs the peer's scalars of call c+1 to finish c+1), so what it writes for c+2
//    lands in the half the peer finished with c.
//  * no warp is set aside for communication, and the wait is taken off the critical path
//    by software pipelining inside every warp instead.  A warp owns three shared-memory
//    stages, each holding one TILE of tokens' slice rows (filled by TMA bulk copies).  In
//    step j it (1) takes tile j from its stage, forms the sums of squares and pushes
//    them, (2) only then collects the peers' scalars of tile j-1 -- pushed a whole step
//    ago, so normally already there -- and scales and writes tile j-1 from ITS stage,
//    (3) refills that stage with tile j+2.  Tile j+1 is in flight during all of step j.
//    Rows are read from shared memory twice instead of being held in registers, which
//    keeps the register count low enough for 16 and more warps per SM.
//  * S_global is a pairwise tree over the rank index (log2 N shuffle steps for all tokens of a
//    tile at once) instead of a loop over the ranks; the tree is the same on every rank, so
//    all ranks still get identical bits.
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

constexpr int kTpStages = 3;        // shared-memory stages per warp
constexpr int kTpMaxCtaWarps = 8;
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
  int stage_bytes;        // one stage: the tile's Q rows, then its K rows (multiple of 128)
  int q_row_stride;       // bytes between consecutive tokens' Q rows inside a stage (row + bank skew)
  int k_row_stride;
  int k_base;             // byte offset of the K rows inside a stage
  int gamma_bytes;        // shared memory in front of the stages: gamma_q slice, gamma_k slice (multiple of 128)
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
// one log2(g)-step shuffle tree gives all R scalars, one store instruction pushes 32
// (token, rank) pairs (pair p*R + r: token r to rank p), one poll loop collects them, N
// broadcasts per tensor form all R sums.  R * N <= 32.
template <int LOG_G, class IO>
__global__ void __launch_bounds__(kTpMaxCtaWarps * 32, 2)
tp_kernel(const __grid_constant__ TpParams P) {
  constexpr int GV = IO::kGammaVecs;
  extern __shared__ __align__(128) unsigned char tp_smem[];  // gamma_q, gamma_k, then kTpStages stages per warp
  __shared__ __align__(8) unsigned long long bars[kTpMaxCtaWarps][kTpStages];

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int lr = (int)(blockIdx.x % (unsigned)P.n_local);
  const TpRank& R = P.r[lr];
  const long long cta = blockIdx.x / (unsigned)P.n_local;
  const long long ctas = gridDim.x / (unsigned)P.n_local;
  int* const status = reinterpret_cast<int*>(R.inbox);

  constexpr int g = 1 << LOG_G;
  constexpr int tile = 32 >> LOG_G;  // tokens per tile
  const int s = lane >> LOG_G;       // which token of the tile this lane serves
  const int l = lane & (g - 1);
  const int cq = (P.wq * IO::kBytes) >> 4, ck = (P.wk * IO::kBytes) >> 4;  // 16-byte chunks per slice row
  const int nvq = l < cq ? (cq - l + g - 1) >> LOG_G : 0;                 // chunks of this lane
  const int nvk = l < ck ? (ck - l + g - 1) >> LOG_G : 0;

  const uint32_t smem0 = ptx::smem_u32(tp_smem);
  const uint32_t stages0 = smem0 + (uint32_t)P.gamma_bytes + (uint32_t)warp * kTpStages * (uint32_t)P.stage_bytes;
  const uint32_t bar0 = ptx::smem_u32(&bars[warp][0]);
  if (lane == 0) {
#pragma unroll
    for (int st = 0; st < kTpStages; ++st) ptx::mbar_init(bar0 + 8u * st, 1u);
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
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
  // Short rows (up to 1 KB) that follow one another without a gap both in memory and in the stage:
  // the whole tile of that tensor is ONE bulk copy (issued by the lane of its first row) instead of
  // one per row.  Measured: 320-byte FP8 rows 3.9 -> 4.8 TB/s; rows of 2 KB are faster copied singly.
  const bool whole_tile = my_bytes != 0 && my_bytes <= 1024u && my_pitch == my_bytes &&
                          (issue_q ? (uint32_t)P.q_row_stride : (uint32_t)P.k_row_stride) == my_bytes;

  const int cta_warps = blockDim.x >> 5;
  const long long first = (cta * cta_warps + warp) * tile;
  const long long step = ctas * cta_warps * tile;
  const long long n_tiles = first < P.T ? (P.T - first + step - 1) / step : 0;  // this warp's tiles
  auto arm = [&](long long t0, int st) {  // whole warp: the tile that starts at token t0 into stage st
    const long long left = P.T - t0;
    const int n = left < tile ? (int)left : tile;
    const uint32_t bar = bar0 + 8u * (uint32_t)st;
    if (lane == 0) ptx::mbar_arrive_expect_tx(bar, (uint32_t)n * row_bytes);
    __syncwarp();
    if (whole_tile) {
      if (is == 0)
        ptx::bulk_load(stages0 + (uint32_t)st * (uint32_t)P.stage_bytes + my_dst,
                       my_src + (unsigned long long)t0 * my_pitch, (uint32_t)n * my_bytes, bar, policy);
    } else if (my_bytes && is < n) {
      ptx::bulk_load(stages0 + (uint32_t)st * (uint32_t)P.stage_bytes + my_dst,
                     my_src + (unsigned long long)(t0 + is) * my_pitch, my_bytes, bar, policy);
    }
  };
  __syncwarp();
  if (n_tiles > 0) arm(first, 0);
  if (n_tiles > 1) arm(first + step, 1);

  // gamma of the slice, once per CTA: gamma_q chunks, then gamma_k chunks, in row order
  uint4* const gsm = reinterpret_cast<uint4*>(tp_smem);
  const int gq_vecs = cq * GV, gk_vecs = ck * GV;
  bool gamma_f16 = false;
  {
    bool fits = true;
    for (int i = threadIdx.x; i < gq_vecs + gk_vecs; i += blockDim.x) {
      const uint4 gv = i < gq_vecs ? __ldg(reinterpret_cast<const uint4*>(R.gq) + i)
                                   : __ldg(reinterpret_cast<const uint4*>(R.gk) + (i - gq_vecs));
      gsm[i] = gv;
      if (IO::kF16Gamma)
        fits = fits && bf16x2_fits_f16(gv.x) && bf16x2_fits_f16(gv.y) && bf16x2_fits_f16(gv.z) && bf16x2_fits_f16(gv.w);
    }
    if (IO::kF16Gamma) {
      // every gamma value of the slice is also an fp16 value: keep it as fp16 (each thread converts
      // what it wrote) and multiply with the fp16 mixed FMA
      gamma_f16 = __syncthreads_and(fits ? 1 : 0) != 0;
      if (gamma_f16) {
        for (int i = threadIdx.x; i < gq_vecs + gk_vecs; i += blockDim.x) {
          uint4 gv = gsm[i];
          gv.x = bf16x2_to_f16x2(gv.x);
          gv.y = bf16x2_to_f16x2(gv.y);
          gv.z = bf16x2_to_f16x2(gv.z);
          gv.w = bf16x2_to_f16x2(gv.w);
          gsm[i] = gv;
        }
      }
    }
  }
  __syncthreads();  // the last block-level barrier
  const uint32_t gq_u32 = smem0 + (uint32_t)l * 16u * GV;
  const uint32_t gk_u32 = smem0 + (uint32_t)gq_vecs * 16u + (uint32_t)l * 16u * GV;

  // ---- the exchange: lane p * tile + r carries token r of the tile to and from rank p
  // (tile * N <= 32, the host chooses the tile so) ----------------------------------------------------
  const int parity = (int)(P.epoch & 1u);
  const int xr = lane & (tile - 1);       // token of the tile this lane exchanges
  const int xp = lane >> (5 - LOG_G);     // rank this lane talks to
  const bool remote = xp < P.N && xp != R.rank;
  unsigned long long* push_q = nullptr;        // where this rank's scalars go in rank xp's inbox
  unsigned long long* push_k = nullptr;
  const unsigned long long* poll_q = nullptr;  // where rank xp's scalars land in this rank's inbox
  const unsigned long long* poll_k = nullptr;
  if (remote) {
    unsigned long long* peer = R.peer_inbox[xp];
    if (cq) {
      push_q = peer + tp_slot_index(parity, 0, R.rank, P.N, P.cap) + xr;
      poll_q = R.inbox + tp_slot_index(parity, 0, xp, P.N, P.cap) + xr;
    }
    if (ck) {
      push_k = peer + tp_slot_index(parity, 1, R.rank, P.N, P.cap) + xr;
      poll_k = R.inbox + tp_slot_index(parity, 1, xp, P.N, P.cap) + xr;
    }
  }
  const unsigned long long tag = (unsigned long long)P.epoch << 32;

  const uint32_t sq_lane = (uint32_t)s * (uint32_t)P.q_row_stride + (uint32_t)l * 16u;  // inside a stage
  const uint32_t sk_lane = (uint32_t)P.k_base + (uint32_t)s * (uint32_t)P.k_row_stride + (uint32_t)l * 16u;
  constexpr uint32_t sstride = (uint32_t)g * 16u;
  unsigned char* yq = reinterpret_cast<unsigned char*>(R.yq) + (size_t)l * 16u;
  unsigned char* yk = reinterpret_cast<unsigned char*>(R.yk) + (size_t)l * 16u;
  const unsigned long long q_row = (unsigned long long)P.ldyq * IO::kBytes, k_row = (unsigned long long)P.ldyk * IO::kBytes;

  // sum of squares of this lane's chunks of one row, from shared memory; fixed order
  auto sumsq_row = [&](uint32_t base, int nv) -> float {
    float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f, c4 = 0.f, c5 = 0.f, c6 = 0.f, c7 = 0.f;
    int j = 0;
    for (; j + 4 <= nv; j += 4, base += 4u * sstride) {
      const uint4 a = ptx::lds128(base), b = ptx::lds128(base + sstride);
      const uint4 c = ptx::lds128(base + 2u * sstride), d = ptx::lds128(base + 3u * sstride);
      IO::sumsq_word(a.x, c0, c1); IO::sumsq_word(b.x, c2, c3); IO::sumsq_word(c.x, c4, c5); IO::sumsq_word(d.x, c6, c7);
      IO::sumsq_word(a.y, c0, c1); IO::sumsq_word(b.y, c2, c3); IO::sumsq_word(c.y, c4, c5); IO::sumsq_word(d.y, c6, c7);
      IO::sumsq_word(a.z, c0, c1); IO::sumsq_word(b.z, c2, c3); IO::sumsq_word(c.z, c4, c5); IO::sumsq_word(d.z, c6, c7);
      IO::sumsq_word(a.w, c0, c1); IO::sumsq_word(b.w, c2, c3); IO::sumsq_word(c.w, c4, c5); IO::sumsq_word(d.w, c6, c7);
    }
    for (; j < nv; ++j, base += sstride) {
      const uint4 a = ptx::lds128(base);
      IO::sumsq_word(a.x, c0, c1); IO::sumsq_word(a.y, c2, c3); IO::sumsq_word(a.z, c4, c5); IO::sumsq_word(a.w, c6, c7);
    }
    return ((c0 + c1) + (c2 + c3)) + ((c4 + c5) + (c6 + c7));
  };
  // (x * gamma) * RMS^-1 of this lane's chunks of one row: shared memory -> global, one write
  auto scale_row = [&](uint32_t base, int nv, uint32_t gbase, unsigned char* dst, float r, auto f16_gamma) {
    const float2 r2 = make_float2(r, r);
#pragma unroll 4
    for (int j = 0; j < nv; ++j, base += sstride, gbase += sstride * GV, dst += sstride) {
      const uint4 x = ptx::lds128(base);
      const uint4 ga = ptx::lds128(gbase);
      const uint4 gb = GV > 1 ? ptx::lds128(gbase + 16u) : ga;
      uint4 o;
      if constexpr (decltype(f16_gamma)::value) o = IO::scale_chunk_g16(x, ga, gb, r2);
      else o = IO::scale_chunk(x, ga, gb, r2);
      st_stream(reinterpret_cast<uint4*>(dst), o);
    }
  };
  // stage and mbarrier parity of the tile a step starts with; both advance once per step
  int st_cur = 0;            // j % kTpStages
  uint32_t par_bits = 0u;    // bit st: parity the next wait on stage st expects
  auto next_stage = [](int st) { return st + 1 == kTpStages ? 0 : st + 1; };
  auto wait_stage = [&](int st) -> bool {  // bounded
    const bool ok = ptx::mbar_wait_bounded(bar0 + 8u * (uint32_t)st, (par_bits >> st) & 1u);
    par_bits ^= 1u << st;
    return ok;
  };
  auto give_up = [&](int code, long long token, int rank_missing, bool copy_pending, int st_pending) {
    if (lane == 0 && atomicCAS(status, kTpOk, code) == kTpOk) {
      status[1] = (int)(token & 0x7fffffff);
      status[2] = rank_missing;
    }
    if (copy_pending) wait_stage(st_pending);  // the warp's own copy still in flight
  };

  float held_q = 0.f, held_k = 0.f;  // this lane's pair values of the tile pushed one step ago
  long long t_cur = first;   // first token of tile j
  for (long long j = 0; j <= n_tiles; ++j, t_cur += step, st_cur = next_stage(st_cur)) {
    float mine_q = 0.f, mine_k = 0.f;
    const int st_next = next_stage(st_cur);                       // stage of tile j+1, in flight
    const int st_prev = next_stage(st_next);                      // stage of tile j-1 (= of tile j+2)
    if (j < n_tiles) {
      // ---- step part 1: Phase A of tile j and the push (Phase B, communication path) ---------------
      if (!wait_stage(st_cur)) {
        give_up(kTpStageTimeout, t_cur, -1, j + 1 < n_tiles, st_next);
        return;
      }
      const long long t0 = t_cur;
      const uint32_t st = stages0 + (uint32_t)st_cur * (uint32_t)P.stage_bytes;
      float pq = sumsq_row(st + sq_lane, nvq), pk = sumsq_row(st + sk_lane, nvk);
      // the same tree in every lane of a group: all g lanes end with the same bits
      if (g > 16) { pq += __shfl_xor_sync(0xffffffffu, pq, 16); pk += __shfl_xor_sync(0xffffffffu, pk, 16); }
      if (g > 8) { pq += __shfl_xor_sync(0xffffffffu, pq, 8); pk += __shfl_xor_sync(0xffffffffu, pk, 8); }
      if (g > 4) { pq += __shfl_xor_sync(0xffffffffu, pq, 4); pk += __shfl_xor_sync(0xffffffffu, pk, 4); }
      if (g > 2) { pq += __shfl_xor_sync(0xffffffffu, pq, 2); pk += __shfl_xor_sync(0xffffffffu, pk, 2); }
      if (g > 1) { pq += __shfl_xor_sync(0xffffffffu, pq, 1); pk += __shfl_xor_sync(0xffffffffu, pk, 1); }
      mine_q = __shfl_sync(0xffffffffu, pq, xr << LOG_G);
      mine_k = __shfl_sync(0xffffffffu, pk, xr << LOG_G);
      if (t0 + xr < P.T) {  // a short last tile: rows past the end are stale and never published
        if (push_q) ptx::st_relaxed_sys_u64(push_q + t0, tag | (unsigned long long)__float_as_uint(mine_q));
        if (push_k) ptx::st_relaxed_sys_u64(push_k + t0, tag | (unsigned long long)__float_as_uint(mine_k));
      }
      if (t0 + s < P.T && l == 0) {
        if (R.partial_q != nullptr) R.partial_q[t0 + s] = pq;
        if (R.partial_k != nullptr) R.partial_k[t0 + s] = pk;
      }
    }
    if (j >= 1) {
      // ---- step part 2: tile j-1, pushed one step ago: collect, S_global, Phases B/C -------------
      const long long t0 = t_cur - step;
      const long long t = t0 + s;
      const bool live = t < P.T, xlive = t0 + xr < P.T;
      // lane p*tile + r: rank p's scalars of token r (its own for p == rank, nothing for p >= N)
      float inq = xp < P.N ? held_q : 0.f, ink = xp < P.N ? held_k : 0.f;
      bool got = true;
      if (remote && xlive) got = tp_poll2(poll_q ? poll_q + t0 : nullptr, poll_k ? poll_k + t0 : nullptr, P.epoch, P.wait_ns, status, inq, ink);
      const unsigned missing = __ballot_sync(0xffffffffu, !got);
      if (missing != 0u) {
        const int bad = __ffs((int)missing) - 1;
        give_up(kTpPeerTimeout, t0 + (bad & (tile - 1)), bad >> (5 - LOG_G), j + 1 < n_tiles, st_next);
        return;
      }
      // S_global: the N scalars of a token added pairwise over the rank index (ranks 2i and 2i+1,
      // then pairs of pairs, ...).  Every rank runs the same tree on the same N values, so all ranks
      // get the same bits; log2 steps instead of N.
#pragma unroll
      for (int o = tile; o < 32; o <<= 1) {
        inq += __shfl_xor_sync(0xffffffffu, inq, o);
        ink += __shfl_xor_sync(0xffffffffu, ink, o);
      }
      const float totq = __shfl_sync(0xffffffffu, inq, s);  // lane s = (rank 0, token s) holds token s's sum
      const float totk = __shfl_sync(0xffffffffu, ink, s);
      const float rq = rstd_of(totq, P.inv_dq, P.eps);
      const float rk = rstd_of(totk, P.inv_dk, P.eps);
      if (live) {
        if (l == 0) {
          if (R.rstd_q != nullptr) R.rstd_q[t] = rq;
          if (R.rstd_k != nullptr) R.rstd_k[t] = rk;
        }
        const uint32_t st = stages0 + (uint32_t)st_prev * (uint32_t)P.stage_bytes;
        unsigned char* dq_ = yq + (unsigned long long)t * q_row;
        unsigned char* dk_ = yk + (unsigned long long)t * k_row;
        if (IO::kF16Gamma && gamma_f16) {
          scale_row(st + sq_lane, nvq, gq_u32, dq_, rq, std::true_type{});
          scale_row(st + sk_lane, nvk, gk_u32, dk_, rk, std::true_type{});
        } else {
          scale_row(st + sq_lane, nvq, gq_u32, dq_, rq, std::false_type{});
          scale_row(st + sk_lane, nvk, gk_u32, dk_, rk, std::false_type{});
        }
      }
    }
    // ---- step part 3: the stage tile j-1 lived in takes tile j+2 ---------------------------------
    __syncwarp();
    if (j + 2 < n_tiles) arm(t_cur + 2 * step, st_prev);
    held_q = mine_q;
    held_k = mine_k;
  }
}

using TpKernel = void (*)(const TpParams);
TpKernel tp_kernel_for(int log_g, int elem_bytes);  // log_g in 2..5

}  // namespace qknorm

// Host side of the tiled kernel (qknorm_tp.cuh): validation, tile and grid choice, launch --
// cooperative for the tensor-parallel entry points of include/qknorm_tp.h, plain for the narrow
// unsharded rows the main entry points hand to the same kernel.
// Included by qknorm_api.cu INSIDE its unnamed namespace, after the helpers it uses (device cache,
// occupancy cache, overlap test).
#pragma once

int tp_inbox_bytes(int num_ranks, long long cap, long long* bytes) {
  if (!bytes) return QKNORM_ERR_NULL;
  if (num_ranks < 1 || num_ranks > kMaxShards) return QKNORM_ERR_SHARDS;
  if (cap < 1 || cap > (1LL << 31)) return QKNORM_ERR_SHAPE;
  *bytes = 8LL * (kTpHeaderWords + 4LL * num_ranks * cap);
  return QKNORM_OK;
}

// Tile shape, stage layout, CTA size and kernel for the slice widths in P (wq, wk, N already set).
// Host arithmetic only; QKNORM_ERR_SHAPE when a slice row pair is too long for the kernel.
// `sm_count` (0 = unknown) lets short calls take smaller CTAs so that every SM gets one.
int tp_configure(TpParams& P, int elem_bytes, int sm_count, int* warps_out, int* smem_out, TpKernel* fn_out) {
  const int wq = P.wq, wk = P.wk, N = P.N;
  // Tokens per warp tile: R = 32 / g lane groups of g lanes, one token each.  More tokens per tile
  // spread the per-tile work (barrier waits, copy issue, shuffles, push, poll) over more rows; the
  // tile's bytes times the three stages times the warps must fit the SM's shared memory.  Measured
  // on B200 (8 ranks on one GPU): tiles of 9-12 KB are fastest, 5 KB and 18 KB both cost 15-30 %.
  const int cq = wq * elem_bytes / 16, ck = wk * elem_bytes / 16;
  const int row_bytes = (wq + wk) * elem_bytes;
  // (With a single rank, nothing to exchange and bf16 rows, small tiles and more warps win instead:
  // rows of 640 and 1280 bytes run 7-8 % faster with tiles of at most 3 KB, longer rows the same.
  // FP8 rows cost more instructions per byte and lose 20-40 % that way.)
  // Rows shorter than 2304 bytes still want two tokens per tile (1536-byte rows: 148 us with one,
  // 109 us with two).
  int tile_bytes_default = 12000;
  if (N == 1 && elem_bytes == 2) tile_bytes_default = (row_bytes < 2304 && 2 * row_bytes > 3000) ? 2 * row_bytes : 3000;
  const int tile_bytes_max = env_int("QKNORM_TP_TILE_BYTES", tile_bytes_default);
  const int forced_log_g = env_int("QKNORM_TP_LOG_G", -1);
  int log_g = 5;
  for (int lg = 2; lg <= 5; ++lg) {
    const int tile = 32 >> lg;
    if (tile * N > 32) continue;  // one lane per (token, rank) pair
    if (forced_log_g >= 0 ? lg != forced_log_g : (tile > 1 && tile * row_bytes > tile_bytes_max)) continue;
    log_g = lg;
    break;
  }
  TpKernel fn = tp_kernel_for(log_g, elem_bytes);
  if (!fn) return QKNORM_ERR_SHAPE;
  const int tile = 32 >> log_g;
  {
    const int g = 1 << log_g;
    P.log_g = log_g;
    // rows of a tile side by side in the stage; the skew keeps lane groups that read in the same
    // quarter-warp on different banks
    const bool contiguous = P.ldxq == wq && P.ldxk == wk && env_int("QKNORM_TP_BULK", 1) != 0;
    const int skew = (tile > 1 && g < 8 && !contiguous) ? g * 16 : 0;  // contiguous rows: one copy per tile instead
    P.q_row_stride = cq ? wq * elem_bytes + skew : 0;
    P.k_row_stride = ck ? wk * elem_bytes + skew : 0;
    P.k_base = tile * P.q_row_stride;
    P.stage_bytes = round_up(P.k_base + tile * P.k_row_stride, 128);
    P.gamma_bytes = round_up((wq + wk) * 2, 128);
  }

  // Warps per CTA: the CTA size that puts the most warps on an SM (three stages per warp and one
  // copy of gamma per CTA against the SM's shared memory; 128 registers per thread allow 16 warps);
  // among equals the larger CTA, which shares gamma between more warps.
  constexpr int kSmemPerCta = 227 * 1024;  // sm_100: opt-in maximum of dynamic shared memory per CTA
  constexpr int kSmemPerSm = 228 * 1024;   // and what one SM has, of which every resident CTA reserves 1 KB
  const int forced_warps = env_int("QKNORM_TP_WARPS", 0);
  int max_warps = kTpMaxCtaWarps;
  if (sm_count > 0) {  // few tiles: no more warps per CTA than leaves a CTA for every SM (and every local rank)
    const long long tiles = (P.T + tile - 1) / tile;
    const long long fair = (tiles * P.n_local + sm_count - 1) / sm_count;
    if (fair < max_warps) max_warps = fair < 1 ? 1 : (int)fair;
  }
  int warps = 0, best_per_sm = 0;
  for (int w = max_warps; w >= 1; --w) {
    if (forced_warps > 0 && w != forced_warps) continue;
    const int bytes = P.gamma_bytes + w * kTpStages * P.stage_bytes;
    if (bytes > kSmemPerCta) continue;
    int per_sm = (kSmemPerSm / (bytes + 1024 + 256)) * w;
    if (per_sm > 16) per_sm = 16;
    if (per_sm > best_per_sm) {
      best_per_sm = per_sm;
      warps = w;
    }
  }
  if (warps == 0) return QKNORM_ERR_SHAPE;  // a slice row pair too long for three stages of shared memory
  const int smem = P.gamma_bytes + warps * kTpStages * P.stage_bytes;

  *warps_out = warps;
  *smem_out = smem;
  *fn_out = fn;
  return QKNORM_OK;
}

int run_tp(int elem_bytes, const qknorm_tp_rank* ranks, int n_local, int N, long long T, long long cap,
           int wq, int wk, const int64_t* ld, float eps, uint32_t epoch, uint32_t wait_limit_us,
           cudaStream_t stream) {
  if (N < 1 || N > kMaxShards || n_local < 1 || n_local > N) return QKNORM_ERR_SHARDS;
  if (T < 0 || wq < 0 || wk < 0 || cap < 1 || T > cap || cap > (1LL << 31)) return QKNORM_ERR_SHAPE;
  if ((long long)wq * N > kMaxDim || (long long)wk * N > kMaxDim) return QKNORM_ERR_SHAPE;
  if (!(eps >= 0.0f)) return QKNORM_ERR_EPS;
  if (T == 0) return QKNORM_OK;
  if (wq == 0 && wk == 0) return QKNORM_ERR_SHAPE;
  if (epoch == 0u) return QKNORM_ERR_SHAPE;
  if (!ranks) return QKNORM_ERR_NULL;

  TpParams P;
  memset(&P, 0, sizeof(P));
  P.n_local = n_local;
  P.N = N;
  P.T = T;
  P.cap = cap;
  P.wq = wq;
  P.wk = wk;
  P.ldxq = (ld && ld[0]) ? ld[0] : wq;
  P.ldxk = (ld && ld[1]) ? ld[1] : wk;
  P.ldyq = (ld && ld[2]) ? ld[2] : wq;
  P.ldyk = (ld && ld[3]) ? ld[3] : wk;
  if (P.ldxq < wq || P.ldyq < wq || P.ldxk < wk || P.ldyk < wk) return QKNORM_ERR_SHAPE;
  P.inv_dq = wq ? 1.0f / (float)(wq * N) : 0.0f;
  P.inv_dk = wk ? 1.0f / (float)(wk * N) : 0.0f;
  P.eps = eps;
  P.epoch = epoch;
  P.wait_ns = 1000ull * (wait_limit_us ? wait_limit_us : 1000000u);

  const uintptr_t eb = (uintptr_t)elem_bytes;
  if ((wq * elem_bytes) % 16 || (wk * elem_bytes) % 16) return QKNORM_ERR_ALIGN;
  if ((P.ldxq * elem_bytes) % 16 || (P.ldxk * elem_bytes) % 16 || (P.ldyq * elem_bytes) % 16 || (P.ldyk * elem_bytes) % 16)
    return QKNORM_ERR_ALIGN;
  long long inbox_bytes = 0;
  int rc = tp_inbox_bytes(N, cap, &inbox_bytes);
  if (rc != QKNORM_OK) return rc;

  unsigned seen = 0;
  Region outs[2 * kMaxShards], ins[2 * kMaxShards], others[8 * kMaxShards];
  int n_out = 0, n_other = 0;
  for (int i = 0; i < n_local; ++i) {
    const qknorm_tp_rank& a = ranks[i];
    TpRank& r = P.r[i];
    if (a.rank < 0 || a.rank >= N || (seen >> a.rank) & 1u) return QKNORM_ERR_SHARDS;
    seen |= 1u << a.rank;
    if (wq && (!a.q || !a.gamma_q || !a.out_q)) return QKNORM_ERR_NULL;
    if (wk && (!a.k || !a.gamma_k || !a.out_k)) return QKNORM_ERR_NULL;
    if (!a.inbox || (N > 1 && !a.peer_inbox)) return QKNORM_ERR_NULL;
    r.rank = a.rank;
    r.xq = wq ? a.q : nullptr;
    r.xk = wk ? a.k : nullptr;
    r.gq = wq ? (const uint16_t*)a.gamma_q : nullptr;
    r.gk = wk ? (const uint16_t*)a.gamma_k : nullptr;
    r.yq = wq ? a.out_q : nullptr;
    r.yk = wk ? a.out_k : nullptr;
    r.rstd_q = wq ? a.rstd_q : nullptr;
    r.rstd_k = wk ? a.rstd_k : nullptr;
    r.partial_q = wq ? a.partial_q : nullptr;
    r.partial_k = wk ? a.partial_k : nullptr;
    r.inbox = (unsigned long long*)a.inbox;
    if (!aligned16(r.xq) || !aligned16(r.xk) || !aligned16(r.gq) || !aligned16(r.gk) || !aligned16(r.yq) || !aligned16(r.yk))
      return QKNORM_ERR_ALIGN;
    if (((uintptr_t)a.inbox) & 7u) return QKNORM_ERR_ALIGN;
    if ((((uintptr_t)a.rstd_q) | ((uintptr_t)a.rstd_k) | ((uintptr_t)a.partial_q) | ((uintptr_t)a.partial_k)) & 3u)
      return QKNORM_ERR_ALIGN;
    for (int p = 0; p < N; ++p) {
      if (p == a.rank) continue;
      const void* peer = a.peer_inbox[p];
      if (!peer) return QKNORM_ERR_NULL;
      if (((uintptr_t)peer) & 7u) return QKNORM_ERR_ALIGN;
      r.peer_inbox[p] = (unsigned long long*)peer;
    }
    const uintptr_t rows = (uintptr_t)T;
    if (wq) {
      ins[n_out] = {(uintptr_t)a.q, rows, (uintptr_t)wq * eb, (uintptr_t)P.ldxq * eb};
      outs[n_out++] = {(uintptr_t)a.out_q, rows, (uintptr_t)wq * eb, (uintptr_t)P.ldyq * eb};
      others[n_other++] = {(uintptr_t)a.gamma_q, 1, (uintptr_t)wq * 2u, (uintptr_t)wq * 2u};
    }
    if (wk) {
      ins[n_out] = {(uintptr_t)a.k, rows, (uintptr_t)wk * eb, (uintptr_t)P.ldxk * eb};
      outs[n_out++] = {(uintptr_t)a.out_k, rows, (uintptr_t)wk * eb, (uintptr_t)P.ldyk * eb};
      others[n_other++] = {(uintptr_t)a.gamma_k, 1, (uintptr_t)wk * 2u, (uintptr_t)wk * 2u};
    }
    others[n_other++] = {(uintptr_t)a.inbox, 1, (uintptr_t)inbox_bytes, (uintptr_t)inbox_bytes};
    float* aux[4] = {r.rstd_q, r.rstd_k, r.partial_q, r.partial_k};
    for (float* x : aux)
      if (x) others[n_other++] = {(uintptr_t)x, 1, 4u * rows, 4u * rows};
  }
  // an output may be exactly its own input; any other overlap with a buffer of the call is an error
  for (int i = 0; i < n_out; ++i) {
    for (int j = 0; j < n_out; ++j) {
      if (may_overlap(outs[i], ins[j]) && !(i == j && same_region(outs[i], ins[j]))) return QKNORM_ERR_ALIAS;
      if (j != i && may_overlap(outs[i], outs[j])) return QKNORM_ERR_ALIAS;
    }
    for (int j = 0; j < n_other; ++j)
      if (may_overlap(outs[i], others[j])) return QKNORM_ERR_ALIAS;
  }

  int warps = 0, smem = 0;
  TpKernel fn = nullptr;
  rc = tp_configure(P, elem_bytes, 0, &warps, &smem, &fn);  // host-only: does the shape fit at all?
  if (rc != QKNORM_OK) return rc;
  const int tile = 32 >> P.log_g;

  const DeviceInfo* dev = nullptr;
  rc = current_device(&dev);
  if (rc != QKNORM_OK) return rc;
  rc = tp_configure(P, elem_bytes, dev->sm_count, &warps, &smem, &fn);
  if (rc != QKNORM_OK) return rc;
  if (smem > dev->smem_per_block) return QKNORM_ERR_SHAPE;
  rc = allow_dynamic_smem((const void*)fn, smem);
  if (rc != QKNORM_OK) return rc;
  int resident = 1;
  rc = resident_blocks((const void*)fn, warps * 32, smem, &resident);
  if (rc != QKNORM_OK) return rc;
  const int cap_ctas = env_int("QKNORM_TP_CTAS_PER_SM", 0);
  if (cap_ctas > 0 && cap_ctas < resident) resident = cap_ctas;
  // bounded grid (Section III-D): every CTA of every rank served here is resident at once
  long long per_rank = (long long)resident * dev->sm_count / n_local;
  const long long tiles = (T + tile - 1) / tile;
  const long long needed = (tiles + warps - 1) / warps;
  if (per_rank > needed) per_rank = needed;
  if (per_rank < 1) return QKNORM_ERR_SHARDS;  // more local ranks than resident CTAs
  const unsigned grid = (unsigned)(per_rank * n_local);
  void* args[] = {(void*)&P};
  cudaError_t e = cudaLaunchCooperativeKernel((const void*)fn, dim3(grid), dim3(warps * 32), args, (size_t)smem, stream);
  if (e != cudaSuccess) return set_cuda_error(e);
  return finish_launch("tp");
}



// Unsharded rows on the tiled kernel with a single rank and therefore no exchange -- several tokens
// side by side per warp, three stages per warp.  Short rows are normally served by the warp kernel
// with several tokens per warp (6.0-6.5 TB/s against 5.6-6.0 TB/s here); this path remains for
// QKNORM_FORCE_VARIANT=tile and for shapes the warp kernel has no instantiation for.  Returns
// QKNORM_OK with *done = false when the call is not of that kind.
int launch_tile(const Params& P, const DeviceInfo& dev, cudaStream_t stream, bool* done) {
  *done = false;
  if (P.S != 1) return QKNORM_OK;
  const int row_bytes = (P.q.d + P.k.d) * P.elem_bytes;
  const int limit = env_int("QKNORM_TILE_MAX_ROW_BYTES", P.elem_bytes == 1 ? 4096 : 2816);
  if (row_bytes > limit) return QKNORM_OK;
  TpParams T;
  memset(&T, 0, sizeof(T));
  T.n_local = 1;
  T.N = 1;
  T.T = P.T;
  T.cap = P.T;
  T.wq = P.q.d;
  T.wk = P.k.d;
  T.ldxq = P.q.ldx;
  T.ldxk = P.k.ldx;
  T.ldyq = P.q.ldy;
  T.ldyk = P.k.ldy;
  T.inv_dq = P.q.inv_d;
  T.inv_dk = P.k.inv_d;
  T.eps = P.eps;
  T.epoch = 1u;  // no peer, nothing is ever polled
  T.wait_ns = 1000000000ull;
  TpRank& r = T.r[0];
  r.rank = 0;
  r.xq = P.q.x[0];
  r.xk = P.k.x[0];
  r.gq = P.q.gamma[0];
  r.gk = P.k.gamma[0];
  r.yq = P.q.y[0];
  r.yk = P.k.y[0];
  r.rstd_q = P.q.rstd;
  r.rstd_k = P.k.rstd;
  r.partial_q = P.q.partials;  // with one slice the slice's scalar is the row's
  r.partial_k = P.k.partials;
  r.inbox = reinterpret_cast<unsigned long long*>(dev.ring_error);  // only its status words are used
  int warps = 0, smem = 0;
  TpKernel fn = nullptr;
  int rc = tp_configure(T, P.elem_bytes, dev.sm_count, &warps, &smem, &fn);
  if (rc != QKNORM_OK) return QKNORM_OK;  // does not fit: another variant takes the call
  if (smem > dev.smem_per_block) return QKNORM_OK;
  rc = allow_dynamic_smem((const void*)fn, smem);
  if (rc != QKNORM_OK) return rc;
  int resident = 1;
  rc = resident_blocks((const void*)fn, warps * 32, smem, &resident);
  if (rc != QKNORM_OK) return rc;
  const int tile = 32 >> T.log_g;
  const long long tiles = (P.T + tile - 1) / tile;
  const long long needed = (tiles + warps - 1) / warps;
  long long grid = (long long)resident * dev.sm_count;  // bounded grid of co-resident CTAs
  if (grid > needed) grid = needed;
  fn<<<(unsigned)grid, warps * 32, smem, stream>>>(T);
  rc = finish_launch("tile");
  *done = rc == QKNORM_OK;
  return rc;
}

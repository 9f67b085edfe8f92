// C ABI of libqknorm: argument validation, variant choice, launch.
// No forward entry point allocates device memory, copies, or synchronises (the inbox
// helpers of the tensor-parallel path, qknorm_tp_host.cuh, are the only routines that do).
#include <cuda_runtime.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "../../include/qknorm.h"
#include "qknorm_baselines.cuh"
#include "qknorm_general.cuh"
#include "qknorm_head.cuh"
#include "qknorm_params.h"
#include "qknorm_ring.cuh"
#include "qknorm_rows.cuh"
#include "../../include/qknorm_tp.h"
#include "qknorm_tp.cuh"
#include "qknorm_warp.cuh"

namespace qknorm {

// per-N factories, defined in qknorm_rows_inst.cu (one translation unit per N)
#define QKNORM_DECL_N(n)                       \
  RowsKernel rows_kernel_n##n(int elem_bytes); \
  RingKernel ring_kernel_n##n();
QKNORM_DECL_N(1) QKNORM_DECL_N(2) QKNORM_DECL_N(3) QKNORM_DECL_N(4) QKNORM_DECL_N(6) QKNORM_DECL_N(8)

RowsKernel rows_kernel_for(int n, int elem_bytes) {
  switch (n) {
    case 1: return rows_kernel_n1(elem_bytes);
    case 2: return rows_kernel_n2(elem_bytes);
    case 3: return rows_kernel_n3(elem_bytes);
    case 4: return rows_kernel_n4(elem_bytes);
    case 6: return rows_kernel_n6(elem_bytes);
    case 8: return rows_kernel_n8(elem_bytes);
    default: return nullptr;
  }
}

RingKernel ring_kernel_for(int n) {
  switch (n) {
    case 1: return ring_kernel_n1();
    case 2: return ring_kernel_n2();
    case 3: return ring_kernel_n3();
    case 4: return ring_kernel_n4();
    case 6: return ring_kernel_n6();
    case 8: return ring_kernel_n8();
    default: return nullptr;
  }
}

// per-(L, format) factories, defined in qknorm_warp_inst.cu (one translation unit each)
#define QKNORM_DECL_L(l)                     \
  WarpKernel warp_kernel_bf16_l##l(bool exact); \
  WarpKernel warp_kernel_e4m3_l##l(bool exact);
QKNORM_DECL_L(4) QKNORM_DECL_L(8) QKNORM_DECL_L(12) QKNORM_DECL_L(16) QKNORM_DECL_L(20)
QKNORM_DECL_L(24) QKNORM_DECL_L(28) QKNORM_DECL_L(32) QKNORM_DECL_L(36) QKNORM_DECL_L(40)

int warp_round_up_l(int n) {
  if (n < 1 || n > 40) return -1;
  return ((n + 3) / 4) * 4;
}

WarpKernel warp_kernel_for(int l, bool exact, int elem_bytes) {
#define QKNORM_CASE_L(l) \
  case l: return elem_bytes == 1 ? warp_kernel_e4m3_l##l(exact) : warp_kernel_bf16_l##l(exact);
  switch (l) {
    QKNORM_CASE_L(4) QKNORM_CASE_L(8) QKNORM_CASE_L(12) QKNORM_CASE_L(16) QKNORM_CASE_L(20)
    QKNORM_CASE_L(24) QKNORM_CASE_L(28) QKNORM_CASE_L(32) QKNORM_CASE_L(36) QKNORM_CASE_L(40)
    default: return nullptr;
  }
#undef QKNORM_CASE_L
}

// Set by a ring kernel whose bounded wait ran out (0 = never happened).
__device__ __align__(8) int g_ring_error[8] = {0, 0, 0, 0, 0, 0, 0, 0};  // word 0 is the error word; 1-2: where it happened

// Token queues of the warp-per-token kernel: two 64-bit words per slot (tokens handed out, warps
// gone), zero between launches.  A slot belongs to one stream of one device, and kernels of one
// stream never run at the same time, so no two launches in flight share a slot.
constexpr int kQueueSlots = 256;
__device__ __align__(16) unsigned long long g_token_queue[kQueueSlots][2];

// Built-in scratch of qknorm_baseline_two_pass_static: 1 MiB of device memory that every
// GPU which loads this library holds until the process exits.  In host code this name is
// only a handle for cudaGetSymbolAddress, never a device address.
constexpr size_t kStaticScratchFloats = 262144;
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];


namespace {

thread_local int tl_cuda_error = 0;
thread_local const char* tl_variant = "none";
thread_local long long tl_launches = 0;

struct DeviceInfo {
  bool known = false;
  int index = 0;
  int sm_count = 0;
  int smem_per_sm = 0;       // bytes
  int smem_per_block = 0;    // opt-in maximum, bytes
  int* ring_error = nullptr; // device address of g_ring_error on this device
  unsigned long long* token_queue = nullptr;  // device address of g_token_queue on this device
  // which stream owns which queue slot (slot i belongs to queue_stream[i]); guarded by g_devices_mutex
  cudaStream_t queue_stream[kQueueSlots];
  int queue_slots_used = 0;
};
constexpr int kMaxDevices = 64;
DeviceInfo g_devices[kMaxDevices];
std::mutex g_devices_mutex;

int set_cuda_error(cudaError_t e) {
  tl_cuda_error = (int)e;
  return QKNORM_ERR_CUDA;
}

// Facts about the current device, cached.
int current_device(const DeviceInfo** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevices) return set_cuda_error(cudaErrorInvalidDevice);
  std::lock_guard<std::mutex> lock(g_devices_mutex);
  DeviceInfo& d = g_devices[dev];
  if (!d.known) {
    int n = 0;
    e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return set_cuda_error(e);
    d.sm_count = n;
    e = cudaDeviceGetAttribute(&d.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
    if (e != cudaSuccess) return set_cuda_error(e);
    e = cudaDeviceGetAttribute(&d.smem_per_block, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return set_cuda_error(e);
    // the symbol's name is only a host-side handle: ask for its address on this device
    e = cudaGetSymbolAddress((void**)&d.ring_error, g_ring_error);
    if (e != cudaSuccess) return set_cuda_error(e);
    e = cudaGetSymbolAddress((void**)&d.token_queue, g_token_queue);
    if (e != cudaSuccess) return set_cuda_error(e);
    d.index = dev;
    d.known = true;
  }
  *out = &d;
  return QKNORM_OK;
}

// The token queue a launch on `stream` may use, or nullptr when it has to keep the fixed schedule:
//  * a launch that is being captured into a CUDA graph (the graph can later be replayed on any
//    stream, next to anything), and the per-thread default stream handle (one handle, a different
//    stream in every host thread) get no queue;
//  * every other stream of a device gets a slot of its own the first time it is seen and keeps it
//    (a destroyed stream's handle may come back as a new stream: still one stream at a time);
//  * when all slots are taken, further streams get none.
// The legacy default stream has two handles (0 and cudaStreamLegacy); both map to one slot.
int token_queue_for(int dev_index, cudaStream_t stream, unsigned long long** out) {
  *out = nullptr;
  if (stream == cudaStreamPerThread) return QKNORM_OK;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  cudaError_t e = cudaStreamIsCapturing(stream, &cap);
  if (e != cudaSuccess) return set_cuda_error(e);
  if (cap != cudaStreamCaptureStatusNone) return QKNORM_OK;
  if (stream == cudaStreamLegacy) stream = nullptr;
  std::lock_guard<std::mutex> lock(g_devices_mutex);
  DeviceInfo& d = g_devices[dev_index];
  int slot = -1;
  for (int i = 0; i < d.queue_slots_used; ++i)
    if (d.queue_stream[i] == stream) { slot = i; break; }
  if (slot < 0 && d.queue_slots_used < kQueueSlots) {
    slot = d.queue_slots_used++;
    d.queue_stream[slot] = stream;
  }
  if (slot >= 0) *out = d.token_queue + 2 * (size_t)slot;
  return QKNORM_OK;
}

// A buffer of the call: `rows` rows of `row_bytes` bytes, `pitch` bytes apart.
struct Region {
  uintptr_t base;
  uintptr_t rows, row_bytes, pitch;
  uintptr_t end() const { return base + (rows - 1) * pitch + row_bytes; }
};

// Conservative: true unless the two regions are certainly disjoint.  Strided views
// that interleave (the Q and K columns of one fused QKV buffer) are disjoint when
// they share the pitch and their column intervals inside a row do not meet.
bool may_overlap(const Region& a, const Region& b) {
  if (a.rows == 0 || b.rows == 0 || a.row_bytes == 0 || b.row_bytes == 0) return false;
  if (a.base >= b.end() || b.base >= a.end()) return false;
  if (a.pitch == b.pitch && a.pitch > 0 && a.row_bytes <= a.pitch && b.row_bytes <= b.pitch) {
    const uintptr_t p = a.pitch;
    const uintptr_t delta = b.base >= a.base ? (b.base - a.base) % p : (p - (a.base - b.base) % p) % p;
    // inside one period a covers [0, a.row_bytes), b covers [delta, delta + b.row_bytes)
    if (delta >= a.row_bytes && delta + b.row_bytes <= p) return false;
  }
  return true;
}

inline bool same_region(const Region& a, const Region& b) {
  return a.base == b.base && a.row_bytes == b.row_bytes && (a.rows <= 1 || a.pitch == b.pitch);
}

// Every output against every other buffer of the call.  An output may be exactly
// its own input (in place); anything else that may overlap is an error.
int check_alias(const Params& P, int64_t T, int rstd_per_token_q = 1, int rstd_per_token_k = 1) {
  Region in[2 * kMaxShards], gm[2 * kMaxShards], out[2 * kMaxShards], aux[4];
  int n = 0, naux = 0;
  const TensorArgs* ts[2] = {&P.q, &P.k};
  const uintptr_t rows = (uintptr_t)T, eb = (uintptr_t)P.elem_bytes;
  for (const TensorArgs* a : ts) {
    if (a->d == 0) continue;
    const uintptr_t row_bytes = (uintptr_t)a->w * eb;
    for (int s = 0; s < P.S; ++s) {
      in[n] = {(uintptr_t)a->x[s], rows, row_bytes, (uintptr_t)a->ldx * eb};
      gm[n] = {(uintptr_t)a->gamma[s], 1, (uintptr_t)a->w * 2u, (uintptr_t)a->w * 2u};
      out[n] = {(uintptr_t)a->y[s], rows, row_bytes, (uintptr_t)a->ldy * eb};
      ++n;
    }
    const uintptr_t rpt = (uintptr_t)(a == &P.q ? rstd_per_token_q : rstd_per_token_k);
    if (a->rstd) aux[naux++] = {(uintptr_t)a->rstd, 1, 4u * rows * rpt, 4u * rows * rpt};
    if (a->partials) aux[naux++] = {(uintptr_t)a->partials, 1, 4u * rows * (uintptr_t)P.S, 4u * rows * (uintptr_t)P.S};
  }
  for (int i = 0; i < n; ++i) {
    for (int j = 0; j < n; ++j) {
      if (may_overlap(out[i], gm[j])) return QKNORM_ERR_ALIAS;
      if (may_overlap(out[i], in[j]) && !(i == j && same_region(out[i], in[j]))) return QKNORM_ERR_ALIAS;
      if (j != i && may_overlap(out[i], out[j])) return QKNORM_ERR_ALIAS;
    }
    for (int j = 0; j < naux; ++j)
      if (may_overlap(out[i], aux[j])) return QKNORM_ERR_ALIAS;
  }
  for (int i = 0; i < naux; ++i) {
    for (int j = 0; j < n; ++j)
      if (may_overlap(aux[i], in[j]) || may_overlap(aux[i], gm[j])) return QKNORM_ERR_ALIAS;
    for (int j = i + 1; j < naux; ++j)
      if (may_overlap(aux[i], aux[j])) return QKNORM_ERR_ALIAS;
  }
  return QKNORM_OK;
}

inline bool aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }

bool vector_path_ok(const Params& P) {
  const TensorArgs* ts[2] = {&P.q, &P.k};
  for (const TensorArgs* a : ts) {
    if (a->d == 0) continue;
    if ((a->w * P.elem_bytes) % 16 != 0) return false;
    if ((a->ldx * P.elem_bytes) % 16 != 0 || (a->ldy * P.elem_bytes) % 16 != 0) return false;
    for (int s = 0; s < P.S; ++s)
      if (!aligned16(a->x[s]) || !aligned16(a->gamma[s]) || !aligned16(a->y[s])) return false;
  }
  return true;
}

// The experiment knobs (QKNORM_FORCE_VARIANT, QKNORM_WARPS, ...) are looked at only in a process that
// was started with QKNORM_DEBUG_ENV set: a production process makes no getenv call per launch and
// cannot be steered by a stray variable.
bool debug_env_enabled() {
  static const bool on = [] {
    const char* v = getenv("QKNORM_DEBUG_ENV");
    return v != nullptr && *v != '\0' && *v != '0';
  }();
  return on;
}

const char* env_str(const char* name) { return debug_env_enabled() ? getenv(name) : nullptr; }

int env_int(const char* name, int fallback) {
  const char* v = env_str(name);
  if (!v || !*v) return fallback;
  return atoi(v);
}

struct RowsPlan {
  int n = 0;        // 16-byte chunks per thread
  int threads = 0;  // CTA size
  int log_sub = 5;  // lane-group size (log2)
  int Gq = 0, Gk = 0;
};

inline int round_up(int v, int m) { return ((v + m - 1) / m) * m; }

// Thread layout of the vectorised kernels (qknorm_rowmap.cuh): N chunks per
// thread, G_q / G_k threads per Q / K slice, lane groups of 16 or 32.
//  throughput: wide CTAs with few chunks per thread (many warps hide the latency
//              of the per-token reduction), as few idle lanes as possible;
//  latency (few tokens): CTAs of about 256 threads; every load of a thread is issued
//              before the first use, so a few chunks per thread still cost one round trip.
bool plan_rows(const Params& P, bool latency, RowsPlan* plan) {
  const int cq = P.q.d ? P.q.w * P.elem_bytes / 16 : 0, ck = P.k.d ? P.k.w * P.elem_bytes / 16 : 0;
  const int force_n = env_int("QKNORM_FORCE_N", 0);
  const int force_sub = env_int("QKNORM_FORCE_SUB", 0);
  const int ns[] = {1, 2, 3, 4, 6, 8};
  double best_cost = 1e30;
  bool found = false;
  for (int n : ns) {
    if (force_n && n != force_n) continue;
    for (int log_sub = 5; log_sub >= 4; --log_sub) {
      const int sub = 1 << log_sub;
      if (force_sub && sub != force_sub) continue;
      const int Gq = cq ? round_up((cq + n - 1) / n, sub) : 0;
      const int Gk = ck ? round_up((ck + n - 1) / n, sub) : 0;
      const int threads = round_up(P.S * (Gq + Gk), 32);
      if (threads > max_threads_for(n)) continue;
      if (P.S * (Gq + Gk) / sub > kMaxSlots) continue;
      // Prefill (the rows too wide for the warp kernel): estimated warp instructions per token,
      // per chunk position ~45, per token and thread ~60 plus the slots it has to add up.
      // Decode sizes: measured under CUDA-graph replay, CTAs of about 256 threads with ~4
      // chunks per thread are fastest (2.4 us per call against 2.8-3.5 us for 1024-thread CTAs).
      const int warps = threads / 32;
      const int slots = P.S * (Gq > Gk ? Gq : Gk) / sub;
      double cost = latency ? (double)(threads > 256 ? threads - 256 : 256 - threads) + 0.1 * n
                            : (double)warps * (45.0 * n + 60.0 + 2.0 * slots);
      if (log_sub == 4) cost *= 1.001;  // tie: full-warp groups (fewer slots to add up)
      if (cost < best_cost) {
        best_cost = cost;
        plan->n = n;
        plan->threads = threads;
        plan->log_sub = log_sub;
        plan->Gq = Gq;
        plan->Gk = Gk;
        found = true;
      }
    }
  }
  return found;
}

void apply_plan(Params& P, const RowsPlan& plan) {
  P.log_sub = plan.log_sub;
  P.q.G = plan.Gq;
  P.q.first_thread = 0;
  P.k.G = plan.Gk;
  P.k.first_thread = P.S * plan.Gq;
}

struct OccKey {
  const void* fn;
  int threads;
  int smem;
  int dev;
  int blocks;
};
constexpr int kOccCache = 256;
OccKey g_occ[kOccCache];
int g_occ_n = 0;
std::mutex g_occ_mutex;

// Resident CTAs per SM for (kernel, CTA size) on the current device: B_res of Section III-D.
int resident_blocks(const void* fn, int threads, int smem, int* out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_cuda_error(e);
  std::lock_guard<std::mutex> lock(g_occ_mutex);
  for (int i = 0; i < g_occ_n; ++i)
    if (g_occ[i].fn == fn && g_occ[i].threads == threads && g_occ[i].smem == smem && g_occ[i].dev == dev) {
      *out = g_occ[i].blocks;
      return QKNORM_OK;
    }
  int blocks = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, fn, threads, smem);
  if (e != cudaSuccess) return set_cuda_error(e);
  if (blocks < 1) blocks = 1;
  if (g_occ_n < kOccCache) g_occ[g_occ_n++] = OccKey{fn, threads, smem, dev, blocks};
  *out = blocks;
  return QKNORM_OK;
}

// Largest dynamic shared memory a kernel has been allowed so far, per (kernel, device).
struct SmemKey {
  const void* fn;
  int dev;
  int bytes;
};
SmemKey g_smem[kOccCache];
int g_smem_n = 0;

int allow_dynamic_smem(const void* fn, int bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_cuda_error(e);
  std::lock_guard<std::mutex> lock(g_occ_mutex);
  for (int i = 0; i < g_smem_n; ++i)
    if (g_smem[i].fn == fn && g_smem[i].dev == dev) {
      if (g_smem[i].bytes >= bytes) return QKNORM_OK;
      e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
      if (e != cudaSuccess) return set_cuda_error(e);
      g_smem[i].bytes = bytes;
      return QKNORM_OK;
    }
  e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return set_cuda_error(e);
  if (g_smem_n < kOccCache) g_smem[g_smem_n++] = SmemKey{fn, dev, bytes};
  return QKNORM_OK;
}

int finish_launch(const char* variant) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error(e);
  tl_variant = variant;
  ++tl_launches;
  return QKNORM_OK;
}

// Launch with programmatic stream serialisation: the kernel may begin while the previous kernel of
// the stream is still running; the kernel itself waits for that kernel's completion
// (griddepcontrol.wait) before its first access to global memory.  QKNORM_PDL=0 (a debug knob)
// launches the plain way.
template <class... KArgs, class... Args>
cudaError_t launch_overlapped(void (*fn)(KArgs...), unsigned grid, unsigned threads, size_t smem, cudaStream_t stream,
                              Args... args) {
  if (!env_int("QKNORM_PDL", 1)) {
    fn<<<grid, threads, smem, stream>>>(args...);
    return cudaSuccess;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, fn, args...);
}

#include "qknorm_tp_host.cuh"  // run_tp, launch_tile

// The TMA ring kernel (prefill sizes).  Returns QKNORM_OK with *done = false when
// the shape does not fit it and another variant should run.
int launch_ring(Params& P, const DeviceInfo& dev, cudaStream_t stream, bool* done) {
  *done = false;
  RowsPlan plan;
  if (P.elem_bytes != 2) return QKNORM_OK;  // bf16 only
  if (!plan_rows(P, /*latency=*/false, &plan)) return QKNORM_OK;
  RingKernel fn = ring_kernel_for(plan.n);
  if (!fn) return QKNORM_OK;
  const int row_bytes = (P.q.d + P.k.d) * 2;
  const int stage_bytes = ((row_bytes + 16 + 127) / 128) * 128;  // the row, then >= 16 bytes of zeros
  // Split the SM's shared memory between `ctas` resident CTAs, each with as deep a ring as fits.
  int ctas = env_int("QKNORM_CTAS_PER_SM", 0);
  if (ctas < 1) {
    ctas = 2048 / plan.threads;  // as many as the SM's thread slots allow ...
    if (ctas > 3) ctas = 3;
    if (ctas < 1) ctas = 1;
  }
  const int reserve = 2048;  // static shared memory + the per-CTA system reservation
  int nst = 0;
  for (; ctas >= 1; --ctas) {   // ... as long as every CTA still gets a ring of >= 3 stages
    int budget = dev.smem_per_sm / ctas - reserve;
    if (budget > dev.smem_per_block - reserve) budget = dev.smem_per_block - reserve;
    nst = budget / stage_bytes;
    if (nst >= 3 || ctas == 1) break;
  }
  const int forced = env_int("QKNORM_RING_STAGES", 0);
  if (forced > 0 && forced < nst) nst = forced;
  if (nst > kRingMaxStages) nst = kRingMaxStages;
  if (nst < 2) return QKNORM_OK;
  const int smem = nst * stage_bytes;
  int rc = allow_dynamic_smem((const void*)fn, smem);
  if (rc != QKNORM_OK) return rc;
  int bres = 1;
  rc = resident_blocks((const void*)fn, plan.threads, smem, &bres);
  if (rc != QKNORM_OK) return rc;
  if (bres > ctas) bres = ctas;
  long long grid = (long long)bres * dev.sm_count;  // bounded grid of co-resident CTAs
  if (grid > P.T) grid = P.T;
  apply_plan(P, plan);
  fn<<<(unsigned)grid, plan.threads, smem, stream>>>(P, nst, stage_bytes, dev.ring_error);
  rc = finish_launch("ring");
  *done = rc == QKNORM_OK;
  return rc;
}

// Chunk slots per lane the warp-per-token kernel would need for this call.
int warp_slots_needed(const Params& P) {
  int log_g = 5;
  while ((P.S << log_g) > 32) --log_g;
  const int g = 1 << log_g;
  const int cq = P.q.d ? P.q.w * P.elem_bytes / 16 : 0, ck = P.k.d ? P.k.w * P.elem_bytes / 16 : 0;
  return round_up((cq + g - 1) / g, 4) + (ck + g - 1) / g;
}

// The warp-per-token kernel (prefill sizes, gathered rows of up to 40 chunks per lane).
int launch_warp(Params& P, const DeviceInfo& dev, cudaStream_t stream, bool* done, int tokens_per_warp = 1) {
  *done = false;
  if (tokens_per_warp > 1 && P.S != 1) return QKNORM_OK;  // tokens side by side only for unsharded rows
  const int groups = tokens_per_warp > 1 ? tokens_per_warp : P.S;  // lane groups: tokens of a tile, or slices
  int log_g = 5;
  while ((groups << log_g) > 32) --log_g;  // g = largest power of two <= 32 / groups
  const int g = 1 << log_g;
  const int cq = P.q.d ? P.q.w * P.elem_bytes / 16 : 0, ck = P.k.d ? P.k.w * P.elem_bytes / 16 : 0;
  WarpArgs wa;
  wa.log_g = log_g;
  wa.nq = (cq + g - 1) / g;
  wa.nk = (ck + g - 1) / g;
  wa.nq4 = round_up(wa.nq, 4);
  const int l = warp_round_up_l(wa.nq4 + wa.nk);
  if (l < 0) return QKNORM_OK;
  wa.tokens_per_warp = tokens_per_warp > 1 ? tokens_per_warp : 1;
  const long long units = (P.T + wa.tokens_per_warp - 1) / wa.tokens_per_warp;  // tokens, or tiles of tokens
  const bool exact = (groups << log_g) == 32 && cq % g == 0 && ck % g == 0 && wa.nq % 4 == 0 && wa.nk % 4 == 0 &&
                     P.T % wa.tokens_per_warp == 0;
  WarpKernel fn = warp_kernel_for(l, exact, P.elem_bytes);
  if (!fn) return QKNORM_OK;
  // stage layout: Q slices, K slices (each slice row followed by the bank skew), 16 zero bytes
  // rows of consecutive lane groups start g*16 bytes apart modulo 128, so that the groups that read
  // in the same quarter-warp hit different banks
  auto skew_for = [&](int row_bytes) { return (groups > 1 && g < 8) ? ((g * 16 - row_bytes % 128) % 128 + 128) % 128 : 0; };
  wa.q_slice_stride = cq ? P.q.w * P.elem_bytes + skew_for(P.q.w * P.elem_bytes) : 0;
  wa.k_slice_stride = ck ? P.k.w * P.elem_bytes + skew_for(P.k.w * P.elem_bytes) : 0;
  wa.k_base = groups * wa.q_slice_stride;
  wa.zero_off = wa.k_base + groups * wa.k_slice_stride;
  wa.stage_bytes = round_up(wa.zero_off + 16, 128);
  wa.error_word = dev.ring_error;
  wa.queue = nullptr;
  wa.stagger_cycles = env_int("QKNORM_STAGGER_CYCLES", 900);
  {
    const int qrc = token_queue_for(dev.index, stream, &wa.queue);
    if (qrc != QKNORM_OK) return qrc;
  }
  // One row per warp is always in flight.  Measured on B200: throughput peaks when
  // about 76 KB of rows are in flight per SM and falls off slowly beyond that.
  const int in_flight = 76 * 1024;  // holds for both storage formats (FP8 rows are half as long: twice the warps)
  int rule = (in_flight + wa.stage_bytes / 2) / wa.stage_bytes;
  if (rule < 2) rule = 2;
  // FP8 rows cost twice the instructions per byte and a short call is over before the steady state
  // counts: with fewer than 16 rounds of tokens, half as many warps again are faster (measured, warps
  // per SM: C3 as FP8 8 -> 12, 39.5 -> 37.6 us; C4 as FP8 12 -> 16, 46.4 -> 41.9 us; the 55 rounds of
  // C5 as FP8 stay fastest with 8).
  if (P.elem_bytes == 1 && (double)units < 16.0 * dev.sm_count * rule) rule = rule * 3 / 2;
  if (rule > 16) rule = 16;
  // Among the (CTAs per SM, warps per CTA) pairs near that, prefer one whose last round of
  // tokens is nearly full: with T / (148 * warps) rounds of several microseconds each, a
  // half-empty last round costs short calls more than a warp more or less does.
  const int static_smem = l * 512 * (P.elem_bytes == 1 ? 2 : 1) + 1024;  // gamma + barriers
  const int force_warps = env_int("QKNORM_WARPS", 0), force_ctas = env_int("QKNORM_CTAS_PER_SM", 0);
  int ctas_per_sm = 0, warps = 0;
  double best = -1.0;
  for (int w = 1; w <= kWarpMaxCtaWarps; ++w) {
    if (force_warps && w != force_warps) continue;
    const int smem_w = w * wa.stage_bytes;
    if (smem_w + static_smem > dev.smem_per_block) continue;
    int rc = allow_dynamic_smem((const void*)fn, smem_w);
    if (rc != QKNORM_OK) return rc;
    int resident = 1;
    rc = resident_blocks((const void*)fn, w * 32, smem_w, &resident);
    if (rc != QKNORM_OK) return rc;
    for (int c = 1; c <= resident && c <= 8; ++c) {
      if (force_ctas && c != force_ctas && !(force_ctas > resident && c == resident)) continue;
      const int per_sm = c * w;
      const double rounds = (double)units / ((double)dev.sm_count * per_sm);
      const double tail = rounds / (double)(long long)(rounds + 0.999999);
      const int away = per_sm > rule ? per_sm - rule : rule - per_sm;
      const double score = tail - 0.5 * away / rule - 0.001 * c;  // measured: 25 % off the rule costs ~10 %
      if (score > best) {
        best = score;
        ctas_per_sm = c;
        warps = w;
      }
    }
  }
  if (warps == 0) return QKNORM_OK;  // not even one stage fits: another variant takes the call
  // The token queue pays where a warp runs at the speed of its own memory round trips (measured on
  // bf16 rows of 8-20 KB with 4-8 warps per SM, and on FP8 rows with 4: 2-7 % faster).  FP8 rows with
  // eight or more warps per SM are bound by the SM's instruction issue; there the warps stay level by
  // themselves and the fixed schedule is 6-9 % faster, so those launches take no queue.
  const int want_queue = env_int("QKNORM_QUEUE", -1);
  // Tiles of tokens of at most 4 KB gain nothing either (2-6 % slower with the queue).
  if (want_queue == 0 || (want_queue < 0 && P.elem_bytes == 1 && ctas_per_sm * warps >= 8) ||
      (want_queue < 0 && wa.tokens_per_warp > 1 && wa.stage_bytes <= 4608))
    wa.queue = nullptr;
  // Shared memory per CTA: what the stages need, raised to the SM's share for `ctas_per_sm` CTAs, so
  // that one more CTA never fits.  An overlapped launch (the next call of the stream) then gets its
  // CTAs onto an SM only as this launch's CTAs leave it, exactly `ctas_per_sm` per SM; if an SM could
  // take more, the early leavers' SMs would fill up twice and others would stay empty.
  int smem = warps * wa.stage_bytes;
  {
    int share = dev.smem_per_sm / ctas_per_sm - 1024 - static_smem;  // 1 KB per CTA is the system's
    if (share > dev.smem_per_block - static_smem) share = dev.smem_per_block - static_smem;
    share &= ~127;
    if (share > smem && env_int("QKNORM_FILL_SMEM", 1)) {
      smem = share;
      const int rc2 = allow_dynamic_smem((const void*)fn, smem);
      if (rc2 != QKNORM_OK) return rc2;
    }
  }
  long long grid = (long long)ctas_per_sm * dev.sm_count;  // bounded grid of co-resident CTAs
  const long long needed = (units + warps - 1) / warps;
  if (grid > needed) grid = needed;
  int rc = QKNORM_OK;
  const cudaError_t e = launch_overlapped(fn, (unsigned)grid, (unsigned)warps * 32u, (size_t)smem, stream, P, wa);
  if (e != cudaSuccess) return set_cuda_error(e);
  rc = finish_launch("warp");
  *done = rc == QKNORM_OK;
  return rc;
}

int launch(Params& P, cudaStream_t stream) {
  const DeviceInfo* dev = nullptr;
  int rc = current_device(&dev);
  if (rc != QKNORM_OK) return rc;
  const int sms = dev->sm_count;
  const char* force = env_str("QKNORM_FORCE_VARIANT");
  const bool force_general = force && strcmp(force, "general") == 0;
  const bool force_rows = force && strcmp(force, "rows") == 0;
  const bool force_ring = force && strcmp(force, "ring") == 0;

  if (!force_general && vector_path_ok(P)) {
    const bool force_warp = force && strcmp(force, "warp") == 0;
    const bool force_tile = force && strcmp(force, "tile") == 0;
    // Which regime: the register-resident rows kernel (a CTA per token, nothing staged, no set-up
    // beyond gamma in registers) finishes a call of a thousand or two tokens in fewer microseconds
    // than the TMA-fed kernels need to get going.  Measured on B200 over row widths of 1 to 32 KB and
    // 1 to 16 slices, from L2 and from HBM: the crossover sits between 1000 and 2900 tokens, earlier
    // when the slices are many and narrow (CTAs of more than 384 threads).
    bool latency = P.T < 4LL * sms;
    if (!latency && !force_warp && !force_ring && !force_tile) {
      RowsPlan plan;
      if (plan_rows(P, /*latency=*/true, &plan)) {
        const long long most = env_int("QKNORM_ROWS_MAX_TOKENS", plan.threads <= 384 ? 2048 : 1280);
        if (P.T <= most) latency = true;
      }
    }
    if (!latency && !force_rows && !force_ring && P.S == 1) {
      // short unsharded rows: several tokens side by side per warp
      // Rows of a few KB and less: R consecutive tokens side by side per warp (2, 4 or 8 with a tile
      // of at most 9.5 KB; 16 for rows under 384 bytes), so that the per-token work of a warp (barrier
      // wait, copy issue, shuffle tree, rsqrt) is done once per tile.  Measured on 600 MB of rows of
      // 256-2560 bytes: 6.0-6.5 TB/s, against 5.6-6.0 TB/s for the three-stage tiled kernel and
      // 1.5-6.4 TB/s with one token per warp.
      int tpw = 1;
      const int row_bytes = (P.q.d + P.k.d) * P.elem_bytes;
      while (tpw < 8 && 2 * tpw * row_bytes <= 9728) tpw *= 2;
      if (row_bytes < 384) tpw = 16;
      tpw = env_int("QKNORM_TOKENS_PER_WARP", tpw);
      if (tpw > 16) tpw = 16;
      if (tpw > 1 && !force_tile) {
        bool done = false;
        rc = launch_warp(P, *dev, stream, &done, tpw);
        if (rc != QKNORM_OK || done) return rc;
      }
    }
    if (!latency && !force_rows && !force_ring && !force_warp) {
      bool done = false;
      rc = launch_tile(P, *dev, stream, &done);  // short unsharded rows: several tokens per warp
      if (rc != QKNORM_OK || done) return rc;
    }
    if (!latency && !force_rows && !force_ring) {
      bool done = false;
      rc = launch_warp(P, *dev, stream, &done);
      if (rc != QKNORM_OK || done) return rc;
    }
    // Rows too wide for the warp kernel, cut into 8 or more slices, K much narrower than Q (a large
    // GQA layer under 8-way tensor parallelism): the CTA-per-token layout spends a lane group on every
    // narrow K slice.  Q and K have independent statistics, so each gets its own launch -- Q on the
    // ring kernel, K on the warp kernel.  Measured (16384 + 2048 wide, 8 slices, 8138 tokens): 154 us
    // in one launch, 114 us in two.
    if (!latency && !force && P.q.d != 0 && P.k.d != 0 && P.S >= 8 && P.k.d * 4 <= P.q.d &&
        warp_round_up_l(warp_slots_needed(P)) < 0) {
      Params Q = P, K = P;
      memset(&Q.k, 0, sizeof(Q.k));
      memset(&K.q, 0, sizeof(K.q));
      rc = launch(Q, stream);
      if (rc != QKNORM_OK) return rc;
      return launch(K, stream);
    }
    if (!latency && !force_rows) {
      bool done = false;
      rc = launch_ring(P, *dev, stream, &done);
      if (rc != QKNORM_OK || done) return rc;
    }
    RowsPlan plan;
    if (plan_rows(P, latency, &plan)) {
      RowsKernel fn = rows_kernel_for(plan.n, P.elem_bytes);
      int bres = 1;
      rc = resident_blocks((const void*)fn, plan.threads, 0, &bres);
      if (rc != QKNORM_OK) return rc;
      const int cap = env_int("QKNORM_CTAS_PER_SM", 0);
      if (cap > 0 && cap < bres) bres = cap;
      long long grid = (long long)bres * sms;  // bounded grid of co-resident CTAs
      if (grid > P.T) grid = P.T;
      apply_plan(P, plan);
      const cudaError_t e = launch_overlapped(fn, (unsigned)grid, (unsigned)plan.threads, 0, stream, P);
      if (e != cudaSuccess) return set_cuda_error(e);
      return finish_launch("rows");
    }
    // Q and K together are too wide for one CTA's registers (more than 32768 elements): the two
    // statistics are independent, so each tensor gets its own launch if it fits alone.
    if (P.q.d != 0 && P.k.d != 0) {
      Params Q = P, K = P;
      memset(&Q.k, 0, sizeof(Q.k));
      memset(&K.q, 0, sizeof(K.q));
      RowsPlan pq, pk;
      if (plan_rows(Q, false, &pq) && plan_rows(K, false, &pk)) {
        rc = launch(Q, stream);
        if (rc != QKNORM_OK) return rc;
        return launch(K, stream);
      }
    }
    // a tensor beyond 32768 elements: the vectorised two-pass kernel
    {
      void (*wide)(const Params) = P.elem_bytes == 1 ? wide_kernel<IoE4m3> : wide_kernel<IoBf16>;
      int bres = 1;
      rc = resident_blocks((const void*)wide, kWideThreads, 0, &bres);
      if (rc != QKNORM_OK) return rc;
      long long grid = (long long)bres * sms;
      if (grid > 2 * P.T) grid = 2 * P.T;
      wide<<<(unsigned)grid, kWideThreads, 0, stream>>>(P);
      return finish_launch("wide");
    }
  }
  void (*gen)(const Params) = P.elem_bytes == 1 ? general_kernel<IoE4m3> : general_kernel<IoBf16>;
  int bres = 1;
  rc = resident_blocks((const void*)gen, kGeneralThreads, 0, &bres);
  if (rc != QKNORM_OK) return rc;
  long long grid = (long long)bres * sms;
  if (grid > 2 * P.T) grid = 2 * P.T;
  gen<<<(unsigned)grid, kGeneralThreads, 0, stream>>>(P);
  return finish_launch("general");
}

// Validation shared by the entry points: fills P; *empty = true when there is nothing to do.
// Pointer arrays are host arrays of S entries.
int prepare(Params& P, bool* empty, int elem_bytes, const void* const* q, const void* const* k, const void* const* gq, const void* const* gk,
        int32_t S, int64_t T, int32_t dq, int32_t dk, float eps, void* const* oq, void* const* ok,
        float* partials_q, float* partials_k, float* rstd_q, float* rstd_k,
        const int64_t* ld = nullptr /* {ld_q, ld_k, ld_out_q, ld_out_k}; 0 or NULL = contiguous rows */) {
  *empty = true;
  if (S < 1 || S > kMaxShards) return QKNORM_ERR_SHARDS;
  if (T < 0 || dq < 0 || dk < 0 || dq > kMaxDim || dk > kMaxDim) return QKNORM_ERR_SHAPE;
  if (dq % S != 0 || dk % S != 0) return QKNORM_ERR_SHAPE;
  if (!(eps >= 0.0f)) return QKNORM_ERR_EPS;  // also rejects NaN
  if (T == 0) return QKNORM_OK;
  if (dq == 0 && dk == 0) return QKNORM_ERR_SHAPE;
  if (dq > 0 && (!q || !gq || !oq)) return QKNORM_ERR_NULL;
  if (dk > 0 && (!k || !gk || !ok)) return QKNORM_ERR_NULL;

  memset(&P, 0, sizeof(P));
  P.T = T;
  P.S = S;
  P.eps = eps;
  P.log_sub = 5;
  P.elem_bytes = elem_bytes;
  struct Side {
    TensorArgs* a;
    const void* const* x;
    const void* const* g;
    void* const* y;
    int d;
    float* partials;
    float* rstd;
    int64_t ldx, ldy;
  } sides[2] = {{&P.q, q, gq, oq, dq, partials_q, rstd_q, ld ? ld[0] : 0, ld ? ld[2] : 0},
                {&P.k, k, gk, ok, dk, partials_k, rstd_k, ld ? ld[1] : 0, ld ? ld[3] : 0}};
  for (Side& sd : sides) {
    sd.a->d = sd.d;
    sd.a->w = sd.d / S;
    sd.a->inv_d = sd.d ? 1.0f / (float)sd.d : 0.0f;
    sd.a->ldx = sd.ldx ? sd.ldx : sd.a->w;
    sd.a->ldy = sd.ldy ? sd.ldy : sd.a->w;
    if (sd.d == 0) continue;
    if (sd.a->ldx < sd.a->w || sd.a->ldy < sd.a->w) return QKNORM_ERR_SHAPE;  // rows would overlap
    for (int s = 0; s < S; ++s) {
      if (!sd.x[s] || !sd.g[s] || !sd.y[s]) return QKNORM_ERR_NULL;
      if (((uintptr_t)sd.g[s]) & 1u) return QKNORM_ERR_ALIGN;
      if (elem_bytes == 2 && ((((uintptr_t)sd.x[s]) | ((uintptr_t)sd.y[s])) & 1u)) return QKNORM_ERR_ALIGN;
      sd.a->x[s] = sd.x[s];
      sd.a->gamma[s] = (const uint16_t*)sd.g[s];
      sd.a->y[s] = sd.y[s];
    }
    if ((((uintptr_t)sd.partials) | ((uintptr_t)sd.rstd)) & 3u) return QKNORM_ERR_ALIGN;
    sd.a->partials = sd.partials;
    sd.a->rstd = sd.rstd;
  }
  int rc = check_alias(P, T);
  if (rc != QKNORM_OK) return rc;
  *empty = false;
  return QKNORM_OK;
}

// The fused path: validate, then one launch.
int run(int elem_bytes, const void* const* q, const void* const* k, const void* const* gq, const void* const* gk,
        int32_t S, int64_t T, int32_t dq, int32_t dk, float eps, void* const* oq, void* const* ok,
        float* partials_q, float* partials_k, float* rstd_q, float* rstd_k, void* stream,
        const int64_t* ld = nullptr) {
  Params P;
  bool empty = true;
  const int rc = prepare(P, &empty, elem_bytes, q, k, gq, gk, S, T, dq, dk, eps, oq, ok, partials_q, partials_k,
                         rstd_q, rstd_k, ld);
  if (rc != QKNORM_OK || empty) return rc;
  return launch(P, (cudaStream_t)stream);
}

// A scratch buffer must be non-NULL, aligned, large enough and away from every buffer of the call.
int check_scratch(const Params& P, const void* scratch, size_t have, size_t need, size_t align) {
  if (!scratch || have < need || (((uintptr_t)scratch) & (align - 1)) != 0) return QKNORM_ERR_SCRATCH;
  const Region sc = {(uintptr_t)scratch, 1, (uintptr_t)need, (uintptr_t)need};
  const TensorArgs* ts[2] = {&P.q, &P.k};
  const uintptr_t rows = (uintptr_t)P.T, eb = (uintptr_t)P.elem_bytes;
  for (const TensorArgs* a : ts) {
    if (a->d == 0) continue;
    for (int s = 0; s < P.S; ++s) {
      const Region in = {(uintptr_t)a->x[s], rows, (uintptr_t)a->w * eb, (uintptr_t)a->ldx * eb};
      const Region out = {(uintptr_t)a->y[s], rows, (uintptr_t)a->w * eb, (uintptr_t)a->ldy * eb};
      const Region gm = {(uintptr_t)a->gamma[s], 1, (uintptr_t)a->w * 2u, (uintptr_t)a->w * 2u};
      if (may_overlap(sc, in) || may_overlap(sc, out) || may_overlap(sc, gm)) return QKNORM_ERR_SCRATCH;
    }
    if (a->rstd && may_overlap(sc, Region{(uintptr_t)a->rstd, 1, 4u * rows, 4u * rows})) return QKNORM_ERR_SCRATCH;
    if (a->partials) {
      const uintptr_t n = 4u * rows * (uintptr_t)P.S;
      if (may_overlap(sc, Region{(uintptr_t)a->partials, 1, n, n})) return QKNORM_ERR_SCRATCH;
    }
  }
  return QKNORM_OK;
}

template <class K, class... Args>
int launch_simple(K kernel, int threads, long long work_items, const DeviceInfo& dev, cudaStream_t stream,
                  const char* variant, Args... args) {
  int bres = 1;
  int rc = resident_blocks((const void*)kernel, threads, 0, &bres);
  if (rc != QKNORM_OK) return rc;
  long long grid = (long long)bres * dev.sm_count;
  if (grid > work_items) grid = work_items;
  if (grid < 1) grid = 1;
  kernel<<<(unsigned)grid, threads, 0, stream>>>(args...);
  return finish_launch(variant);
}

// Baseline stand-in 1: copy the slices side by side into `scratch` (full rows), then normalise from there.
int run_gather_then_norm(Params& P, void* scratch, size_t scratch_bytes, cudaStream_t stream) {
  const size_t need = (size_t)P.T * ((size_t)P.q.d + (size_t)P.k.d) * (size_t)P.elem_bytes;
  int rc = check_scratch(P, scratch, scratch_bytes, need, 16);
  if (rc != QKNORM_OK) return rc;
  const DeviceInfo* dev = nullptr;
  rc = current_device(&dev);
  if (rc != QKNORM_OK) return rc;
  const bool vec = vector_path_ok(P);
  const long long units = (long long)(need / (vec ? 16 : 1));
  const long long ctas = (units + kBaselineThreads - 1) / kBaselineThreads;
  rc = vec ? launch_simple(gather_kernel<true>, kBaselineThreads, ctas, *dev, stream, "gather", P, (unsigned char*)scratch)
           : launch_simple(gather_kernel<false>, kBaselineThreads, ctas, *dev, stream, "gather", P, (unsigned char*)scratch);
  if (rc != QKNORM_OK) return rc;
  // the normalisation reads the gathered rows: slice s of a tensor is a column block of the scratch
  Params G = P;
  const long long pitch = (long long)P.q.d + P.k.d;  // elements
  unsigned char* base = (unsigned char*)scratch;
  for (int s = 0; s < P.S; ++s) {
    if (P.q.d) G.q.x[s] = base + (size_t)s * P.q.w * P.elem_bytes;
    if (P.k.d) G.k.x[s] = base + ((size_t)P.q.d + (size_t)s * P.k.w) * P.elem_bytes;
  }
  G.q.ldx = G.k.ldx = pitch;
  return launch(G, stream);
}

// Baseline stand-in 2: a statistics pass that writes every slice's scalar to `scratch`, then a scale pass.
int run_two_pass(Params& P, float* scratch, cudaStream_t stream) {
  const DeviceInfo* dev = nullptr;
  int rc = current_device(&dev);
  if (rc != QKNORM_OK) return rc;
  const bool vec = vector_path_ok(P);
  const long long items = P.T * 2 * P.S;
  const long long ctas = (items + kBaselineThreads / 32 - 1) / (kBaselineThreads / 32);
  rc = vec ? launch_simple(stat_kernel<IoBf16, true>, kBaselineThreads, ctas, *dev, stream, "two_pass", P, scratch)
           : launch_simple(stat_kernel<IoBf16, false>, kBaselineThreads, ctas, *dev, stream, "two_pass", P, scratch);
  if (rc != QKNORM_OK) return rc;
  return vec ? launch_simple(scale_kernel<IoBf16, true>, kBaselineThreads, ctas, *dev, stream, "two_pass", P,
                             (const float*)scratch)
             : launch_simple(scale_kernel<IoBf16, false>, kBaselineThreads, ctas, *dev, stream, "two_pass", P,
                             (const float*)scratch);
}

// Headwise granularity: every head of head_dim columns on its own.  The tensors come as S column
// slices (S = 1: whole rows, optional strides); a head never straddles a slice, so the slices are
// independent and one launch serves them all.
int run_headwise(int elem_bytes, const void* const* q, const void* const* k, const void* const* gq,
                 const void* const* gk, int32_t S, int64_t T, int32_t dq, int32_t dk, int32_t head_dim,
                 const int64_t* ld, float eps, void* const* oq, void* const* ok, float* rstd_q, float* rstd_k,
                 void* stream) {
  if (S < 1 || S > kMaxShards) return QKNORM_ERR_SHARDS;
  if (T < 0 || dq < 0 || dk < 0 || dq > kMaxDim || dk > kMaxDim) return QKNORM_ERR_SHAPE;
  if (dq % S != 0 || dk % S != 0) return QKNORM_ERR_SHAPE;
  if (head_dim < 1 || (dq / S) % head_dim != 0 || (dk / S) % head_dim != 0) return QKNORM_ERR_HEADS;
  if (ld)
    for (int i = 0; i < 4; ++i)
      if (ld[i] < 0) return QKNORM_ERR_SHAPE;
  // pointers, widths, strides and the alias rules are those of the layerwise call on the same buffers
  Params P;
  bool empty = true;
  int rc = prepare(P, &empty, elem_bytes, q, k, gq, gk, S, T, dq, dk, eps, oq, ok, nullptr, nullptr, nullptr, nullptr, ld);
  if (rc != QKNORM_OK || empty) return rc;
  if ((((uintptr_t)rstd_q) | ((uintptr_t)rstd_k)) & 3u) return QKNORM_ERR_ALIGN;
  P.q.rstd = dq ? rstd_q : nullptr;
  P.k.rstd = dk ? rstd_k : nullptr;
  rc = check_alias(P, T, dq ? dq / head_dim : 1, dk ? dk / head_dim : 1);
  if (rc != QKNORM_OK) return rc;

  const DeviceInfo* dev = nullptr;
  rc = current_device(&dev);
  if (rc != QKNORM_OK) return rc;
  HeadParams H;
  memset(&H, 0, sizeof(H));
  H.T = T;
  H.head_dim = head_dim;
  H.inv_hd = 1.0f / (float)head_dim;
  H.eps = eps;
  HeadSide* hs[2] = {&H.q, &H.k};
  const TensorArgs* ts[2] = {&P.q, &P.k};
  for (int i = 0; i < 2; ++i) {
    if (ts[i]->d == 0) continue;
    for (int sidx = 0; sidx < S; ++sidx) {
      hs[i]->x[sidx] = ts[i]->x[sidx];
      hs[i]->gamma[sidx] = ts[i]->gamma[sidx];
      hs[i]->y[sidx] = ts[i]->y[sidx];
    }
    hs[i]->rstd = ts[i]->rstd;
    hs[i]->ldx = ts[i]->ldx * elem_bytes;
    hs[i]->ldy = ts[i]->ldy * elem_bytes;
    hs[i]->nh = ts[i]->w / head_dim;
    hs[i]->heads = hs[i]->nh * S;
    hs[i]->inv_nh = 1.0f / (float)hs[i]->nh;
  }
  const char* force = env_str("QKNORM_FORCE_VARIANT");
  const int head_bytes = head_dim * elem_bytes;
  const bool vec = !(force && strcmp(force, "general") == 0) && head_bytes % 16 == 0 && head_bytes <= 512 && vector_path_ok(P);
  const bool fp8 = elem_bytes == 1;
  if (vec) {
    H.hc = head_bytes / 16;
    H.log_lph = 0;
    while ((1 << H.log_lph) < H.hc) ++H.log_lph;
    void (*fn)(const HeadParams) = fp8 ? head_kernel<4, IoE4m3> : head_kernel<4, IoBf16>;
    int bres = 1;
    rc = resident_blocks((const void*)fn, kHeadThreads, 0, &bres);
    if (rc != QKNORM_OK) return rc;
    long long grid = (long long)bres * dev->sm_count;
    const long long needed = (T + kHeadThreads / 32 - 1) / (kHeadThreads / 32);
    if (grid > needed) grid = needed;
    fn<<<(unsigned)grid, kHeadThreads, 0, (cudaStream_t)stream>>>(H);
    return finish_launch("head");
  }
  void (*gen)(const HeadParams) = fp8 ? head_general_kernel<IoE4m3> : head_general_kernel<IoBf16>;
  int bres = 1;
  rc = resident_blocks((const void*)gen, kHeadThreads, 0, &bres);
  if (rc != QKNORM_OK) return rc;
  long long grid = (long long)bres * dev->sm_count;
  const long long items = T * (H.q.heads + H.k.heads);
  const long long needed = (items + kHeadThreads / 32 - 1) / (kHeadThreads / 32);
  if (grid > needed) grid = needed;
  gen<<<(unsigned)grid, kHeadThreads, 0, (cudaStream_t)stream>>>(H);
  return finish_launch("head_general");
}

// Device address of g_static_scratch on the current device, looked up once per device.
float* g_static_scratch_addr[kMaxDevices];
bool g_static_scratch_known[kMaxDevices];
std::mutex g_static_scratch_mutex;

int static_scratch_address(float** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevices) return set_cuda_error(cudaErrorInvalidDevice);
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_known[dev]) {
    float* p = nullptr;
    // `dev` is the current device, so this is the address of ITS copy of the array
    e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
    if (e != cudaSuccess) return set_cuda_error(e);
    g_static_scratch_addr[dev] = p;
    g_static_scratch_known[dev] = true;
  }
  *out = g_static_scratch_addr[dev];
  return QKNORM_OK;
}

}  // namespace
}  // namespace qknorm

#include "qknorm_tp_abi.cuh"  // the tensor-parallel entry points (include/qknorm_tp.h)

extern "C" {

int qknorm_fwd(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
               int32_t dq, int32_t dk, float eps, void* out_q, void* out_k, void* stream) {
  return qknorm::run(2, &q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, eps, &out_q, &out_k, nullptr, nullptr,
                     nullptr, nullptr, stream);
}

int qknorm_fwd_ex(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
                  int32_t dq, int32_t dk, float eps, void* out_q, void* out_k, float* rstd_q, float* rstd_k,
                  void* stream) {
  return qknorm::run(2, &q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, eps, &out_q, &out_k, nullptr, nullptr,
                     rstd_q, rstd_k, stream);
}

int qknorm_fwd_sharded(const void* const* q_shards, const void* const* k_shards,
                       const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                       int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                       void* const* out_q_shards, void* const* out_k_shards, void* stream) {
  return qknorm::run(2, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq, dk, eps,
                     out_q_shards, out_k_shards, nullptr, nullptr, nullptr, nullptr, stream);
}

int qknorm_fwd_sharded_ex(const void* const* q_shards, const void* const* k_shards,
                          const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                          int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                          void* const* out_q_shards, void* const* out_k_shards, float* partials_q,
                          float* partials_k, float* rstd_q, float* rstd_k, void* stream) {
  return qknorm::run(2, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq, dk, eps,
                     out_q_shards, out_k_shards, partials_q, partials_k, rstd_q, rstd_k, stream);
}

int qknorm_baseline_gather_then_norm(const void* const* q_shards, const void* const* k_shards,
                                     const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                     int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                                     void* const* out_q_shards, void* const* out_k_shards, void* scratch,
                                     size_t scratch_bytes, void* stream) {
  qknorm::Params P;
  bool empty = true;
  const int rc = qknorm::prepare(P, &empty, 2, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens,
                                 dq, dk, eps, out_q_shards, out_k_shards, nullptr, nullptr, nullptr, nullptr);
  if (rc != QKNORM_OK || empty) return rc;
  return qknorm::run_gather_then_norm(P, scratch, scratch_bytes, (cudaStream_t)stream);
}

int qknorm_baseline_two_pass(const void* const* q_shards, const void* const* k_shards,
                             const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                             int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                             void* const* out_q_shards, void* const* out_k_shards, float* scratch,
                             size_t scratch_bytes, void* stream) {
  qknorm::Params P;
  bool empty = true;
  int rc = qknorm::prepare(P, &empty, 2, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq,
                           dk, eps, out_q_shards, out_k_shards, nullptr, nullptr, nullptr, nullptr);
  if (rc != QKNORM_OK || empty) return rc;
  const size_t need = (size_t)2 * (size_t)num_shards * (size_t)tokens * sizeof(float);
  rc = qknorm::check_scratch(P, scratch, scratch_bytes, need, 4);
  if (rc != QKNORM_OK) return rc;
  return qknorm::run_two_pass(P, scratch, (cudaStream_t)stream);
}

int qknorm_baseline_two_pass_static(const void* const* q_shards, const void* const* k_shards,
                                    const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                    int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                                    void* const* out_q_shards, void* const* out_k_shards, void* stream) {
  qknorm::Params P;
  bool empty = true;
  int rc = qknorm::prepare(P, &empty, 2, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq,
                           dk, eps, out_q_shards, out_k_shards, nullptr, nullptr, nullptr, nullptr);
  if (rc != QKNORM_OK || empty) return rc;
  if ((uint64_t)2 * (uint64_t)num_shards * (uint64_t)tokens > (uint64_t)qknorm::kStaticScratchFloats)
    return QKNORM_ERR_STATIC_LIMIT;
  float* scratch = nullptr;
  rc = qknorm::static_scratch_address(&scratch);  // first call on a device: the one-time look-up
  if (rc != QKNORM_OK) return rc;
  // Nothing has to be cleared: pass 1 writes every element that pass 2 of the same call reads.
  return qknorm::run_two_pass(P, scratch, (cudaStream_t)stream);
}

int64_t qknorm_static_scratch_capacity(void) { return (int64_t)qknorm::kStaticScratchFloats; }

int qknorm_fwd_strided(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
                       int32_t dq, int32_t dk, int64_t ld_q, int64_t ld_k, float eps, void* out_q, void* out_k,
                       int64_t ld_out_q, int64_t ld_out_k, void* stream) {
  if (ld_q < 0 || ld_k < 0 || ld_out_q < 0 || ld_out_k < 0) return QKNORM_ERR_SHAPE;
  const int64_t ld[4] = {ld_q, ld_k, ld_out_q, ld_out_k};
  return qknorm::run(2, &q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, eps, &out_q, &out_k, nullptr, nullptr,
                     nullptr, nullptr, stream, ld);
}

int qknorm_fwd_strided_e4m3(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
                            int32_t dq, int32_t dk, int64_t ld_q, int64_t ld_k, float eps, void* out_q, void* out_k,
                            int64_t ld_out_q, int64_t ld_out_k, void* stream) {
  if (ld_q < 0 || ld_k < 0 || ld_out_q < 0 || ld_out_k < 0) return QKNORM_ERR_SHAPE;
  const int64_t ld[4] = {ld_q, ld_k, ld_out_q, ld_out_k};
  return qknorm::run(1, &q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, eps, &out_q, &out_k, nullptr, nullptr,
                     nullptr, nullptr, stream, ld);
}

int qknorm_fwd_headwise(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
                        int32_t dq, int32_t dk, int32_t head_dim, int64_t ld_q, int64_t ld_k, float eps,
                        void* out_q, void* out_k, int64_t ld_out_q, int64_t ld_out_k, float* rstd_q,
                        float* rstd_k, void* stream) {
  const int64_t ld[4] = {ld_q, ld_k, ld_out_q, ld_out_k};
  return qknorm::run_headwise(2, &q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, head_dim, ld, eps, &out_q, &out_k,
                              rstd_q, rstd_k, stream);
}

int qknorm_fwd_headwise_e4m3(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
                             int32_t dq, int32_t dk, int32_t head_dim, int64_t ld_q, int64_t ld_k, float eps,
                             void* out_q, void* out_k, int64_t ld_out_q, int64_t ld_out_k, float* rstd_q,
                             float* rstd_k, void* stream) {
  const int64_t ld[4] = {ld_q, ld_k, ld_out_q, ld_out_k};
  return qknorm::run_headwise(1, &q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, head_dim, ld, eps, &out_q, &out_k,
                              rstd_q, rstd_k, stream);
}

int qknorm_fwd_headwise_sharded(const void* const* q_shards, const void* const* k_shards,
                                const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, int32_t head_dim,
                                float eps, void* const* out_q_shards, void* const* out_k_shards, float* rstd_q,
                                float* rstd_k, void* stream) {
  return qknorm::run_headwise(2, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq, dk,
                              head_dim, nullptr, eps, out_q_shards, out_k_shards, rstd_q, rstd_k, stream);
}

int qknorm_fwd_headwise_sharded_e4m3(const void* const* q_shards, const void* const* k_shards,
                                     const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                     int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, int32_t head_dim,
                                     float eps, void* const* out_q_shards, void* const* out_k_shards,
                                     float* rstd_q, float* rstd_k, void* stream) {
  return qknorm::run_headwise(1, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq, dk,
                              head_dim, nullptr, eps, out_q_shards, out_k_shards, rstd_q, rstd_k, stream);
}

int qknorm_fwd_e4m3(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
                    int32_t dq, int32_t dk, float eps, void* out_q, void* out_k, float* rstd_q, float* rstd_k,
                    void* stream) {
  return qknorm::run(1, &q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, eps, &out_q, &out_k, nullptr, nullptr,
                     rstd_q, rstd_k, stream);
}

int qknorm_fwd_sharded_e4m3(const void* const* q_shards, const void* const* k_shards,
                            const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                            int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                            void* const* out_q_shards, void* const* out_k_shards, float* partials_q,
                            float* partials_k, float* rstd_q, float* rstd_k, void* stream) {
  return qknorm::run(1, q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq, dk, eps,
                     out_q_shards, out_k_shards, partials_q, partials_k, rstd_q, rstd_k, stream);
}

const char* qknorm_status_string(int status) {
  switch (status) {
    case QKNORM_OK: return "QKNORM_OK";
    case QKNORM_ERR_NULL: return "QKNORM_ERR_NULL: a required pointer is NULL";
    case QKNORM_ERR_SHAPE: return "QKNORM_ERR_SHAPE: bad token count or width, or width not divisible by num_shards";
    case QKNORM_ERR_ALIGN: return "QKNORM_ERR_ALIGN: pointer not aligned to its element size";
    case QKNORM_ERR_ALIAS: return "QKNORM_ERR_ALIAS: an output overlaps another buffer without being exactly its own input";
    case QKNORM_ERR_SHARDS: return "QKNORM_ERR_SHARDS: num_shards out of range";
    case QKNORM_ERR_EPS: return "QKNORM_ERR_EPS: eps is negative or NaN";
    case QKNORM_ERR_CUDA: return "QKNORM_ERR_CUDA: a CUDA call failed";
    case QKNORM_ERR_HEADS: return "QKNORM_ERR_HEADS: head_dim < 1 or does not divide the width";
    case QKNORM_ERR_SCRATCH: return "QKNORM_ERR_SCRATCH: scratch buffer missing, too small, misaligned or overlapping";
    case QKNORM_ERR_STATIC_LIMIT:
      return "QKNORM_ERR_STATIC_LIMIT: 2 * num_shards * tokens exceeds the 262144 floats of the built-in scratch array";
    default: return "unknown qknorm status";
  }
}

int qknorm_device_error_word(int* out) {
  if (!out) return QKNORM_ERR_NULL;
  cudaError_t e = cudaMemcpyFromSymbol(out, qknorm::g_ring_error, sizeof(int));
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

int qknorm_last_cuda_error(void) { return qknorm::tl_cuda_error; }
const char* qknorm_last_variant(void) { return qknorm::tl_variant; }
int64_t qknorm_launch_count(void) { return qknorm::tl_launches; }
int qknorm_version(void) { return 100; }

}  // extern "C"

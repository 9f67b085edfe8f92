// C ABI of libqknorm: argument validation, variant choice, launch.
// Nothing here allocates device memory, copies, or synchronises.
#include <cuda_runtime.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "../../include/qknorm.h"
#include "qknorm_general.cuh"
#include "qknorm_params.h"
#include "qknorm_rows.cuh"

namespace qknorm {

// per-NQ factories, defined in qknorm_rows_inst.cu
#define QKNORM_DECL_TP(n) RowsKernel rows_throughput_nq##n(int nk);
#define QKNORM_DECL_LAT(n) RowsKernel rows_latency_nq##n(int nk);
QKNORM_DECL_TP(0) QKNORM_DECL_TP(1) QKNORM_DECL_TP(2) QKNORM_DECL_TP(3)
QKNORM_DECL_TP(4) QKNORM_DECL_TP(5) QKNORM_DECL_TP(6) QKNORM_DECL_TP(8)
QKNORM_DECL_LAT(0) QKNORM_DECL_LAT(1) QKNORM_DECL_LAT(2) QKNORM_DECL_LAT(4)

RowsKernel rows_kernel_throughput(int nq, int nk) {
  switch (nq) {
    case 0: return rows_throughput_nq0(nk);
    case 1: return rows_throughput_nq1(nk);
    case 2: return rows_throughput_nq2(nk);
    case 3: return rows_throughput_nq3(nk);
    case 4: return rows_throughput_nq4(nk);
    case 5: return rows_throughput_nq5(nk);
    case 6: return rows_throughput_nq6(nk);
    case 8: return rows_throughput_nq8(nk);
    default: return nullptr;
  }
}

RowsKernel rows_kernel_latency(int nq, int nk) {
  switch (nq) {
    case 0: return rows_latency_nq0(nk);
    case 1: return rows_latency_nq1(nk);
    case 2: return rows_latency_nq2(nk);
    case 4: return rows_latency_nq4(nk);
    default: return nullptr;
  }
}

namespace {

thread_local int tl_cuda_error = 0;
thread_local const char* tl_variant = "none";
thread_local long long tl_launches = 0;

struct DeviceInfo {
  bool known = false;
  int sm_count = 0;
};
constexpr int kMaxDevices = 64;
DeviceInfo g_devices[kMaxDevices];
std::mutex g_devices_mutex;

int set_cuda_error(cudaError_t e) {
  tl_cuda_error = (int)e;
  return QKNORM_ERR_CUDA;
}

// SM count of the current device, cached.
int current_sm_count(int* out) {
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
    d.known = true;
  }
  *out = d.sm_count;
  return QKNORM_OK;
}

struct Range {
  uintptr_t lo, hi;  // [lo, hi)
};
inline bool overlaps(const Range& a, const Range& b) { return a.lo < b.hi && b.lo < a.hi; }

// Every output range against every other range of the call.  An output may be
// identical to its own input (same index in `in`); anything else is an error.
int check_alias(const Params& P, int64_t T) {
  Range in[2 * kMaxShards], gm[2 * kMaxShards], out[2 * kMaxShards], aux[4];
  int n = 0, naux = 0;
  const TensorArgs* ts[2] = {&P.q, &P.k};
  for (const TensorArgs* a : ts) {
    if (a->d == 0) continue;
    const uintptr_t row_bytes = (uintptr_t)a->w * 2u;
    for (int s = 0; s < P.S; ++s) {
      in[n] = {(uintptr_t)a->x[s], (uintptr_t)a->x[s] + row_bytes * (uintptr_t)T};
      gm[n] = {(uintptr_t)a->gamma[s], (uintptr_t)a->gamma[s] + row_bytes};
      out[n] = {(uintptr_t)a->y[s], (uintptr_t)a->y[s] + row_bytes * (uintptr_t)T};
      ++n;
    }
    if (a->rstd) aux[naux++] = {(uintptr_t)a->rstd, (uintptr_t)a->rstd + 4u * (uintptr_t)T};
    if (a->partials)
      aux[naux++] = {(uintptr_t)a->partials, (uintptr_t)a->partials + 4u * (uintptr_t)T * (uintptr_t)P.S};
  }
  for (int i = 0; i < n; ++i) {
    for (int j = 0; j < n; ++j) {
      if (overlaps(out[i], gm[j])) return QKNORM_ERR_ALIAS;
      if (overlaps(out[i], in[j]) && !(i == j && out[i].lo == in[j].lo)) return QKNORM_ERR_ALIAS;
      if (j != i && overlaps(out[i], out[j])) return QKNORM_ERR_ALIAS;
    }
    for (int j = 0; j < naux; ++j)
      if (overlaps(out[i], aux[j])) return QKNORM_ERR_ALIAS;
  }
  for (int i = 0; i < naux; ++i) {
    for (int j = 0; j < n; ++j)
      if (overlaps(aux[i], in[j]) || overlaps(aux[i], gm[j])) return QKNORM_ERR_ALIAS;
    for (int j = i + 1; j < naux; ++j)
      if (overlaps(aux[i], aux[j])) return QKNORM_ERR_ALIAS;
  }
  return QKNORM_OK;
}

inline bool aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }

bool vector_path_ok(const Params& P) {
  const TensorArgs* ts[2] = {&P.q, &P.k};
  for (const TensorArgs* a : ts) {
    if (a->d == 0) continue;
    if (a->w % 8 != 0) return false;
    for (int s = 0; s < P.S; ++s)
      if (!aligned16(a->x[s]) || !aligned16(a->gamma[s]) || !aligned16(a->y[s])) return false;
  }
  return true;
}

int env_int(const char* name, int fallback) {
  const char* v = getenv(name);
  if (!v || !*v) return fallback;
  return atoi(v);
}

struct RowsPlan {
  RowsKernel fn = nullptr;
  int threads = 0, G = 0, logG = 0, nq = 0, nk = 0;
};

// Pick the thread grouping (G threads per slice) of the register-resident kernel.
//  throughput: CTAs of <= 256 threads, as few wasted lanes as possible;
//  latency (few tokens): CTAs of <= 512 threads and as few chunks per thread as possible,
//  so that one load round trip covers the row.
bool plan_rows(const Params& P, bool latency, RowsPlan* plan) {
  const int cq = P.q.d ? P.q.w / 8 : 0, ck = P.k.d ? P.k.w / 8 : 0;
  const int max_threads = latency ? 512 : 256;
  const int forced = env_int("QKNORM_FORCE_G", 0);
  double best_cost = 1e30;
  bool found = false;
  for (int logG = 4; logG <= 9; ++logG) {
    const int G = 1 << logG;
    if (forced && G != forced) continue;
    const int threads = ((P.S * G + 31) / 32) * 32;
    if (threads > max_threads) continue;
    const int nq = rows_round_up_n((cq + G - 1) / G, latency), nk = rows_round_up_n((ck + G - 1) / G, latency);
    if (nq < 0 || nk < 0) continue;
    RowsKernel fn = latency ? rows_kernel_latency(nq, nk) : rows_kernel_throughput(nq, nk);
    if (!fn) continue;
    // lanes issued per useful chunk; latency mode adds a strong preference for few chunks per thread
    double cost = (double)(nq + nk) * threads / (double)((cq + ck) * P.S);
    if (latency) cost += 4.0 * (nq + nk);
    else cost -= 1e-3 * logG;  // tie: wider groups, fewer registers
    if (cost < best_cost) {
      best_cost = cost;
      *plan = RowsPlan{fn, threads, G, logG, nq, nk};
      found = true;
    }
  }
  return found;
}

struct OccKey {
  const void* fn;
  int threads;
  int dev;
  int blocks;
};
constexpr int kOccCache = 256;
OccKey g_occ[kOccCache];
int g_occ_n = 0;
std::mutex g_occ_mutex;

// Resident CTAs per SM for (kernel, CTA size) on the current device: B_res of Section III-D.
int resident_blocks(const void* fn, int threads, int* out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_cuda_error(e);
  std::lock_guard<std::mutex> lock(g_occ_mutex);
  for (int i = 0; i < g_occ_n; ++i)
    if (g_occ[i].fn == fn && g_occ[i].threads == threads && g_occ[i].dev == dev) {
      *out = g_occ[i].blocks;
      return QKNORM_OK;
    }
  int blocks = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, fn, threads, 0);
  if (e != cudaSuccess) return set_cuda_error(e);
  if (blocks < 1) blocks = 1;
  if (g_occ_n < kOccCache) g_occ[g_occ_n++] = OccKey{fn, threads, dev, blocks};
  *out = blocks;
  return QKNORM_OK;
}

int launch(Params& P, cudaStream_t stream) {
  int sms = 0;
  int rc = current_sm_count(&sms);
  if (rc != QKNORM_OK) return rc;
  const char* force = getenv("QKNORM_FORCE_VARIANT");
  const bool force_general = force && strcmp(force, "general") == 0;

  if (!force_general && vector_path_ok(P)) {
    const bool latency = P.T < 4LL * sms;
    RowsPlan plan;
    if (plan_rows(P, latency, &plan)) {
      P.G = plan.G;
      P.logG = plan.logG;
      int bres = 1;
      rc = resident_blocks((const void*)plan.fn, plan.threads, &bres);
      if (rc != QKNORM_OK) return rc;
      const int cap = env_int("QKNORM_CTAS_PER_SM", 0);
      if (cap > 0 && cap < bres) bres = cap;
      long long grid = (long long)bres * sms;  // bounded grid of co-resident CTAs
      if (grid > P.T) grid = P.T;
      plan.fn<<<(unsigned)grid, plan.threads, 0, stream>>>(P);
      cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) return set_cuda_error(e);
      tl_variant = "rows";
      ++tl_launches;
      return QKNORM_OK;
    }
  }
  {
    int bres = 1;
    rc = resident_blocks((const void*)general_kernel, kGeneralThreads, &bres);
    if (rc != QKNORM_OK) return rc;
    long long grid = (long long)bres * sms;
    if (grid > 2 * P.T) grid = 2 * P.T;
    general_kernel<<<(unsigned)grid, kGeneralThreads, 0, stream>>>(P);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_cuda_error(e);
    tl_variant = "general";
    ++tl_launches;
  }
  return QKNORM_OK;
}

// Shared body of the four entry points.  Pointer arrays are host arrays of S entries.
int run(const void* const* q, const void* const* k, const void* const* gq, const void* const* gk,
        int32_t S, int64_t T, int32_t dq, int32_t dk, float eps, void* const* oq, void* const* ok,
        float* partials_q, float* partials_k, float* rstd_q, float* rstd_k, void* stream) {
  if (S < 1 || S > kMaxShards) return QKNORM_ERR_SHARDS;
  if (T < 0 || dq < 0 || dk < 0 || dq > kMaxDim || dk > kMaxDim) return QKNORM_ERR_SHAPE;
  if (dq % S != 0 || dk % S != 0) return QKNORM_ERR_SHAPE;
  if (!(eps >= 0.0f)) return QKNORM_ERR_EPS;  // also rejects NaN
  if (T == 0) return QKNORM_OK;
  if (dq == 0 && dk == 0) return QKNORM_ERR_SHAPE;
  if (dq > 0 && (!q || !gq || !oq)) return QKNORM_ERR_NULL;
  if (dk > 0 && (!k || !gk || !ok)) return QKNORM_ERR_NULL;

  Params P;
  memset(&P, 0, sizeof(P));
  P.T = T;
  P.S = S;
  P.eps = eps;
  P.G = 32;
  P.logG = 5;
  struct Side {
    TensorArgs* a;
    const void* const* x;
    const void* const* g;
    void* const* y;
    int d;
    float* partials;
    float* rstd;
  } sides[2] = {{&P.q, q, gq, oq, dq, partials_q, rstd_q}, {&P.k, k, gk, ok, dk, partials_k, rstd_k}};
  for (Side& sd : sides) {
    sd.a->d = sd.d;
    sd.a->w = sd.d / S;
    if (sd.d == 0) continue;
    for (int s = 0; s < S; ++s) {
      if (!sd.x[s] || !sd.g[s] || !sd.y[s]) return QKNORM_ERR_NULL;
      if ((((uintptr_t)sd.x[s]) | ((uintptr_t)sd.g[s]) | ((uintptr_t)sd.y[s])) & 1u) return QKNORM_ERR_ALIGN;
      sd.a->x[s] = (const uint16_t*)sd.x[s];
      sd.a->gamma[s] = (const uint16_t*)sd.g[s];
      sd.a->y[s] = (uint16_t*)sd.y[s];
    }
    if ((((uintptr_t)sd.partials) | ((uintptr_t)sd.rstd)) & 3u) return QKNORM_ERR_ALIGN;
    sd.a->partials = sd.partials;
    sd.a->rstd = sd.rstd;
  }
  int rc = check_alias(P, T);
  if (rc != QKNORM_OK) return rc;
  return launch(P, (cudaStream_t)stream);
}

}  // namespace
}  // namespace qknorm

extern "C" {

int qknorm_fwd(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
               int32_t dq, int32_t dk, float eps, void* out_q, void* out_k, void* stream) {
  return qknorm::run(&q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, eps, &out_q, &out_k, nullptr, nullptr,
                     nullptr, nullptr, stream);
}

int qknorm_fwd_ex(const void* q, const void* k, const void* gamma_q, const void* gamma_k, int64_t tokens,
                  int32_t dq, int32_t dk, float eps, void* out_q, void* out_k, float* rstd_q, float* rstd_k,
                  void* stream) {
  return qknorm::run(&q, &k, &gamma_q, &gamma_k, 1, tokens, dq, dk, eps, &out_q, &out_k, nullptr, nullptr,
                     rstd_q, rstd_k, stream);
}

int qknorm_fwd_sharded(const void* const* q_shards, const void* const* k_shards,
                       const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                       int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                       void* const* out_q_shards, void* const* out_k_shards, void* stream) {
  return qknorm::run(q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq, dk, eps,
                     out_q_shards, out_k_shards, nullptr, nullptr, nullptr, nullptr, stream);
}

int qknorm_fwd_sharded_ex(const void* const* q_shards, const void* const* k_shards,
                          const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                          int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                          void* const* out_q_shards, void* const* out_k_shards, float* partials_q,
                          float* partials_k, float* rstd_q, float* rstd_k, void* stream) {
  return qknorm::run(q_shards, k_shards, gamma_q_shards, gamma_k_shards, num_shards, tokens, dq, dk, eps,
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
    default: return "unknown qknorm status";
  }
}

int qknorm_last_cuda_error(void) { return qknorm::tl_cuda_error; }
const char* qknorm_last_variant(void) { return qknorm::tl_variant; }
int64_t qknorm_launch_count(void) { return qknorm::tl_launches; }
int qknorm_version(void) { return 100; }

}  // extern "C"

// Kernel parameter block shared by every kernel variant of libqknorm.
// Passed by value (__grid_constant__), so the host pointer arrays of the C ABI
// are consumed during the call and nothing has to be allocated on the device.
#pragma once
#include <stdint.h>

namespace qknorm {

constexpr int kMaxShards = 16;   // QKNORM_MAX_SHARDS
constexpr int kMaxDim = 65536;   // QKNORM_MAX_DIM
constexpr int kMaxSlots = 64;    // shared-memory partial sums per CTA (one per 16- or 32-lane group)

// One tensor (Q or K) held as S equal column slices.  S == 1 is the unsharded case.
struct TensorArgs {
  const void* x[kMaxShards];          // X_local of Algorithm 1, slice s: [T, w] bf16 or FP8-E4M3
  const uint16_t* gamma[kMaxShards];  // W_local, slice s: [w] bf16
  void* y[kMaxShards];                // Y_local, slice s: [T, w], same format as x (may equal x[s])
  float* partials;                    // optional [S, T]: Phase A scalar of every slice
  float* rstd;                        // optional [T]: RMS^-1 of Algorithm 1
  long long ldx;                      // elements between consecutive rows of x[s] (w when rows are contiguous)
  long long ldy;                      // the same for y[s]
  int d;                              // full width H_total (0 = tensor absent)
  int w;                              // slice width d / S
  float inv_d;                        // 1 / H_total
  // thread layout of the vectorised kernels (see qknorm_rowmap.cuh)
  int G;                              // threads serving one slice of this tensor (multiple of `sub`)
  int first_thread;                   // first thread of this tensor's block of S*G threads
};

struct Params {
  TensorArgs q, k;
  long long T;   // tokens
  int S;         // slices per tensor
  float eps;
  int log_sub;   // 4 or 5: lanes that reduce together by shuffle (16 or 32)
  int elem_bytes;  // 2 = bf16 activations, 1 = FP8-E4M3 activations
};

}  // namespace qknorm

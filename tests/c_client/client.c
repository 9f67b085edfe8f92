/*
 * A C program that uses libqknorm through include/qknorm.h only: device memory
 * from the CUDA runtime, plain pointers, no Python, no torch.  It normalises
 * constant rows, whose result has a closed form (Eq. 1 of the paper with
 * x_j = c, gamma_j = g:  y_j = g * c / sqrt(c^2 + eps)), unsharded and as four
 * column shards, and checks every output element.  Exit code 0 = all correct.
 */
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "qknorm.h"

static uint16_t f32_to_bf16(float f) { /* exact for the constants used here */
  uint32_t u;
  memcpy(&u, &f, 4);
  return (uint16_t)(u >> 16);
}
static float bf16_to_f32(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}
#define CK(x)                                                         \
  do {                                                                \
    cudaError_t e_ = (x);                                             \
    if (e_ != cudaSuccess) {                                          \
      fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_));        \
      return 2;                                                       \
    }                                                                 \
  } while (0)

static int check(const uint16_t* y, size_t n, float want, const char* what) {
  const uint16_t w = f32_to_bf16(want);
  for (size_t i = 0; i < n; ++i) {
    int d = (int)y[i] - (int)w; /* same sign and binade: bit patterns are ordered like the values */
    if (d < -1 || d > 1) {
      fprintf(stderr, "%s[%zu] = %g, expected %g\n", what, i, bf16_to_f32(y[i]), want);
      return 1;
    }
  }
  return 0;
}

int main(void) {
  const int64_t T = 2100;
  const int32_t dq = 2048, dk = 512, S = 4;
  const float eps = 1e-6f, cq = 3.0f, ck = -0.5f, gq = 1.25f, gk = 2.0f;
  const size_t nq = (size_t)T * dq, nk = (size_t)T * dk;
  uint16_t* h = (uint16_t*)malloc((nq > nk ? nq : nk) * 2);
  uint16_t *q, *k, *oq, *ok, *gmq, *gmk;
  CK(cudaMalloc((void**)&q, nq * 2));
  CK(cudaMalloc((void**)&k, nk * 2));
  CK(cudaMalloc((void**)&oq, nq * 2));
  CK(cudaMalloc((void**)&ok, nk * 2));
  CK(cudaMalloc((void**)&gmq, dq * 2));
  CK(cudaMalloc((void**)&gmk, dk * 2));
  for (size_t i = 0; i < nq; ++i) h[i] = f32_to_bf16(cq);
  CK(cudaMemcpy(q, h, nq * 2, cudaMemcpyHostToDevice));
  for (size_t i = 0; i < nk; ++i) h[i] = f32_to_bf16(ck);
  CK(cudaMemcpy(k, h, nk * 2, cudaMemcpyHostToDevice));
  for (int i = 0; i < dq; ++i) h[i] = f32_to_bf16(gq);
  CK(cudaMemcpy(gmq, h, dq * 2, cudaMemcpyHostToDevice));
  for (int i = 0; i < dk; ++i) h[i] = f32_to_bf16(gk);
  CK(cudaMemcpy(gmk, h, dk * 2, cudaMemcpyHostToDevice));
  cudaStream_t st;
  CK(cudaStreamCreate(&st));

  const float want_q = gq * cq / sqrtf(cq * cq + eps), want_k = gk * ck / sqrtf(ck * ck + eps);
  int bad = 0;

  /* unsharded */
  int rc = qknorm_fwd(q, k, gmq, gmk, T, dq, dk, eps, oq, ok, st);
  if (rc != QKNORM_OK) { fprintf(stderr, "qknorm_fwd: %s\n", qknorm_status_string(rc)); return 3; }
  CK(cudaStreamSynchronize(st));
  CK(cudaMemcpy(h, oq, nq * 2, cudaMemcpyDeviceToHost));
  bad |= check(h, nq, want_q, "out_q");
  CK(cudaMemcpy(h, ok, nk * 2, cudaMemcpyDeviceToHost));
  bad |= check(h, nk, want_k, "out_k");
  printf("qknorm_fwd: variant %s\n", qknorm_last_variant());

  /* the same buffers read as 4 column shards of [T, d/4] (a constant tensor looks the same either way), in place */
  const void *qs[4], *ks[4], *gqs[4], *gks[4];
  void *oqs[4], *oks[4];
  for (int s = 0; s < S; ++s) {
    qs[s] = q + (size_t)s * T * (dq / S);
    ks[s] = k + (size_t)s * T * (dk / S);
    gqs[s] = gmq + (size_t)s * (dq / S);
    gks[s] = gmk + (size_t)s * (dk / S);
    oqs[s] = (void*)qs[s];
    oks[s] = (void*)ks[s];
  }
  rc = qknorm_fwd_sharded(qs, ks, gqs, gks, S, T, dq, dk, eps, oqs, oks, st);
  if (rc != QKNORM_OK) { fprintf(stderr, "qknorm_fwd_sharded: %s\n", qknorm_status_string(rc)); return 3; }
  CK(cudaStreamSynchronize(st));
  CK(cudaMemcpy(h, q, nq * 2, cudaMemcpyDeviceToHost));
  bad |= check(h, nq, want_q, "sharded in-place q");
  CK(cudaMemcpy(h, k, nk * 2, cudaMemcpyDeviceToHost));
  bad |= check(h, nk, want_k, "sharded in-place k");
  printf("qknorm_fwd_sharded: variant %s\n", qknorm_last_variant());

  /* an overlapping output is refused on the host, nothing is launched */
  rc = qknorm_fwd(q, k, gmq, gmk, T, dq, dk, eps, q + 8, ok, st);
  if (rc != QKNORM_ERR_ALIAS) { fprintf(stderr, "expected QKNORM_ERR_ALIAS, got %d\n", rc); bad = 1; }

  int word = -1;
  rc = qknorm_device_error_word(&word);
  if (rc != QKNORM_OK || word != 0) { fprintf(stderr, "device error word %d (rc %d)\n", word, rc); bad = 1; }
  printf(bad ? "FAILED\n" : "ok\n");
  return bad;
}

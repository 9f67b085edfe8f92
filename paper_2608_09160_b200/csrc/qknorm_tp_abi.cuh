// The extern "C" entry points of include/qknorm_tp.h.  Included by qknorm_api.cu at file scope.
#pragma once

extern "C" {

int qknorm_tp_inbox_bytes(int32_t num_ranks, int64_t token_capacity, int64_t* bytes) {
  long long b = 0;
  const int rc = qknorm::tp_inbox_bytes(num_ranks, token_capacity, bytes ? &b : nullptr);
  if (rc == QKNORM_OK) *bytes = b;
  return rc;
}

int qknorm_fwd_tp(const qknorm_tp_rank* ranks, int32_t n_local, int32_t num_ranks, int64_t tokens,
                  int64_t token_capacity, int32_t wq, int32_t wk, const int64_t* ld, float eps, uint32_t epoch,
                  uint32_t wait_limit_us, void* stream) {
  return qknorm::run_tp(2, ranks, n_local, num_ranks, tokens, token_capacity, wq, wk, ld, eps, epoch,
                        wait_limit_us, (cudaStream_t)stream);
}

int qknorm_fwd_tp_e4m3(const qknorm_tp_rank* ranks, int32_t n_local, int32_t num_ranks, int64_t tokens,
                       int64_t token_capacity, int32_t wq, int32_t wk, const int64_t* ld, float eps, uint32_t epoch,
                       uint32_t wait_limit_us, void* stream) {
  return qknorm::run_tp(1, ranks, n_local, num_ranks, tokens, token_capacity, wq, wk, ld, eps, epoch,
                        wait_limit_us, (cudaStream_t)stream);
}

int qknorm_tp_status(const void* inbox, int32_t* out) {
  if (!inbox || !out) return QKNORM_ERR_NULL;
  cudaError_t e = cudaMemcpy(out, inbox, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

int64_t qknorm_tp_slot_index(int32_t num_ranks, int64_t token_capacity, uint32_t epoch, int32_t tensor, int32_t src_rank) {
  if (num_ranks < 1 || num_ranks > qknorm::kMaxShards || token_capacity < 1 || epoch == 0u) return -1;
  if (tensor < 0 || tensor > 1 || src_rank < 0 || src_rank >= num_ranks) return -1;
  return (int64_t)qknorm::tp_slot_index((int)(epoch & 1u), tensor, src_rank, num_ranks, token_capacity);
}

int qknorm_tp_inbox_peek(const void* inbox, int64_t first_word, int64_t n_words, uint64_t* out) {
  if (!inbox || !out) return QKNORM_ERR_NULL;
  if (first_word < 0 || n_words < 0) return QKNORM_ERR_SHAPE;
  cudaError_t e = cudaMemcpy(out, (const unsigned long long*)inbox + first_word, (size_t)n_words * 8, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

int qknorm_tp_inbox_poke(void* inbox, int64_t first_word, int64_t n_words, const uint64_t* in) {
  if (!inbox || !in) return QKNORM_ERR_NULL;
  if (first_word < 0 || n_words < 0) return QKNORM_ERR_SHAPE;
  cudaError_t e = cudaMemcpy((unsigned long long*)inbox + first_word, in, (size_t)n_words * 8, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

int qknorm_tp_clear_status(void* inbox, void* stream) {
  if (!inbox) return QKNORM_ERR_NULL;
  cudaError_t e = cudaMemsetAsync(inbox, 0, 8 * qknorm::kTpHeaderWords, (cudaStream_t)stream);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

int qknorm_tp_inbox_create(int32_t num_ranks, int64_t token_capacity, void** out) {
  if (!out) return QKNORM_ERR_NULL;
  long long bytes = 0;
  const int rc = qknorm::tp_inbox_bytes(num_ranks, token_capacity, &bytes);
  if (rc != QKNORM_OK) return rc;
  void* p = nullptr;
  cudaError_t e = cudaMalloc(&p, (size_t)bytes);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  e = cudaMemset(p, 0, (size_t)bytes);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    cudaFree(p);
    return qknorm::set_cuda_error(e);
  }
  *out = p;
  return QKNORM_OK;
}

int qknorm_tp_inbox_zero(void* inbox, int32_t num_ranks, int64_t token_capacity, void* stream) {
  if (!inbox) return QKNORM_ERR_NULL;
  long long bytes = 0;
  const int rc = qknorm::tp_inbox_bytes(num_ranks, token_capacity, &bytes);
  if (rc != QKNORM_OK) return rc;
  cudaError_t e = cudaMemsetAsync(inbox, 0, (size_t)bytes, (cudaStream_t)stream);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

int qknorm_tp_inbox_destroy(void* inbox) {
  if (!inbox) return QKNORM_OK;
  cudaError_t e = cudaFree(inbox);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

int qknorm_tp_ipc_export(const void* inbox, unsigned char* handle) {
  static_assert(sizeof(cudaIpcMemHandle_t) == QKNORM_TP_IPC_HANDLE_BYTES, "handle size");
  if (!inbox || !handle) return QKNORM_ERR_NULL;
  cudaIpcMemHandle_t h;
  cudaError_t e = cudaIpcGetMemHandle(&h, const_cast<void*>(inbox));
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  memcpy(handle, &h, sizeof(h));
  return QKNORM_OK;
}

int qknorm_tp_ipc_open(const unsigned char* handle, void** out) {
  if (!handle || !out) return QKNORM_ERR_NULL;
  cudaIpcMemHandle_t h;
  memcpy(&h, handle, sizeof(h));
  void* p = nullptr;
  cudaError_t e = cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  *out = p;
  return QKNORM_OK;
}

int qknorm_tp_ipc_close(void* mapped) {
  if (!mapped) return QKNORM_OK;
  cudaError_t e = cudaIpcCloseMemHandle(mapped);
  if (e != cudaSuccess) return qknorm::set_cuda_error(e);
  return QKNORM_OK;
}

}  // extern "C"

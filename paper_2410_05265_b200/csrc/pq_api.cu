// Context life cycle and status plumbing of the pq library.
#include <new>

#include "pq_common.cuh"

extern "C" {

const char* pq_status_string(pq_status s) {
  switch (s) {
    case PQ_OK: return "PQ_OK";
    case PQ_ERR_INVALID_ARG: return "PQ_ERR_INVALID_ARG";
    case PQ_ERR_SHAPE: return "PQ_ERR_SHAPE";
    case PQ_ERR_ALIGN: return "PQ_ERR_ALIGN";
    case PQ_ERR_WORKSPACE: return "PQ_ERR_WORKSPACE";
    case PQ_ERR_CUDA: return "PQ_ERR_CUDA";
    case PQ_ERR_TIMEOUT: return "PQ_ERR_TIMEOUT";
    case PQ_ERR_UNSUPPORTED: return "PQ_ERR_UNSUPPORTED";
    default: return "PQ_ERR_UNKNOWN";
  }
}

pq_status pq_create(pq_ctx** out) {
  if (!out) return PQ_ERR_INVALID_ARG;
  *out = nullptr;
  pq_ctx* c = new (std::nothrow) pq_ctx();
  if (!c) return PQ_ERR_CUDA;
  c->d_status = nullptr;
  c->d_tickets = nullptr;
  c->n_tickets = PQ_N_TICKETS;
  c->encode_tiled = nullptr;
  c->wait_clocks = PQ_DEFAULT_WAIT_CLOCKS;
  cudaDeviceProp prop;
  if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) {
    delete c;
    return PQ_ERR_CUDA;
  }
  if (prop.major != 10) {  // the kernels are sm_100a only
    delete c;
    return PQ_ERR_UNSUPPORTED;
  }
  c->sm_count = prop.multiProcessorCount;
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete c;
    return PQ_ERR_CUDA;
  }
  c->encode_tiled = fn;
  if (cudaMalloc(&c->d_status, sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc(&c->d_tickets, sizeof(uint32_t) * PQ_N_TICKETS) != cudaSuccess ||
      cudaMemset(c->d_status, 0, sizeof(int32_t)) != cudaSuccess ||
      cudaMemset(c->d_tickets, 0, sizeof(uint32_t) * PQ_N_TICKETS) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess) {
    if (c->d_status) cudaFree(c->d_status);
    if (c->d_tickets) cudaFree(c->d_tickets);
    delete c;
    return PQ_ERR_CUDA;
  }
  *out = c;
  return PQ_OK;
}

pq_status pq_destroy(pq_ctx* ctx) {
  if (!ctx) return PQ_ERR_INVALID_ARG;
  cudaFree(ctx->d_status);
  cudaFree(ctx->d_tickets);
  delete ctx;
  return PQ_OK;
}

pq_status pq_set_wait_limit(pq_ctx* ctx, int64_t sm_clocks) {
  if (!ctx || sm_clocks < 0) return PQ_ERR_INVALID_ARG;
  ctx->wait_clocks = sm_clocks == 0 ? PQ_DEFAULT_WAIT_CLOCKS : static_cast<long long>(sm_clocks);
  return PQ_OK;
}

pq_status pq_check(pq_ctx* ctx, void* stream) {
  if (!ctx) return PQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t h = 0;
  if (cudaMemcpyAsync(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return PQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return PQ_ERR_CUDA;
  if (h != 0) {
    // a kernel that gave up may have left its "last block done" counters half-way: start the next one from zero
    if (cudaMemsetAsync(ctx->d_tickets, 0, sizeof(uint32_t) * PQ_N_TICKETS, st) != cudaSuccess) return PQ_ERR_CUDA;
    if (cudaMemsetAsync(ctx->d_status, 0, sizeof(int32_t), st) != cudaSuccess) return PQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PQ_ERR_CUDA;
  }
  return static_cast<pq_status>(h);
}

}  // extern "C"

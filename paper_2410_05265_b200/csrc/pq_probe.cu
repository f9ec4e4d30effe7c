// Measurement aid: the issue rate of tcgen05.mma kind::i8 with both operands resident in shared memory, i.e. the
// integer tensor-core rate a W4A4 GEMM could reach if nothing but the MMAs had to run (no loads, no nibble
// expansion, no epilogue). The benchmark divides the GEMM's achieved rate by it.
#include "pq_common.cuh"

namespace {

constexpr int PR_M = 128, PR_N = 256;  // one instruction: 128 x 256 x 32 multiply-accumulates
constexpr int PR_SMEM = 1024 + PR_M * 128 + PR_N * 128;  // 128-byte swizzled rows (only the first 32 bytes are read)

__global__ void __launch_bounds__(128, 1) probe_i8_mma_kernel(int iters, long long* cycles, int32_t* status, long long wait_clocks) {
  extern __shared__ uint8_t pr_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(pr_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t done;
  __shared__ uint32_t tmem_base_s;
  for (int i = threadIdx.x; i < (PR_M + PR_N) * 128 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x01010101u;
  if (threadIdx.x == 0) {
    pq::mbar_init(&done, 1);
    pq::mbar_fence_init();
  }
  pq::fence_proxy_async_smem();
  if (threadIdx.x < 32) {
    pq::tmem_alloc(&tmem_base_s, PR_N);
    pq::tmem_relinquish();
  }
  pq::tc_fence_before();
  __syncthreads();
  pq::tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  if (threadIdx.x == 0) {
    const uint64_t a = pq::umma_desc_sw128(pq::smem_u32(smem)), b = pq::umma_desc_sw128(pq::smem_u32(smem + PR_M * 128));
    constexpr uint32_t idesc = pq::umma_idesc_s8(PR_M, PR_N);
    const long long t0 = clock64();
    for (int i = 0; i < iters; ++i) pq::mma_i8_ss(tmem_base, a, b, idesc, i ? 1u : 0u);
    pq::mma_commit(&done);
    const bool ok = pq::mbar_wait_for(&done, 0, wait_clocks);
    const long long t1 = clock64();
    cycles[blockIdx.x] = ok ? t1 - t0 : -1;
    if (!ok) {
      pq::report(status, PQ_ERR_TIMEOUT);
      pq::mbar_wait(&done, 0);  // the instructions in flight finish before tensor memory is released
    }
  }
  pq::tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    pq::tc_fence_after();
    pq::tmem_dealloc(tmem_base, PR_N);
  }
}

// Failure-detection self-test: one thread waits on a barrier that nothing ever completes; the bounded wait runs out
// after the context's limit, the status word takes PQ_ERR_TIMEOUT and the kernel returns.
__global__ void selftest_wait_kernel(int32_t* status, long long wait_clocks, long long* waited) {
  __shared__ __align__(8) uint64_t never;
  pq::mbar_init(&never, 1);
  pq::mbar_fence_init();
  const long long t0 = clock64();
  const bool ok = pq::mbar_wait_for(&never, 0, wait_clocks);
  if (waited) *waited = clock64() - t0;
  if (!ok) pq::report(status, PQ_ERR_TIMEOUT);
}

}  // namespace

extern "C" pq_status pq_selftest_wait(pq_ctx* ctx, int64_t* waited_clocks, void* stream) {
  if (!ctx) return PQ_ERR_INVALID_ARG;
  selftest_wait_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_status, ctx->wait_clocks, reinterpret_cast<long long*>(waited_clocks));
  return pq_launch_status();
}

extern "C" pq_status pq_probe_i8_mma(pq_ctx* ctx, int32_t iters, int64_t* cycles, int32_t n_ctas, void* stream) {
  if (!ctx || !cycles || iters <= 0 || iters > (1 << 20) || n_ctas <= 0 || n_ctas > ctx->sm_count) return PQ_ERR_INVALID_ARG;
  static bool attr_set[64] = {};
  if (ctx->device < 0 || ctx->device >= 64) return PQ_ERR_UNSUPPORTED;
  if (!attr_set[ctx->device]) {
    if (cudaFuncSetAttribute(probe_i8_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PR_SMEM) != cudaSuccess) return PQ_ERR_CUDA;
    attr_set[ctx->device] = true;
  }
  probe_i8_mma_kernel<<<n_ctas, 128, PR_SMEM, static_cast<cudaStream_t>(stream)>>>(iters, reinterpret_cast<long long*>(cycles), ctx->d_status,
                                                                                   ctx->wait_clocks);
  return pq_launch_status();
}

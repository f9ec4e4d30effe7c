// Offline RTN weight quantization, one symmetric INT4 scale per output channel
// (Table 1 "per-channel"; Table 6 "RTN"; Eq. 1). One CTA per weight row, two passes over the row.
#include "pq_common.cuh"

namespace {

constexpr int QW_THREADS = 256;

__global__ void __launch_bounds__(QW_THREADS) quant_weights_kernel(const __nv_bfloat16* __restrict__ W, int64_t N,
                                                                    int64_t K, int64_t ldw, uint8_t* __restrict__ wq,
                                                                    float* __restrict__ s_w) {
  __shared__ float red[QW_THREADS / 32];
  __shared__ float s_scale;
  for (int64_t n = blockIdx.x; n < N; n += gridDim.x) {
    const __nv_bfloat16* row = W + n * ldw;
    float mx = 0.0f;
    for (int64_t k = threadIdx.x; k < K; k += QW_THREADS) mx = fmaxf(mx, fabsf(__bfloat162float(row[k])));
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
      float m = red[0];
      for (int i = 1; i < QW_THREADS / 32; ++i) m = fmaxf(m, red[i]);
      float s = (m == 0.0f) ? 1.0f : __fdiv_rn(m, 7.0f);
      s_scale = s;
      s_w[n] = s;
    }
    __syncthreads();
    const float s = s_scale;
    uint8_t* orow = wq + n * (K / 2);
    for (int64_t j = threadIdx.x; j < K / 2; j += QW_THREADS) {
      float a = __fdiv_rn(__bfloat162float(row[2 * j]), s);      // IEEE fp32 division
      float b = __fdiv_rn(__bfloat162float(row[2 * j + 1]), s);
      int ca = max(-8, min(7, __float2int_rn(a)));                // round-half-even, clamp
      int cb = max(-8, min(7, __float2int_rn(b)));
      orow[j] = static_cast<uint8_t>((ca & 0xF) | ((cb & 0xF) << 4));
    }
    __syncthreads();
  }
}

}  // namespace

extern "C" pq_status pq_quant_weights(pq_ctx* ctx, const void* W, int64_t N, int64_t K, int64_t ldw, uint8_t* wq,
                                      float* s_w, void* stream) {
  if (!ctx || !W || !wq || !s_w) return PQ_ERR_INVALID_ARG;
  if (N < 0 || K < 0 || ldw < K) return PQ_ERR_INVALID_ARG;
  if (K % 2 != 0) return PQ_ERR_SHAPE;
  if (N == 0 || K == 0) return PQ_OK;
  int grid = static_cast<int>(N < 65535 * 4 ? N : 65535 * 4);
  quant_weights_kernel<<<grid, QW_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(W), N, K, ldw, wq, s_w);
  return pq_launch_status();
}

// Sum of the signed 4-bit codes of every weight row (the zero-point correction of the asymmetric activation
// quantizer needs it): a warp per row; `(w << 4) & 0xF0F0F0F0` and `w & 0xF0F0F0F0` are the codes times 16
// as signed bytes, summed four at a time with dp4a.
namespace {
__global__ void __launch_bounds__(256) weight_code_sums_kernel(const uint8_t* wq, int64_t N, int64_t kwords, int32_t* wsum) {
  const int lane = threadIdx.x & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= N) return;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(wq) + row * kwords;
  int acc = 0;
  for (int64_t i = lane; i < kwords; i += 32) {
    const uint32_t w = __ldg(src + i);
    acc = __dp4a(static_cast<int>((w << 4) & 0xF0F0F0F0u), 0x01010101, acc);
    acc = __dp4a(static_cast<int>(w & 0xF0F0F0F0u), 0x01010101, acc);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) wsum[row] = acc >> 4;  // exact: every term carries the factor 16
}
}  // namespace

extern "C" pq_status pq_weight_code_sums(pq_ctx* ctx, const uint8_t* wq, int64_t N, int64_t K, int32_t* wsum, void* stream) {
  if (!ctx || !wq || !wsum || N < 0 || K <= 0) return PQ_ERR_INVALID_ARG;
  if (K % 8 != 0) return PQ_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(wq) & 3) return PQ_ERR_ALIGN;
  if (N == 0) return PQ_OK;
  weight_code_sums_kernel<<<static_cast<unsigned>((N + 7) / 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(wq, N, K / 8, wsum);
  return pq_launch_status();
}

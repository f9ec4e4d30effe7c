// Entry point of the W4A4 linear layer: argument checks and the choice between the tensor-core
// kernels (prefill-shaped) and the weight-streaming kernel (decode-shaped).
#include "pq_common.cuh"

pq_status pq_gemm_pair_launch(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w,
                              void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg, cudaStream_t st,
                              bool a8, const float* s_row, const int32_t* zp, const int32_t* wsum);
pq_status pq_gemm_pair_ts_launch(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w,
                                 void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg, cudaStream_t st,
                                 const float* s_row, const int32_t* zp, const int32_t* wsum);
pq_status pq_gemm_stream_launch(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a,
                                const float* s_w, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K,
                                int32_t* acc_dbg, cudaStream_t st, bool per_token, bool a8, const int32_t* zp,
                                const int32_t* wsum);

extern "C" size_t pq_w4a4_gemm_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }

extern "C" pq_status pq_w4a4_gemm(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a,
                                  const float* s_w, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K,
                                  int64_t row_begin, int32_t* acc_dbg, void* ws, size_t ws_bytes, void* stream) {
  (void)ws;
  (void)ws_bytes;
  if (!ctx || !xq || !wq || !s_a || !s_w || !out) return PQ_ERR_INVALID_ARG;
  if (M < 0 || N < 0 || K < 0 || row_begin < 0 || ldo < N) return PQ_ERR_INVALID_ARG;
  if (K % 32 != 0 || K > 65536 || M > (1 << 30) || N > (1 << 30)) return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(xq) & 15) || (reinterpret_cast<uintptr_t>(wq) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 1))
    return PQ_ERR_ALIGN;
  if (row_begin >= M || N == 0) return PQ_OK;
  const int64_t m = M - row_begin;
  const uint8_t* xq0 = xq + row_begin * (K / 2);
  void* out0 = static_cast<__nv_bfloat16*>(out) + row_begin * ldo;
  int32_t* dbg0 = acc_dbg ? acc_dbg + row_begin * N : nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (K == 0) return PQ_ERR_SHAPE;
  if (m <= 16) return pq_gemm_stream_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, false, false, nullptr, nullptr);
  // Two CTA-pair kernels (every 4-bit setting takes the same choice): with the token operand in shared memory the accumulator is double-buffered
  // and the epilogue is free, which wins for short K; with the token operand in tensor memory the
  // expansion costs a third less shared-memory traffic, which wins once a tile's K loop is long enough
  // to hide the single accumulator's epilogue (measured crossover near K = 8192).
  if (K >= 8192) return pq_gemm_pair_ts_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, nullptr, nullptr, nullptr);
  return pq_gemm_pair_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, false, nullptr, nullptr, nullptr);
}

// W4A8 (Sec. 5.1): the token operand is one s8 code per element: the weight-streaming kernel for up to 16
// tokens, the CTA-pair tensor-core kernel above that.
extern "C" pq_status pq_w4a8_gemm(pq_ctx* ctx, const int8_t* xq8, const uint8_t* wq, const float* s_a,
                                  const float* s_w, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K,
                                  int64_t row_begin, int32_t* acc_dbg, void* stream) {
  if (!ctx || !xq8 || !wq || !s_a || !s_w || !out) return PQ_ERR_INVALID_ARG;
  if (M < 0 || N < 0 || K < 0 || row_begin < 0 || ldo < N) return PQ_ERR_INVALID_ARG;
  // |code_a * 16 code_w| <= 128 * 128 per term: K <= 65536 keeps the int32 accumulator exact
  if (K % 32 != 0 || K == 0 || K > 65536 || M > (1 << 30) || N > (1 << 30)) return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(xq8) & 15) || (reinterpret_cast<uintptr_t>(wq) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 1))
    return PQ_ERR_ALIGN;
  if (row_begin >= M || N == 0) return PQ_OK;
  const int64_t m = M - row_begin;
  const uint8_t* xq0 = reinterpret_cast<const uint8_t*>(xq8) + row_begin * K;
  void* out0 = static_cast<__nv_bfloat16*>(out) + row_begin * ldo;
  int32_t* dbg0 = acc_dbg ? acc_dbg + row_begin * N : nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (m <= 16) return pq_gemm_stream_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, false, true, nullptr, nullptr);
  return pq_gemm_pair_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, true, nullptr, nullptr, nullptr);
}

// W4A4 with per-token dynamic activation steps (Table 1, O1): out[t,n] = bf16(acc * s_tok[t] * s_w[n]).
extern "C" pq_status pq_w4a4_gemm_rows(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_tok,
                                       const float* s_w, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K,
                                       int64_t row_begin, int32_t* acc_dbg, void* stream) {
  if (!ctx || !xq || !wq || !s_tok || !s_w || !out) return PQ_ERR_INVALID_ARG;
  if (M < 0 || N < 0 || K < 0 || row_begin < 0 || ldo < N) return PQ_ERR_INVALID_ARG;
  if (K % 32 != 0 || K == 0 || K > 65536 || M > (1 << 30) || N > (1 << 30)) return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(xq) & 15) || (reinterpret_cast<uintptr_t>(wq) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 1))
    return PQ_ERR_ALIGN;
  if (row_begin >= M || N == 0) return PQ_OK;
  const int64_t m = M - row_begin;
  const uint8_t* xq0 = xq + row_begin * (K / 2);
  const float* s0 = s_tok + row_begin;
  void* out0 = static_cast<__nv_bfloat16*>(out) + row_begin * ldo;
  int32_t* dbg0 = acc_dbg ? acc_dbg + row_begin * N : nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (m <= 16) return pq_gemm_stream_launch(ctx, xq0, wq, s0, s_w, out0, ldo, m, N, K, dbg0, st, true, false, nullptr, nullptr);
  if (K >= 8192) return pq_gemm_pair_ts_launch(ctx, xq0, wq, nullptr, s_w, out0, ldo, m, N, K, dbg0, st, s0, nullptr, nullptr);
  return pq_gemm_pair_launch(ctx, xq0, wq, nullptr, s_w, out0, ldo, m, N, K, dbg0, st, false, s0, nullptr, nullptr);
}

// W4A4 with the activation quantizer of Eq. 1 as printed (zero point z): the stored token codes are u - 8,
// out[t,n] = bf16(s_a * s_w[n] * sum_k (u[t,k] - z) * w[n,k]); wsum[n] = sum_k w[n,k] comes from pq_weight_code_sums.
extern "C" pq_status pq_w4a4_gemm_asym(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a,
                                       const int32_t* z_a, const float* s_w, const int32_t* wsum, void* out, int64_t ldo,
                                       int64_t M, int64_t N, int64_t K, int64_t row_begin, int32_t* acc_dbg,
                                       void* stream) {
  if (!ctx || !xq || !wq || !s_a || !z_a || !s_w || !wsum || !out) return PQ_ERR_INVALID_ARG;
  if (M < 0 || N < 0 || K < 0 || row_begin < 0 || ldo < N) return PQ_ERR_INVALID_ARG;
  if (K % 32 != 0 || K == 0 || K > 65536 || M > (1 << 30) || N > (1 << 30)) return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(xq) & 15) || (reinterpret_cast<uintptr_t>(wq) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 1))
    return PQ_ERR_ALIGN;
  if (row_begin >= M || N == 0) return PQ_OK;
  const int64_t m = M - row_begin;
  const uint8_t* xq0 = xq + row_begin * (K / 2);
  void* out0 = static_cast<__nv_bfloat16*>(out) + row_begin * ldo;
  int32_t* dbg0 = acc_dbg ? acc_dbg + row_begin * N : nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (m <= 16) return pq_gemm_stream_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, false, false, z_a, wsum);
  if (K >= 8192) return pq_gemm_pair_ts_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, nullptr, z_a, wsum);
  return pq_gemm_pair_launch(ctx, xq0, wq, s_a, s_w, out0, ldo, m, N, K, dbg0, st, false, nullptr, z_a, wsum);
}

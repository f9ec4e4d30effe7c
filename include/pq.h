/*
 * pq.h — C ABI of the B200 (sm_100a) W4A4KV4 inference hot path of PrefixQuant in its static
 * setting ("O2" in Table 1: per-channel weights, per-tensor static activations, per-head static
 * KV cache), where the outlier tokens are prefixed and their K/V stay in full precision (Eq. 3).
 *
 * General rules
 *   - Every tensor pointer is a DEVICE pointer on the device that was current at pq_create(),
 *     owned by the caller. The library allocates only inside pq_create() (a few KB: a status
 *     word and ticket counters) and frees only inside pq_destroy(). Scratch memory is a caller
 *     buffer sized by the matching *_workspace_bytes() function.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return at once.
 *     Argument errors are reported synchronously through the return value and enqueue nothing.
 *     Errors found on the device (a bounded wait that ran out, a KV append past capacity) are
 *     written to a status word read by pq_check().
 *   - Nothing aborts, traps or prints. Every wait inside a kernel is bounded.
 *   - One pq_ctx must not be used from two streams at the same time (ticket counters are shared).
 *   - bf16 / fp16 tensors are raw 16-bit patterns. Packed INT4 tensors hold element 2j in the low
 *     nibble and element 2j+1 in the high nibble of byte j, two's complement, packed along the
 *     contraction (K) or head (D) dimension.
 *   - The signed 4-bit code of a value v with step s is clamp(round_half_even(v / s), -8, 7): Eq. (1)
 *     with N = 4 in its symmetric reading (zero-point fixed at 8, s = max|v| / 7).
 */
#ifndef PQ_H_
#define PQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t pq_status;
enum {
  PQ_OK = 0,
  PQ_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad enum */
  PQ_ERR_SHAPE = 2,       /* size outside what the kernels support, KV append past Tmax */
  PQ_ERR_ALIGN = 3,       /* pointer or leading dimension not aligned as documented */
  PQ_ERR_WORKSPACE = 4,   /* workspace missing or too small */
  PQ_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed */
  PQ_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out */
  PQ_ERR_UNSUPPORTED = 7
};

typedef struct pq_ctx pq_ctx;

/* Human-readable name of a status code (static storage). */
const char* pq_status_string(pq_status s);

/* Creates a context on the current device: caches the SM count, resolves the tensor-map encoder,
 * allocates the device status word and the ticket counters. */
pq_status pq_create(pq_ctx** out);
pq_status pq_destroy(pq_ctx* ctx);

/* Synchronizes `stream`, returns the device status word (PQ_OK if no kernel reported anything)
 * and clears it. */
pq_status pq_check(pq_ctx* ctx, void* stream);

/* Bound of the device-side waits (a consumer waiting for a copy or for a producer, a producer waiting for
 * a free buffer) of the kernels launched through this context from now on, in SM clocks; 0 restores the
 * default of 2^31 clocks (about a second). A wait that runs out makes its kernel wind down in an orderly
 * way (copies in flight are awaited, tensor memory is released) and leaves PQ_ERR_TIMEOUT in the status
 * word; the kernel's output is then undefined. Failure-detection tests set a bound of a few clocks so that
 * an ordinary wait runs out. */
pq_status pq_set_wait_limit(pq_ctx* ctx, int64_t sm_clocks);

/* ---------------------------------------------------------------------------------------------
 * Offline weight quantization: round-to-nearest, one symmetric scale per output channel
 * (Table 1 "per-channel" weights; the "RTN" row of Table 6; Eq. 1).
 *   W    bf16 [N, K], row stride ldw elements (ldw >= K)
 *   wq   u8   [N, K/2] packed codes (dense rows)
 *   s_w  f32  [N]: s_w[n] = max_k |W[n,k]| / 7 in fp32 (1 for an all-zero row)
 *   code = clamp(rint(W[n,k] / s_w[n]), -8, 7) with IEEE fp32 division.
 * K must be even. */
pq_status pq_quant_weights(pq_ctx* ctx, const void* W, int64_t N, int64_t K, int64_t ldw, uint8_t* wq, float* s_w,
                           void* stream);

/* ---------------------------------------------------------------------------------------------
 * Online rotation (App. B, "Online Rotation": the Walsh-Hadamard transform applied to a linear
 * layer's input) fused with the static per-tensor quantizer (Table 1, O2; Sec. 3 "Dynamic and
 * Static") and the nibble pack.
 * For every row t >= row_begin and every contiguous had_block-wide block of that row:
 *     y = x_block * H / sqrt(had_block),  H[i][j] = (-1)^popcount(i & j)   (Sylvester order)
 *     xq = pack(clamp(round_half_even(y / s_a), -8, 7))
 *   x    bf16 [M, K], row stride ldx elements (even, >= K), base 4-byte aligned
 *   xq   u8   [M, K/2] dense rows, base 16-byte aligned
 *   s_a  f32 scalar on the device (static: calibrated offline, never recomputed here)
 *   had_block: a power of two in [128, 8192] dividing K, or 0 for "no rotation" (K % 128 == 0).
 * Rows below row_begin are the prefixed outlier tokens: they are neither read nor written. */
pq_status pq_hadamard_quant_act(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                int64_t row_begin, const float* s_a, uint8_t* xq, void* stream);

/* Calibration helper for the static activation scale: over rows >= row_begin of a calibration
 * batch, *s_a = max(*s_a, max |y| / 7) with y the rotated rows as above. *s_a must be initialised
 * by the caller (0 to start); several batches may be folded into it. The prefixed rows never
 * take part (Sec. 5.5: isolating the >1e3 outliers is what makes the static scale usable). */
pq_status pq_calib_act_scale(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                             int64_t row_begin, float* s_a, void* stream);

/* The same quantizer with the SwiGLU of the MLP in front (App. B: the online rotation R4 sits between the
 * activation function and down_proj): the transform's input is bf16(SiLU(gate) * up), formed in registers with
 * the arithmetic and the rounding of pq_silu_mul, so the result equals pq_silu_mul followed by
 * pq_hadamard_quant_act bit for bit while the [M, K] activation tensor never goes to memory.
 *   gate, up  bf16 [M, K] with ld_in elements between rows (the two halves of a concatenated gate|up output) */
pq_status pq_swiglu_hadamard_quant_act(pq_ctx* ctx, const void* gate, const void* up, int64_t M, int64_t K, int64_t ld_in,
                                       int had_block, int64_t row_begin, const float* s_a, uint8_t* xq, void* stream);

/* The same quantizer with the RMSNorm of the block in front (App. B figure: RMSNorm feeds the q/k/v and the gate/up
 * linears): the transform's input is bf16(x * r * g), r = 1 / sqrt(mean(x^2) + eps), formed in registers with the
 * arithmetic and the rounding of pq_rmsnorm, so the result equals pq_rmsnorm followed by pq_hadamard_quant_act with
 * had_block = K bit for bit while the normalised tensor never goes to memory.
 *   K a power of two in [128, 8192] (the row is one transform block); g bf16 [K], 4-byte aligned. */
pq_status pq_rmsnorm_hadamard_quant_act(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, const void* g, float eps,
                                        int64_t row_begin, const float* s_a, uint8_t* xq, void* stream);

/* ---------------------------------------------------------------------------------------------
 * W4A4 linear layer (Sec. 3: low-bit matrix multiplication; Table 1, O2):
 *     acc[t, n] = sum_k xq[t, k] * wq[n, k]          exact, int32
 *     out[t, n] = bf16( acc[t, n] * s_a * s_w[n] )   for rows t >= row_begin
 *   xq   u8 [M, K/2], wq u8 [N, K/2] dense packed rows, bases 16-byte aligned
 *   s_a  f32 scalar (device), s_w f32 [N] (device)
 *   out  bf16 [M, N], row stride ldo elements
 *   acc_dbg  nullable int32 [M, N] dense: receives the raw accumulators (parity checks)
 *   K % 32 == 0, K <= 65536. Output rows below row_begin are left untouched.
 * Shapes with M - row_begin > 16 run on the tensor-core kernel (TMA + tcgen05, kind::i8);
 * smaller M runs the weight-streaming kernel. No workspace is needed (ws may be NULL).
 * Weights are static (Sec. 3: quantized offline): the weight-streaming kernel starts fetching wq
 * while the kernel before it in the stream is still draining (programmatic dependent launch), and
 * only xq, the scales and out are ordered behind that kernel. wq (and wsum of the _asym call)
 * must therefore be complete before the kernel that precedes this call in the stream starts.
 * Weights written earlier in the same stream by pq_quant_weights / pq_weight_code_sums or by a copy
 * always are: those never let a successor start early. This holds for pq_w4a4_gemm, pq_w4a8_gemm,
 * pq_w4a4_gemm_rows and pq_w4a4_gemm_asym alike. */
size_t pq_w4a4_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
pq_status pq_w4a4_gemm(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w,
                       void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int64_t row_begin, int32_t* acc_dbg,
                       void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * W4A8 linear layer (the W4A8KV4 precision of Sec. 5.1; Eq. 1 with N = 8; static per-tensor
 * activations as in Table 1, O2). The same pipeline with one signed byte per activation code:
 *     xq8 = clamp(round_half_even(y / s_a), -128, 127)     y the rotated row, as above
 *     *s_a = max(*s_a, max |y| / 127)                      calibration helper
 *     acc[t, n] = sum_k xq8[t, k] * wq[n, k]   exact, int32;   out[t, n] = bf16(acc * s_a * s_w[n])
 *   xq8  s8 [M, K] dense rows, base 16-byte aligned; every other argument as in the 4-bit calls.
 * Above 16 tokens the GEMM runs on the tensor-core kernel (the token bytes go to the MMA operand
 * buffer untouched, only the weights are expanded), else on the weight-streaming kernel;
 * K % 32 == 0, K <= 65536. */
pq_status pq_hadamard_quant_act8(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                 int64_t row_begin, const float* s_a, int8_t* xq8, void* stream);
pq_status pq_calib_act_scale8(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                              int64_t row_begin, float* s_a, void* stream);
/* The 4-bit quantizer of pq_hadamard_quant_act (same step s_a = max|y| / 7, same codes in [-8, 7], bit for bit) with
 * the codes stored one per byte in the layout of pq_hadamard_quant_act8: xq8 s8 [M, K], 16-byte aligned. Given to
 * pq_w4a8_gemm with that s_a, the sums and outputs are those of pq_w4a4_gemm on the packed codes, and the prefill
 * kernel skips the expansion of the token operand; the activation tensor is twice as large. */
pq_status pq_hadamard_quant_act_c8(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                   int64_t row_begin, const float* s_a, int8_t* xq8, void* stream);
pq_status pq_w4a8_gemm(pq_ctx* ctx, const int8_t* xq8, const uint8_t* wq, const float* s_a, const float* s_w, void* out,
                       int64_t ldo, int64_t M, int64_t N, int64_t K, int64_t row_begin, int32_t* acc_dbg, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Per-token dynamic activations (Table 1, O1; Sec. 3 "Dynamic and Static": the step is computed online
 * from every token instead of offline per tensor). Symmetric form of Eq. 1 with one clipping factor per
 * layer shared by all tokens:
 *     s_tok[t] = clip * max_k |y[t, k]| / 7          pq_dyn_act_scale   (first pass; 0 < clip <= 1)
 *     xq[t, :] = pack(clamp(rne(y[t, :] / s_tok[t]), -8, 7))   pq_hadamard_quant_act_rows (second pass)
 *     out[t, n] = bf16(acc[t, n] * s_tok[t] * s_w[n])          pq_w4a4_gemm_rows
 *   s_tok  f32 [M] on the device; rows below row_begin are neither read nor written; an all-zero row
 *   gets step 0 and codes 0. Every other argument as in the static calls; the GEMM picks its kernel as
 *   pq_w4a4_gemm does. */
pq_status pq_dyn_act_scale(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                           int64_t row_begin, float clip, float* s_tok, void* stream);
/* The first and the second pass in one call (same passage): s_tok [M] and xq [M, K/2] are both outputs, with the bits
 * the two calls give. When a row is a single transform block of 2048 or more elements (had_block == K) the activations
 * are read once and the call is one launch; otherwise it runs the two passes. */
pq_status pq_dyn_hadamard_quant_act(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                    int64_t row_begin, float clip, float* s_tok, uint8_t* xq, void* stream);
pq_status pq_hadamard_quant_act_rows(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                     int64_t row_begin, const float* s_tok, uint8_t* xq, void* stream);
pq_status pq_w4a4_gemm_rows(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_tok, const float* s_w,
                            void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int64_t row_begin,
                            int32_t* acc_dbg, void* stream);

/* ---------------------------------------------------------------------------------------------
 * KV cache with a full-precision prefix region and a 4-bit region (Sec. 4.2, Eq. 3; Table 1, O2:
 * per-head static KV scales). All buffers are the caller's.
 *   prefix_k, prefix_v  fp16 [Hkv, n_prefix, D]  K/V of the prefixed tokens, computed once by the
 *                       full-precision model and shared by every sequence
 *   kq, vq              u8 [B, Hkv, Tmax, D/2]   packed codes of the ordinary tokens
 *   s_k, s_v            f32 [Hkv]                static per-head steps
 *   len                 int32 [B] on the device  number of 4-bit entries of each sequence
 * D must be 128; Hq a multiple of Hkv with Hq / Hkv <= 8; kq, vq, prefix_k and prefix_v 16-byte aligned.
 *
 * Group-wise dynamic KV (Table 1, O1: the comparison setting; group size 128 = one (token, head) vector): when
 * sk_tok and sv_tok are both non-null, every cached vector carries its own step max |x| / 7, computed when the
 * token is written, in
 *   sk_tok, sv_tok      f32 [B, Hkv, Tmax]       (s_k, s_v are then not used and may be null)
 * pq_kv4_append(_strided) writes codes and steps, pq_decode_attn_kv4_prefix and pq_prefill_attn_kv4_prefix scale
 * every key's score and every value row by the key's own step. The one-launch forms (pq_kv4_append_decode_attn,
 * pq_rope_kv4_append) and the allocation-free entry point serve the static setting only (PQ_ERR_UNSUPPORTED). */
typedef struct pq_kv4_cache {
  const void* prefix_k;
  const void* prefix_v;
  uint8_t* kq;
  uint8_t* vq;
  const float* s_k;
  const float* s_v;
  int32_t* len;
  int32_t B, Hq, Hkv, D, n_prefix, Tmax;
  float* sk_tok; /* null in the static setting */
  float* sv_tok;
} pq_kv4_cache;

/* Calibration helper for the static per-head KV steps (Table 1, O2): over a calibration batch
 * x bf16 [n_tok, Hkv, D] with ld_tok elements between tokens, s[h] = max(s[h], max |x[:, h, :]| / 7).
 * s must be initialised by the caller (0 to start); K and V are calibrated by separate calls. */
pq_status pq_calib_kv_scale(pq_ctx* ctx, const void* x, int64_t n_tok, int32_t Hkv, int32_t D, int64_t ld_tok, float* s,
                            void* stream);

/* Quantize-on-write: k, v bf16 [B, T_new, Hkv, D] are quantized with s_k[h], s_v[h] and written at
 * positions len[b] .. len[b]+T_new-1, then len[b] += T_new (on the device, in stream order).
 * If any sequence would exceed Tmax nothing is written, len is unchanged and PQ_ERR_SHAPE is
 * left in the status word. */
pq_status pq_kv4_append(pq_ctx* ctx, const pq_kv4_cache* cache, const void* k, const void* v, int32_t T_new,
                        void* stream);
/* The same with ld_tok elements between consecutive tokens of k and of v (ld_tok >= Hkv * D, a multiple
 * of 8): the k and v parts of a concatenated q|k|v projection output are appended without a copy. */
pq_status pq_kv4_append_strided(pq_ctx* ctx, const pq_kv4_cache* cache, const void* k, const void* v, int32_t T_new,
                                int64_t ld_tok, void* stream);

/* Decode attention, one query token per sequence, over [prefix || 4-bit cache] (Eq. 3):
 *     score_j = q . K_j * sm_scale,  K_j = prefix_k[h, j] (j < n_prefix) or s_k[h] * code
 *     out     = softmax(score) . V   with V_j = prefix_v[h, j] or s_v[h] * code
 *   q, out  bf16 [B, Hq, D] (q 16-byte, out 8-byte aligned); query head g reads KV head g / (Hq / Hkv)
 *   ws      scratch of pq_decode_attn_workspace_bytes(cache) bytes, 16-byte aligned
 * Every cached entry is visible (no mask). */
size_t pq_decode_attn_workspace_bytes(const pq_kv4_cache* cache);
pq_status pq_decode_attn_kv4_prefix(pq_ctx* ctx, const pq_kv4_cache* cache, const void* q, void* out, float sm_scale,
                                    void* ws, size_t ws_bytes, void* stream);

/* pq_kv4_append (T_new = 1) and pq_decode_attn_kv4_prefix in one launch: the new token's k, v bf16 [B, 1, Hkv, D]
 * (dense) are quantized and written at position len[b], the attention sees every prefixed key, the cached keys
 * 0 .. len[b] - 1 and the new one (as its dequantized codes, exactly what a later call reads back), and
 * len[b] advances by one. If any sequence is full nothing is appended anywhere, the attention runs over the
 * cache as it is and PQ_ERR_SHAPE is reported through the status word. Arguments as in the two calls.
 * The kernel may be placed while its predecessor in the stream still runs (programmatic dependent launch) and
 * requests its first cache rows before it waits for that predecessor; only q, k and v are read after the wait.
 * The cache rows below len[b], the lengths and the steps must therefore not be written by the two kernels that
 * precede this call in the stream (in a decode loop their last writer is the same layer's call of the step
 * before, many kernels back). pq_decode_attn_kv4_prefix has no such condition: it waits before it reads anything. */
pq_status pq_kv4_append_decode_attn(pq_ctx* ctx, const pq_kv4_cache* cache, const void* k, const void* v, const void* q,
                                    void* out, float sm_scale, void* ws, size_t ws_bytes, void* stream);

/* Causal prefill attention of one sequence over [prefix || 4-bit cache] (Sec. 4.2, Eq. 3): query
 * token t sees every prefixed key and the cached keys 0..t of sequence `seq` (the cache rows must
 * already hold the T tokens: call pq_kv4_append first).
 *     out[t, g, :] = softmax_j(q[t, g, :] . K_j * sm_scale) . V   over j in prefix and j <= t
 *   q  bf16 [T, Hq, D] with ldq elements between tokens (the q part of a concatenated q|k|v output; ldq a
 *   multiple of 8), out bf16 [T, Hq, D] dense, both 16-byte aligned; D = 128; Hq / Hkv in {1, 2, 4, 8};
 *   T <= Tmax; n_prefix <= 64; sm_scale > 0; prefix_k, prefix_v, kq, vq 16-byte aligned. No workspace. */
pq_status pq_prefill_attn_kv4_prefix(pq_ctx* ctx, const pq_kv4_cache* cache, int32_t seq, const void* q, int64_t ldq,
                                     int32_t T, void* out, float sm_scale, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Element-wise glue of a Llama transformer block around the quantized linears (the block of the
 * rotation figure in App. B: RMSNorm -> linears -> rotary embedding -> attention -> SwiGLU, with
 * residual connections). bf16 in, fp32 arithmetic (fp64 angles), one rounding to bf16 out. Every
 * pointer is 16-byte aligned and every leading dimension a multiple of 8 elements.
 *
 *   pq_rmsnorm       y[t,:] = x[t,:] / sqrt(mean(x[t,:]^2) + eps) * g      x, y [M,K], g [K]; K % 8 == 0, K <= 16384
 *   pq_rope          rotate-half pairing, head dim D = 128: for i < 64 and token t at position pos0 + t,
 *                    angle = (pos0 + t) * theta^(-2i/D), y[i] = x[i] cos - x[i+64] sin,
 *                    y[i+64] = x[i+64] cos + x[i] sin       x, y [T,H,D] with ld elements between tokens
 *                    (ld >= H*D, so the q and k heads of a concatenated q|k|v output are rotated in one
 *                    call); y may alias x
 *   pq_rope_rotate   the same followed by the online head-wise rotation R3 (App. B, "Online Rotation": the
 *                    outputs of q_proj and k_proj after RoPE): y = RoPE(x) H_D / sqrt(D) per head, H in
 *                    Sylvester order; scores q . k are unchanged, K is quantized in the rotated basis
 *   pq_silu_mul      y = gate / (1 + exp(-gate)) * up        gate, up [M,F] with row stride ld_in (the two
 *                    halves of a concatenated gate|up GEMM output), y [M,F] with row stride ldy; F % 8 == 0
 *   pq_residual_add  y = a + b over n elements, n % 8 == 0; y may alias a or b */
pq_status pq_rmsnorm(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, const void* g, float eps, void* y,
                     int64_t ldy, void* stream);
pq_status pq_rope(pq_ctx* ctx, const void* x, int64_t T, int32_t H, int32_t D, int64_t ld, int64_t pos0, double theta,
                  void* y, void* stream);
pq_status pq_rope_rotate(pq_ctx* ctx, const void* x, int64_t T, int32_t H, int32_t D, int64_t ld, int64_t pos0, double theta,
                  void* y, void* stream);
pq_status pq_silu_mul(pq_ctx* ctx, const void* gate, const void* up, int64_t M, int64_t F, int64_t ld_in, void* y,
                      int64_t ldy, void* stream);
pq_status pq_residual_add(pq_ctx* ctx, const void* a, const void* b, void* y, int64_t n, void* stream);

/* Rotary embedding and KV4 quantize-on-write of a prefill in one launch (App. B block order: q|k|v projection ->
 * rotary embedding (-> R3) -> cache): qkv bf16 [T, (Hq + 2 Hkv) * D] with ld elements between tokens is the
 * concatenated projection output of T tokens of sequence `seq` at positions pos0 .. pos0 + T - 1. The q and k heads
 * are rotated in place (pq_rope, or pq_rope_rotate when rotate != 0), the rotated k heads and the v heads are
 * quantized with s_k[h], s_v[h] and written at positions len[seq] .. len[seq] + T - 1, and len[seq] += T: the result
 * of pq_rope / pq_rope_rotate followed by pq_kv4_append_strided, bit for bit. If the sequence would exceed Tmax the
 * rotation still happens, nothing is appended and PQ_ERR_SHAPE is left in the status word.
 *   qkv, kq, vq 16-byte aligned, ld a multiple of 8, D = 128. */
pq_status pq_rope_kv4_append(pq_ctx* ctx, const pq_kv4_cache* cache, int32_t seq, void* qkv, int64_t T, int64_t ld, int64_t pos0,
                             double theta, int32_t rotate, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Decode attention for callers that may not allocate. (The paper has no counterpart: this is a
 * packaging variant of pq_decode_attn_kv4_prefix, same kernel, same arguments and result.)
 *
 * Who needs it: code that runs where device allocation is forbidden or unavailable - inside a
 * region that must not synchronise the device, under a memory pool it does not own, in a plug-in
 * that is handed buffers but no allocator, or in a start-up path that runs before an allocator
 * exists. Such callers can create neither a pq_ctx (pq_create allocates) nor a workspace, so this
 * entry point takes neither: the split partials and the ticket counters live in a fixed array
 * inside the library's device image (8 MiB + 16 KiB, held by every GPU that loads the library
 * until the process exits). The caller still passes the inputs and the output.
 *
 *   - Limits: B * Hkv <= 4096 and B * Hkv * splits * (Hq / Hkv) * 520 bytes <= 8 MiB, where
 *     splits = min(32, Tmax / 64, 4 * SM count / (B * Hkv)), at least 1. Anything larger returns
 *     PQ_ERR_WORKSPACE and enqueues nothing. Other argument rules are those of
 *     pq_decode_attn_kv4_prefix.
 *   - It calls no cudaMalloc, cudaFree or other allocating routine. The first call on each device
 *     resolves the array's device address and reads the SM count (with that device current);
 *     make that first call before any stream capture begins.
 *   - Every call on a device shares the one array and the array keeps the previous call's
 *     contents: the counters are cleared in stream order at the start of each call, the partials
 *     are fully rewritten before they are read. Two calls that overlap on the GPU (different
 *     streams, or different host threads without ordering) race on it and give wrong results;
 *     issue them in one stream or order them yourself.
 *   - There is no status word without a context: should a bounded wait inside the kernel run out
 *     (PQ_ERR_TIMEOUT of the regular entry point), this entry point cannot report it and the output
 *     is then undefined. */
pq_status pq_decode_attn_kv4_prefix_noalloc(const pq_kv4_cache* cache, const void* q, void* out, float sm_scale,
                                            void* stream);

/* ---------------------------------------------------------------------------------------------
 * Eq. 1 as printed: asymmetric static per-tensor activation quantizer with a zero point (N = 4),
 *     s = (max y - min y) / 15,  z = -floor(min y / s)        max-min initialisation (gamma = beta = 1);
 *                                                             the zero point takes the floor the equation prints
 *     u = clamp(round_half_even(y / s) + z, 0, 15),           dequantized value s (u - z)
 *     out[t, n] = bf16(s_a * s_w[n] * sum_k (u[t,k] - z) * w[n,k])
 *   pq_calib_act_asym           range of the rotated rows >= row_begin of one calibration batch -> *s_a, *z_a
 *                               (device scalars, overwritten; a constant batch gives s = 1, z = 0)
 *   pq_hadamard_quant_act_asym  xq [M, K/2]: the packed signed nibbles hold u - 8 (the operand format of the
 *                               symmetric path, so the same GEMM kernels read it)
 *   pq_weight_code_sums         wsum[n] = sum_k w[n,k] over the packed codes of pq_quant_weights (offline), K % 8 == 0
 *   pq_w4a4_gemm_asym           the GEMM; its epilogue subtracts (z - 8) * wsum[n] from the exact integer sum
 *                               (acc_dbg, when given, receives sum_k (u - z) w). Other arguments as in pq_w4a4_gemm.
 * Any s, z can be passed to the quantizer and the GEMM; pq_grid_search_act_asym below searches them. */
pq_status pq_calib_act_asym(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block, int64_t row_begin,
                            float* s_a, int32_t* z_a, void* stream);
pq_status pq_hadamard_quant_act_asym(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                     int64_t row_begin, const float* s_a, const int32_t* z_a, uint8_t* xq, void* stream);
pq_status pq_weight_code_sums(pq_ctx* ctx, const uint8_t* wq, int64_t N, int64_t K, int32_t* wsum, void* stream);
pq_status pq_w4a4_gemm_asym(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const int32_t* z_a,
                            const float* s_w, const int32_t* wsum, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K,
                            int64_t row_begin, int32_t* acc_dbg, void* stream);

/* Grid search for the static s and z (Sec. 3, "Initialization of Quantization Parameters": for per-tensor
 * static quantization the parameters are searched directly, by mean squared error). Offline. Over one calibration
 * batch, with mn / mx the range of its rotated rows >= row_begin, the n_grid x n_grid candidates
 *     gamma_i = 1 - i * step,  beta_j = 1 - j * step,  step = (1 - lo) / (n_grid - 1)      (candidate i * n_grid + j)
 *     s = (gamma_i * mx - beta_j * mn) / 15,  z = -floor(beta_j * mn / s) clamped to [0, 15]      (Eq. 1)
 * are formed, sse[c] = sum (y - s (u - z))^2 with u = clamp(round_half_even(y / s) + z, 0, 15) is taken over those
 * rows for each, and the candidate with the smallest error (the first among equals) is written to *s_a, *z_a.
 * Candidate 0 is the max-min pair of pq_calib_act_asym, so the result is never worse than that one. The paper
 * measures the error on block outputs; this entry point measures it on the quantized tensor itself.
 *   n_grid in [1, 16], lo in (0, 1]; cand_s f32 [n_grid^2], cand_z int32 [n_grid^2], sse f64 [n_grid^2] (8-byte
 *   aligned): device buffers of the caller that receive the candidates and their errors. Other arguments as in
 *   pq_calib_act_asym. */
pq_status pq_grid_search_act_asym(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block, int64_t row_begin,
                                  int32_t n_grid, float lo, float* s_a, int32_t* z_a, float* cand_s, int32_t* cand_z, double* sse,
                                  void* stream);

/* Grid search for the clipping factor of per-token dynamic quantization (same passage: gamma is shared by all tokens
 * of a layer and chosen by mean squared error; symmetric form, as pq_dyn_act_scale takes it). Offline. Candidates
 *     gamma_i = 1 - i * (1 - lo) / (n_grid - 1),  i = 0 .. n_grid - 1                 (gamma_0 = 1: no clipping)
 * every row t >= row_begin takes the step gamma_i * s_tok[t] with s_tok[t] = max |y_t| / 7 its unclipped step (the
 * product in fp32; pq_dyn_act_scale(clip = gamma) forms gamma * max / 7 and may differ from it in the last bit),
 * sse[i] = sum (y - s q)^2 with q = clamp(round_half_even(y / s), -8, 7) over those rows, and the factor with the
 * smallest error (the first among equals) is written to *gamma.
 *   n_grid in [1, 256], lo in (0, 1]; s_tok f32 [M] (rows >= row_begin are overwritten with the unclipped steps),
 *   cand f32 [n_grid], sse f64 [n_grid] (8-byte aligned): device buffers of the caller. Other arguments as in
 *   pq_dyn_act_scale. */
pq_status pq_grid_search_clip_dyn(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block, int64_t row_begin,
                                  int32_t n_grid, float lo, float* gamma, float* s_tok, float* cand, double* sse, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Outlier tokens (Sec. 4.1, "Definition of Outlier Token", Eq. 2), the cheap part of the offline analysis
 * that decides which tokens are prefixed:
 *     M[i] = max_c |x[i, c]|,  R[i] = M[i] / median(M),
 *     flags[i] = 1 (upper outlier) when R[i] > eta1, 2 (lower outlier) when 1 / R[i] > eta2, else 0
 *   x bf16 [T, C], row stride ldx (16-byte aligned, C and ldx multiples of 8), T <= 8192;
 *   M, R f32 [T], flags int32 [T], median f32 scalar, all on the device. The median of an even number of
 *   tokens is the mean of the two middle values; ratios and comparisons are fp32. The paper uses
 *   eta1 = 64, eta2 = 8. */
pq_status pq_outlier_tokens(pq_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ldx, float eta1, float eta2, float* M,
                            float* R, int32_t* flags, float* median, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Measurement aid (the paper has no counterpart): n_ctas CTAs (at most one per SM) each issue `iters`
 * tcgen05.mma kind::i8 instructions of 128 x 256 x 32 multiply-accumulates on operands that stay in shared
 * memory, and write the SM clocks from the first issue to the completion of the last into cycles[cta]
 * (device, int64; -1 if the wait ran out). iters * 128 * 256 * 32 / cycles is the integer tensor-core rate
 * per SM and clock that a GEMM reaches when nothing else has to happen: the benchmark's attainable INT8 peak. */
pq_status pq_probe_i8_mma(pq_ctx* ctx, int32_t iters, int64_t* cycles, int32_t n_ctas, void* stream);

/* Failure-detection self-test (the paper has no counterpart): launches one thread that waits on a barrier nothing
 * ever completes. The bounded wait runs out after the context's limit (pq_set_wait_limit; keep it short for this
 * call), PQ_ERR_TIMEOUT is left in the status word, the kernel returns and the context stays usable.
 * waited_clocks (device int64, nullable) receives the SM clocks the wait took. */
pq_status pq_selftest_wait(pq_ctx* ctx, int64_t* waited_clocks, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PQ_H_ */

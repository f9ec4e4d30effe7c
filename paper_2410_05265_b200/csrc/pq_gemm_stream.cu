// W4A4 GEMM for decode-shaped problems (at most 16 tokens): the packed weights are streamed
// from HBM exactly once with 128-bit loads and the kernel is bound by that stream.
//
// One CTA owns 16 output channels; its 8 warps split K in 128-element steps and meet in shared
// memory at the end. Each warp multiplies with the warp-level integer MMA (m16n8k32, s8): the 16
// weight rows are the M side, up to 8 tokens the N side. A lane loads one 16-byte chunk (32 codes)
// from two weight rows and from one token row, expands the nibbles to s8 values scaled by 16
// (even-position codes in one word, odd-position codes in the next) and feeds word pairs to four
// MMAs. Weights and tokens apply the same permutation of k inside a chunk, so the dot product is
// unchanged; the factor 16*16 is shifted out exactly in the epilogue. (Staging the rows through shared
// memory with bulk copies was measured and is slower here: copies below 2 KB do not reach the memory's
// rate, and the short layers are bound by the dependent chain wait -> token rows -> MMA -> store, which
// direct loads keep shortest.)
#include "pq_common.cuh"

namespace {

constexpr int GS_WARPS = 8;
constexpr int GS_THREADS = GS_WARPS * 32;
constexpr int GS_CH = 16;     // output channels per CTA

__device__ __forceinline__ void mma_s8_16832(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void expand(const uint4& w, uint32_t (&o)[8]) {
  o[0] = pq::nib_lo_x16(w.x), o[1] = pq::nib_hi_x16(w.x);
  o[2] = pq::nib_lo_x16(w.y), o[3] = pq::nib_hi_x16(w.y);
  o[4] = pq::nib_lo_x16(w.z), o[5] = pq::nib_hi_x16(w.z);
  o[6] = pq::nib_lo_x16(w.w), o[7] = pq::nib_hi_x16(w.w);
}

// Streaming load of weight bytes that are used once: do not keep them in L1.
__device__ __forceinline__ uint4 ld_stream(const uint8_t* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// 32 s8 activation codes of a K step (two 16-byte loads) in the order the expanded weights have: the
// even-position codes of every eight in one word, the odd-position codes in the next. The value fed to the
// MMA is the code itself (the weights carry their factor 16 alone: the sum is shifted by 4, not 8).
__device__ __forceinline__ void permute_s8(const uint4& lo, const uint4& hi, uint32_t (&o)[8]) {
  o[0] = __byte_perm(lo.x, lo.y, 0x6420), o[1] = __byte_perm(lo.x, lo.y, 0x7531);
  o[2] = __byte_perm(lo.z, lo.w, 0x6420), o[3] = __byte_perm(lo.z, lo.w, 0x7531);
  o[4] = __byte_perm(hi.x, hi.y, 0x6420), o[5] = __byte_perm(hi.x, hi.y, 0x7531);
  o[6] = __byte_perm(hi.z, hi.w, 0x6420), o[7] = __byte_perm(hi.z, hi.w, 0x7531);
}

// HALF_ROWS: the CTA owns 8 output channels instead of 16 (rows 8..15 of the MMA tile stay zero), which
// doubles the CTA count of narrow layers.
// A8: the token operand is one s8 code per element ([M, K] bytes) instead of packed nibbles (W4A8).
// DEEP (long K): batches of two steps in two register buffers, so that the next batch's loads are in flight while
// this one is multiplied; else one buffer of four steps (a K of 4096 is a single batch per warp, and the lower
// register count keeps more CTAs on an SM, which is what the short layers need).
template <bool TWO_GROUPS, bool HALF_ROWS, bool A8, bool DEEP>
__global__ void __launch_bounds__(GS_THREADS)
    gemm_w4a4_stream_kernel(const uint8_t* __restrict__ xq, const uint8_t* __restrict__ wq,
                            const float* __restrict__ s_a, const float* __restrict__ s_w,
                            __nv_bfloat16* __restrict__ out, int64_t ldo, int M, int N, int K,
                            int32_t* __restrict__ acc_dbg, int sa_stride, const int32_t* __restrict__ zp,
                            const int32_t* __restrict__ wsum) {
  __shared__ int red[GS_WARPS][GS_CH][16];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  constexpr int CH = HALF_ROWS ? GS_CH / 2 : GS_CH;  // output channels of this CTA
  const int n0 = blockIdx.x * CH;
  const int kbytes = K / 2;
  const int n_steps = (K + 127) / 128;

  const bool w0_ok = n0 + g < N, w1_ok = !HALF_ROWS && n0 + g + 8 < N;
  const bool x0_ok = g < M, x1_ok = TWO_GROUPS && (g + 8 < M);
  const uint8_t* w0p = wq + static_cast<int64_t>(n0 + g) * kbytes + t * 16;
  const uint8_t* w1p = wq + static_cast<int64_t>(n0 + g + 8) * kbytes + t * 16;
  constexpr int XS = A8 ? 2 : 1;  // activation bytes per packed weight byte
  const uint8_t* x0p = xq + (static_cast<int64_t>(g) * kbytes + t * 16) * XS;
  const uint8_t* x1p = xq + (static_cast<int64_t>(g + 8) * kbytes + t * 16) * XS;

  int c0[4] = {0, 0, 0, 0}, c1[4] = {0, 0, 0, 0};
  const uint4 zero = make_uint4(0, 0, 0, 0);

  // The weights are static, the activations and the output may belong to the kernel before this one
  // in the stream: let the next kernel start early, fetch the first weight chunks, and only then wait
  // for the previous kernel (programmatic dependent launch; both instructions do nothing without it).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // One batch = GS_UNROLL K steps of this warp (their loads are in flight together). Two register buffers: the
  // loads of batch b + 1 are issued before batch b is multiplied, so the memory pipe never drains inside a CTA.
  constexpr int GS_UNROLL = DEEP ? 2 : 4;  // K steps per batch
  struct Batch {
    uint4 wa[GS_UNROLL], wb[HALF_ROWS ? 1 : GS_UNROLL], xa[GS_UNROLL], xb[TWO_GROUPS ? GS_UNROLL : 1];
    uint4 xa2[A8 ? GS_UNROLL : 1], xb2[(A8 && TWO_GROUPS) ? GS_UNROLL : 1];  // second half of a lane's 32 s8 codes
  };
  constexpr int STRIDE = GS_WARPS * GS_UNROLL;
  auto load_w = [&](Batch& b, int base) {
#pragma unroll
    for (int u = 0; u < GS_UNROLL; ++u) {
      const int ks = base + u * GS_WARPS;
      const int off = ks * 64;
      const bool in_k = ks < n_steps && off + t * 16 < kbytes;
      b.wa[u] = (in_k && w0_ok) ? ld_stream(w0p + off) : zero;
      if (!HALF_ROWS) b.wb[u] = (in_k && w1_ok) ? ld_stream(w1p + off) : zero;
    }
  };
  auto load_x = [&](Batch& b, int base) {
#pragma unroll
    for (int u = 0; u < GS_UNROLL; ++u) {
      const int ks = base + u * GS_WARPS;
      const int off = ks * 64;
      const bool in_k = ks < n_steps && off + t * 16 < kbytes;
      b.xa[u] = (in_k && x0_ok) ? __ldg(reinterpret_cast<const uint4*>(x0p + off * XS)) : zero;
      if (TWO_GROUPS) b.xb[u] = (in_k && x1_ok) ? __ldg(reinterpret_cast<const uint4*>(x1p + off * XS)) : zero;
      if (A8) {
        b.xa2[u] = (in_k && x0_ok) ? __ldg(reinterpret_cast<const uint4*>(x0p + off * XS) + 1) : zero;
        if (TWO_GROUPS) b.xb2[u] = (in_k && x1_ok) ? __ldg(reinterpret_cast<const uint4*>(x1p + off * XS) + 1) : zero;
      }
    }
  };
  auto multiply = [&](const Batch& b) {
#pragma unroll
    for (int u = 0; u < GS_UNROLL; ++u) {
      uint32_t ea[8], eb[8], ex[8];
      expand(b.wa[u], ea);
      if (HALF_ROWS) {
#pragma unroll
        for (int i = 0; i < 8; ++i) eb[i] = 0u;
      } else {
        expand(b.wb[u], eb);
      }
      if (A8) permute_s8(b.xa[u], b.xa2[u], ex);
      else expand(b.xa[u], ex);
#pragma unroll
      for (int j = 0; j < 4; ++j) mma_s8_16832(c0, ea[2 * j], eb[2 * j], ea[2 * j + 1], eb[2 * j + 1], ex[2 * j], ex[2 * j + 1]);
      if (TWO_GROUPS) {
        if (A8) permute_s8(b.xb[u], b.xb2[u], ex);
        else expand(b.xb[u], ex);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mma_s8_16832(c1, ea[2 * j], eb[2 * j], ea[2 * j + 1], eb[2 * j + 1], ex[2 * j], ex[2 * j + 1]);
      }
    }
  };
  // what the epilogue needs is requested now, not after the reduction: the output channel's step (static, like the
  // weights) ahead of the wait, the token's step and the zero point right after it
  const int e_tok = threadIdx.x & 15, e_ch = threadIdx.x >> 4;  // 16 channels x 16 tokens: consecutive threads read consecutive words
  const int e_n = n0 + e_ch;
  const bool e_ok = e_tok < M && e_n < N && e_ch < CH && (TWO_GROUPS || e_tok < 8);
  const float e_sw = e_ok ? __ldg(s_w + e_n) : 0.0f;
  const int e_wsum = (e_ok && zp) ? __ldg(wsum + e_n) : 0;
  Batch b0;
  int base = warp;
  if (base < n_steps) load_w(b0, base);               // static weights: requested ahead of the wait
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the token rows may come from the previous kernel
  const float e_sa = e_ok ? __ldg(s_a + e_tok * sa_stride) : 0.0f;  // stride 1: one step per token
  const int e_zp8 = (e_ok && zp) ? __ldg(zp) - 8 : 0;
  if (base < n_steps) load_x(b0, base);
  if (DEEP) {
    Batch b1;
    while (base < n_steps) {
      if (base + STRIDE < n_steps) load_w(b1, base + STRIDE), load_x(b1, base + STRIDE);
      multiply(b0);
      base += STRIDE;
      if (base >= n_steps) break;
      if (base + STRIDE < n_steps) load_w(b0, base + STRIDE), load_x(b0, base + STRIDE);
      multiply(b1);
      base += STRIDE;
    }
  } else {
    while (base < n_steps) {
      multiply(b0);
      base += STRIDE;
      if (base < n_steps) load_w(b0, base), load_x(b0, base);
    }
  }
  // accumulator layout: c[0], c[1] -> channel g, tokens 2t, 2t+1; c[2], c[3] -> channel g+8
  red[warp][g][2 * t] = c0[0];
  red[warp][g][2 * t + 1] = c0[1];
  red[warp][g + 8][2 * t] = c0[2];
  red[warp][g + 8][2 * t + 1] = c0[3];
  if (TWO_GROUPS) {
    red[warp][g][8 + 2 * t] = c1[0];
    red[warp][g][8 + 2 * t + 1] = c1[1];
    red[warp][g + 8][8 + 2 * t] = c1[2];
    red[warp][g + 8][8 + 2 * t + 1] = c1[3];
  }
  __syncthreads();
  if (e_ok) {
    int s = 0;
#pragma unroll
    for (int w = 0; w < GS_WARPS; ++w) s += red[w][e_ch][e_tok];
    s >>= A8 ? 4 : 8;            // exact: every product carries the factor 16 once per 4-bit operand
    if (zp) s -= e_zp8 * e_wsum;  // zero-point form of Eq. 1: sum (u - z) w from sum (u - 8) w
    const float f = static_cast<float>(s) * (e_sa * e_sw);
    out[static_cast<int64_t>(e_tok) * ldo + e_n] = __float2bfloat16_rn(f);
    if (acc_dbg) acc_dbg[static_cast<int64_t>(e_tok) * N + e_n] = s;
  }
}

}  // namespace

// Rows [0, M) of xq/out, M <= 16 (the caller has already applied row_begin).
template <bool TWO, bool HALF, bool A8, bool DEEP>
static pq_status launch_stream_k(const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w, void* out,
                               int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg, cudaStream_t st,
                               int sa_stride, const int32_t* zp, const int32_t* wsum) {
  const int ch = HALF ? GS_CH / 2 : GS_CH;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>((N + ch - 1) / ch));
  cfg.blockDim = dim3(GS_THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  // the kernel may start while its predecessor in the stream drains; it waits for it on the device
  // before it touches anything but the weights
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemm_w4a4_stream_kernel<TWO, HALF, A8, DEEP>, xq, wq, s_a, s_w, static_cast<__nv_bfloat16*>(out), ldo,
                         static_cast<int>(M), static_cast<int>(N), static_cast<int>(K), acc_dbg, sa_stride, zp, wsum) != cudaSuccess)
    return PQ_ERR_CUDA;
  return pq_launch_status();
}

template <bool TWO, bool HALF, bool A8>
static pq_status launch_stream(const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w, void* out,
                               int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg, cudaStream_t st,
                               int sa_stride, const int32_t* zp, const int32_t* wsum) {
  // more than one four-step batch per warp: pipeline the batches
  if (K > GS_WARPS * 4 * 128) return launch_stream_k<TWO, HALF, A8, true>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum);
  return launch_stream_k<TWO, HALF, A8, false>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum);
}

pq_status pq_gemm_stream_launch(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w,
                                void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg,
                                cudaStream_t st, bool per_token, bool a8, const int32_t* zp, const int32_t* wsum) {
  const int sa_stride = per_token ? 1 : 0;  // s_a is then an array of M per-token steps
  // 8 channels per CTA when all those CTAs are resident at once (four 64-register CTAs per SM), else 16: CTAs of a
  // second wave start after the programmatic launch's early weight requests have been spent (q|k|v with 768 CTAs of 8
  // channels: 4.8 us, with 384 of 16: 3.2 us). Only for up to 8 tokens: with two token groups the narrower CTA repeats
  // too much of the activation expansion.
  const bool half = M <= 8 && (N + GS_CH / 2 - 1) / (GS_CH / 2) <= 4LL * ctx->sm_count;
  if (a8) {
    if (M <= 8)
      return half ? launch_stream<false, true, true>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum)
                  : launch_stream<false, false, true>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum);
    return launch_stream<true, false, true>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum);
  }
  if (M <= 8)
    return half ? launch_stream<false, true, false>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum)
                : launch_stream<false, false, false>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum);
  return launch_stream<true, false, false>(xq, wq, s_a, s_w, out, ldo, M, N, K, acc_dbg, st, sa_stride, zp, wsum);
}

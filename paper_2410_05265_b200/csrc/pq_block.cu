// Element-wise glue of a Llama transformer block around the W4A4 linears and the KV4 attention
// (App. B places the rotations inside such a block): RMSNorm, rotary embedding, SwiGLU gate and
// residual addition. Each kernel reads bf16, computes in fp32 (angles in fp64) and rounds once to
// bf16, so every tensor that crosses HBM is a bf16 tensor. All are bound by HBM bandwidth.
#include <math.h>

#include "pq_common.cuh"

namespace {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// One rotate-half pair: (a, b) -> (a cos - b sin, b cos + a sin), spelled out in single operations so that every
// kernel that rotates (stand-alone, with R3, fused with the KV4 append) produces the same bits.
__device__ __forceinline__ void rope_pair(float a, float b, float c, float s, float& lo, float& hi) {
  lo = __fmaf_rn(a, c, -__fmul_rn(b, s));
  hi = __fmaf_rn(b, c, __fmul_rn(a, s));
}

// ---- RMSNorm: y = x * rsqrt(mean(x^2) + eps) * g; one CTA per row, the row is read once ---------
constexpr int RN_THREADS = 256;
constexpr int RN_MAX_VEC = 8;  // 8-element vectors per thread kept in registers: K <= 256 * 8 * 8 = 16384

__global__ void __launch_bounds__(RN_THREADS)
    rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const __nv_bfloat16* __restrict__ g, float eps,
                   __nv_bfloat16* __restrict__ y, int64_t ldy, int64_t M, int K) {
  __shared__ float red[RN_THREADS / 32];
  __shared__ float s_r;
  const int n_vec = K / 8;
  for (int64_t row = blockIdx.x; row < M; row += gridDim.x) {
    const uint4* xr = reinterpret_cast<const uint4*>(x + row * ldx);
    uint4 v[RN_MAX_VEC];
    float ss = 0.0f;
#pragma unroll
    for (int i = 0; i < RN_MAX_VEC; ++i) {
      const int j = threadIdx.x + i * RN_THREADS;
      v[i] = j < n_vec ? __ldg(xr + j) : make_uint4(0, 0, 0, 0);
      const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) ss = fmaf(bf16_lo(w[e]), bf16_lo(w[e]), fmaf(bf16_hi(w[e]), bf16_hi(w[e]), ss));
    }
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.0f;
      for (int i = 0; i < RN_THREADS / 32; ++i) t += red[i];
      s_r = 1.0f / sqrtf(t / static_cast<float>(K) + eps);
    }
    __syncthreads();
    const float r = s_r;
    uint4* yr = reinterpret_cast<uint4*>(y + row * ldy);
    const uint4* gr = reinterpret_cast<const uint4*>(g);
#pragma unroll
    for (int i = 0; i < RN_MAX_VEC; ++i) {
      const int j = threadIdx.x + i * RN_THREADS;
      if (j < n_vec) {
        const uint4 gv = __ldg(gr + j);
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w}, gw[4] = {gv.x, gv.y, gv.z, gv.w};
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e] = pack_bf16(bf16_lo(w[e]) * r * bf16_lo(gw[e]), bf16_hi(w[e]) * r * bf16_hi(gw[e]));
        yr[j] = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
    __syncthreads();
  }
}

// ---- rotary embedding, rotate-half pairing, head_dim 128 -----------------------------------------
// One CTA per token: 64 threads build cos/sin of pos * theta^(-2i/128) in fp64 (positions reach the
// thousands, where an fp32 angle already costs a visible part of a bf16 ulp), then every thread
// rotates 8-element vectors of the token's heads.
constexpr int RP_THREADS = 128;

__global__ void __launch_bounds__(RP_THREADS)
    rope_kernel(const __nv_bfloat16* x, __nv_bfloat16* y, int64_t T, int H, int64_t ld, int64_t pos0,
                double log2_theta) {
  __shared__ float cs[64], sn[64];
  for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
    if (threadIdx.x < 64) {
      const double inv_freq = exp2(-2.0 * static_cast<double>(threadIdx.x) / 128.0 * log2_theta);
      double s, c;
      sincos(static_cast<double>(pos0 + t) * inv_freq, &s, &c);
      cs[threadIdx.x] = static_cast<float>(c), sn[threadIdx.x] = static_cast<float>(s);
    }
    __syncthreads();
    // a work item = (head, group of 8 consecutive i in [0, 64)): reads x[i..i+7] and x[64+i..64+i+7]
    for (int item = threadIdx.x; item < H * 8; item += RP_THREADS) {
      const int hd = item >> 3, i0 = (item & 7) * 8;
      const __nv_bfloat16* px = x + t * ld + hd * 128;
      __nv_bfloat16* py = y + t * ld + hd * 128;
      const uint4 a = *reinterpret_cast<const uint4*>(px + i0), b = *reinterpret_cast<const uint4*>(px + 64 + i0);  // y may alias x
      const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
      uint32_t oa[4], ob[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float c0 = cs[i0 + 2 * e], s0 = sn[i0 + 2 * e], c1 = cs[i0 + 2 * e + 1], s1 = sn[i0 + 2 * e + 1];
        const float a0 = bf16_lo(aw[e]), a1 = bf16_hi(aw[e]), b0 = bf16_lo(bw[e]), b1 = bf16_hi(bw[e]);
        float l0, h0, l1, h1;
        rope_pair(a0, b0, c0, s0, l0, h0);
        rope_pair(a1, b1, c1, s1, l1, h1);
        oa[e] = pack_bf16(l0, l1);
        ob[e] = pack_bf16(h0, h1);
      }
      *reinterpret_cast<uint4*>(py + i0) = make_uint4(oa[0], oa[1], oa[2], oa[3]);
      *reinterpret_cast<uint4*>(py + 64 + i0) = make_uint4(ob[0], ob[1], ob[2], ob[3]);
    }
    __syncthreads();
  }
}

// One head of RoPE + R3 in the warp layout (lane l holds elements 2l, 2l+1, 64+2l, 65+2l): returns the two packed
// bf16 words (elements 2l, 2l+1 and 64+2l, 65+2l).
__device__ __forceinline__ void rope_rotate_head(float a0, float a1, float b0, float b1, float c0, float s0, float c1, float s1,
                                                 int lane, uint32_t& pa, uint32_t& pb) {
  float v0, v1, v2, v3;
  rope_pair(a0, b0, c0, s0, v0, v2);
  rope_pair(a1, b1, c1, s1, v1, v3);
  float u;
  u = v0, v0 = u + v1, v1 = u - v1;  // index bit 0
  u = v2, v2 = u + v3, v3 = u - v3;
  u = v0, v0 = u + v2, v2 = u - v2;  // index bit 6
  u = v1, v1 = u + v3, v3 = u - v3;
#pragma unroll
  for (int m = 1; m < 32; m <<= 1) {  // index bits 1..5: the upper partner holds the difference
    const bool up = lane & m;
    const float o0 = __shfl_xor_sync(0xffffffffu, v0, m), o1 = __shfl_xor_sync(0xffffffffu, v1, m);
    const float o2 = __shfl_xor_sync(0xffffffffu, v2, m), o3 = __shfl_xor_sync(0xffffffffu, v3, m);
    v0 = up ? o0 - v0 : v0 + o0, v1 = up ? o1 - v1 : v1 + o1;
    v2 = up ? o2 - v2 : v2 + o2, v3 = up ? o3 - v3 : v3 + o3;
  }
  const float norm = 0.08838834764831845f;  // 1 / sqrt(128)
  pa = pack_bf16(v0 * norm, v1 * norm);
  pb = pack_bf16(v2 * norm, v3 * norm);
}

// Rotary embedding followed by the online head-wise rotation R3 (App. B): y = RoPE(x) H_128 / sqrt(128)
// per head, H in Sylvester order. One warp per head: lane l holds the elements 2l, 2l+1, 64+2l, 65+2l
// (both rotate-half pairs are inside the lane); the butterflies on index bits 0 and 6 run inside
// the lane, those on bits 1..5 across lanes. fp32 throughout, one rounding to bf16.
__global__ void __launch_bounds__(RP_THREADS)
    rope_rotate_kernel(const __nv_bfloat16* x, __nv_bfloat16* y, int64_t T, int H, int64_t ld, int64_t pos0,
                       double log2_theta) {
  __shared__ float cs[64], sn[64];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
    if (threadIdx.x < 64) {
      const double inv_freq = exp2(-2.0 * static_cast<double>(threadIdx.x) / 128.0 * log2_theta);
      double s, c;
      sincos(static_cast<double>(pos0 + t) * inv_freq, &s, &c);
      cs[threadIdx.x] = static_cast<float>(c), sn[threadIdx.x] = static_cast<float>(s);
    }
    __syncthreads();
    const float c0 = cs[2 * lane], s0 = sn[2 * lane], c1 = cs[2 * lane + 1], s1 = sn[2 * lane + 1];
    for (int hd = warp; hd < H; hd += RP_THREADS / 32) {
      const __nv_bfloat16* px = x + t * ld + hd * 128;
      __nv_bfloat16* py = y + t * ld + hd * 128;
      const uint32_t wa = *reinterpret_cast<const uint32_t*>(px + 2 * lane);  // y may alias x: the warp reads its head first
      const uint32_t wb = *reinterpret_cast<const uint32_t*>(px + 64 + 2 * lane);
      const float a0 = bf16_lo(wa), a1 = bf16_hi(wa), b0 = bf16_lo(wb), b1 = bf16_hi(wb);
      uint32_t pa, pb;
      rope_rotate_head(a0, a1, b0, b1, c0, s0, c1, s1, lane, pa, pb);
      __syncwarp();
      *reinterpret_cast<uint32_t*>(py + 2 * lane) = pa;
      *reinterpret_cast<uint32_t*>(py + 64 + 2 * lane) = pb;
    }
    __syncthreads();
  }
}

// Rotary embedding (optionally + R3) of the q and k heads of a concatenated q|k|v row, in place, and the KV4
// quantize-on-write of the rotated k heads and of the v heads in the same launch (what pq_rope / pq_rope_rotate followed
// by pq_kv4_append_strided do, bit for bit). One CTA per token, one warp per head in the layout above; a lane's four
// elements are two bytes of the head's packed row. The last CTA to finish advances the sequence's length.
__device__ __forceinline__ int kv_code(float x, float s) { return max(-8, min(7, __float2int_rn(__fdiv_rn(x, s)))); }

__global__ void __launch_bounds__(RP_THREADS)
    rope_kv4_append_kernel(__nv_bfloat16* qkv, int64_t T, int Hq, int Hkv, int64_t ld, int64_t pos0, double log2_theta, int rotate,
                           uint8_t* __restrict__ kq, uint8_t* __restrict__ vq, const float* __restrict__ s_k,
                           const float* __restrict__ s_v, int32_t* len, int Tmax, int32_t* status, uint32_t* ticket) {
  __shared__ float cs[64], sn[64];
  __shared__ int last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int len0 = __ldcg(len);
  const bool bad = len0 < 0 || len0 + T > Tmax;  // every CTA reaches the same verdict: then nothing is appended
  const int n_heads = Hq + 2 * Hkv;
  for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
    if (threadIdx.x < 64) {
      const double inv_freq = exp2(-2.0 * static_cast<double>(threadIdx.x) / 128.0 * log2_theta);
      double s, c;
      sincos(static_cast<double>(pos0 + t) * inv_freq, &s, &c);
      cs[threadIdx.x] = static_cast<float>(c), sn[threadIdx.x] = static_cast<float>(s);
    }
    __syncthreads();
    const float c0 = cs[2 * lane], s0 = sn[2 * lane], c1 = cs[2 * lane + 1], s1 = sn[2 * lane + 1];
    for (int hd = warp; hd < n_heads; hd += RP_THREADS / 32) {
      __nv_bfloat16* px = qkv + t * ld + hd * 128;
      uint32_t pa = *reinterpret_cast<const uint32_t*>(px + 2 * lane), pb = *reinterpret_cast<const uint32_t*>(px + 64 + 2 * lane);
      if (hd < Hq + Hkv) {  // q and k heads are rotated; v passes through
        const float a0 = bf16_lo(pa), a1 = bf16_hi(pa), b0 = bf16_lo(pb), b1 = bf16_hi(pb);
        if (rotate) {
          rope_rotate_head(a0, a1, b0, b1, c0, s0, c1, s1, lane, pa, pb);
        } else {
          float l0, h0, l1, h1;
          rope_pair(a0, b0, c0, s0, l0, h0);
          rope_pair(a1, b1, c1, s1, l1, h1);
          pa = pack_bf16(l0, l1), pb = pack_bf16(h0, h1);
        }
        *reinterpret_cast<uint32_t*>(px + 2 * lane) = pa;
        *reinterpret_cast<uint32_t*>(px + 64 + 2 * lane) = pb;
      }
      if (hd >= Hq && !bad) {
        const bool is_v = hd >= Hq + Hkv;
        const int kvh = is_v ? hd - Hq - Hkv : hd - Hq;
        const float s = __ldg((is_v ? s_v : s_k) + kvh);
        uint8_t* row = (is_v ? vq : kq) + (static_cast<int64_t>(kvh) * Tmax + len0 + t) * 64;
        row[lane] = static_cast<uint8_t>((kv_code(bf16_lo(pa), s) & 0xF) | ((kv_code(bf16_hi(pa), s) & 0xF) << 4));
        row[32 + lane] = static_cast<uint8_t>((kv_code(bf16_lo(pb), s) & 0xF) | ((kv_code(bf16_hi(pb), s) & 0xF) << 4));
      }
    }
    __syncthreads();
  }
  if (bad) {
    if (blockIdx.x == 0 && threadIdx.x == 0) pq::report(status, PQ_ERR_SHAPE);
    return;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    if (last) {
      *len = len0 + static_cast<int>(T);
      *ticket = 0;
    }
  }
}

// ---- SwiGLU gate: y = gate / (1 + exp(-gate)) * up ------------------------------------------------
constexpr int EW_THREADS = 256;

__global__ void __launch_bounds__(EW_THREADS)
    silu_mul_kernel(const __nv_bfloat16* __restrict__ gate, const __nv_bfloat16* __restrict__ up, int64_t ld_in,
                    __nv_bfloat16* __restrict__ y, int64_t ldy, int64_t M, int F) {
  const int vec_per_row = F / 8;
  const int64_t n_vec = M * vec_per_row;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * EW_THREADS + threadIdx.x; i < n_vec;
       i += static_cast<int64_t>(gridDim.x) * EW_THREADS) {
    const int64_t row = i / vec_per_row;
    const int col = static_cast<int>(i % vec_per_row) * 8;
    const uint4 gv = __ldg(reinterpret_cast<const uint4*>(gate + row * ld_in + col));
    const uint4 uv = __ldg(reinterpret_cast<const uint4*>(up + row * ld_in + col));
    const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, uw[4] = {uv.x, uv.y, uv.z, uv.w};
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float g0 = bf16_lo(gw[e]), g1 = bf16_hi(gw[e]);
      o[e] = pack_bf16(pq::silu_mul_f32(g0, bf16_lo(uw[e])), pq::silu_mul_f32(g1, bf16_hi(uw[e])));
    }
    *reinterpret_cast<uint4*>(y + row * ldy + col) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// ---- residual: y = a + b -----------------------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
    add_kernel(const __nv_bfloat16* a, const __nv_bfloat16* b, __nv_bfloat16* y,
               int64_t n_vec) {
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * EW_THREADS + threadIdx.x; i < n_vec;
       i += static_cast<int64_t>(gridDim.x) * EW_THREADS) {
    const uint4 av = reinterpret_cast<const uint4*>(a)[i], bv = reinterpret_cast<const uint4*>(b)[i];  // y may alias a or b
    const uint32_t aw[4] = {av.x, av.y, av.z, av.w}, bw[4] = {bv.x, bv.y, bv.z, bv.w};
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) o[e] = pack_bf16(bf16_lo(aw[e]) + bf16_lo(bw[e]), bf16_hi(aw[e]) + bf16_hi(bw[e]));
    reinterpret_cast<uint4*>(y)[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// ---- calibration helper: per-head static KV step = max |x| / 7 over a calibration batch ------------
__global__ void __launch_bounds__(EW_THREADS)
    calib_kv_scale_kernel(const __nv_bfloat16* __restrict__ x, int64_t n_tok, int Hkv, int64_t ld_tok,
                          float* __restrict__ s) {
  const int lane = threadIdx.x & 31;
  const int64_t n_rows = n_tok * Hkv;  // one warp per (token, head) row of 128 values
  for (int64_t row = (static_cast<int64_t>(blockIdx.x) * EW_THREADS + threadIdx.x) >> 5; row < n_rows;
       row += (static_cast<int64_t>(gridDim.x) * EW_THREADS) >> 5) {
    const int64_t tok = row / Hkv;
    const int h = static_cast<int>(row % Hkv);
    const uint2 w = __ldg(reinterpret_cast<const uint2*>(x + tok * ld_tok + h * 128) + lane);
    float m = fmaxf(fmaxf(fabsf(bf16_lo(w.x)), fabsf(bf16_hi(w.x))), fmaxf(fabsf(bf16_lo(w.y)), fabsf(bf16_hi(w.y))));
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0 && m > 0.0f) atomicMax(reinterpret_cast<int*>(s + h), __float_as_int(__fdiv_rn(m, 7.0f)));
  }
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
int grid_for(pq_ctx* ctx, int64_t work_items, int per_cta) {
  int64_t g = (work_items + per_cta - 1) / per_cta;
  const int64_t cap = 16LL * ctx->sm_count;
  return static_cast<int>(g < 1 ? 1 : (g > cap ? cap : g));
}

}  // namespace

pq_status pq_rmsnorm_pow2_launch(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, const void* g, float eps, void* y,
                                 int64_t ldy, void* stream);

extern "C" pq_status pq_rmsnorm(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, const void* g, float eps,
                                void* y, int64_t ldy, void* stream) {
  if (!ctx || !x || !g || !y) return PQ_ERR_INVALID_ARG;
  if (M < 0 || K <= 0 || ldx < K || ldy < K) return PQ_ERR_INVALID_ARG;
  if (K % 8 != 0 || K > RN_THREADS * RN_MAX_VEC * 8) return PQ_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(g) || !aligned16(y) || ldx % 8 != 0 || ldy % 8 != 0) return PQ_ERR_ALIGN;
  if (M == 0) return PQ_OK;
  // a row that is one transform block of the online rotation takes the first pass of that kernel, so that
  // pq_rmsnorm_hadamard_quant_act equals this call followed by pq_hadamard_quant_act bit for bit
  if ((K & (K - 1)) == 0 && K >= 128 && K <= 8192) return pq_rmsnorm_pow2_launch(ctx, x, M, K, ldx, g, eps, y, ldy, stream);
  rmsnorm_kernel<<<grid_for(ctx, M, 1), RN_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(x), ldx, static_cast<const __nv_bfloat16*>(g), eps,
      static_cast<__nv_bfloat16*>(y), ldy, M, static_cast<int>(K));
  return pq_launch_status();
}

extern "C" pq_status pq_rope(pq_ctx* ctx, const void* x, int64_t T, int32_t H, int32_t D, int64_t ld, int64_t pos0,
                             double theta, void* y, void* stream) {
  if (!ctx || !x || !y) return PQ_ERR_INVALID_ARG;
  if (T < 0 || H <= 0 || pos0 < 0 || !(theta > 1.0) || ld < static_cast<int64_t>(H) * 128) return PQ_ERR_INVALID_ARG;
  if (D != 128) return PQ_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(y) || ld % 8 != 0) return PQ_ERR_ALIGN;
  if (T == 0) return PQ_OK;
  rope_kernel<<<grid_for(ctx, T, 1), RP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(y), T, H, ld, pos0, log2(theta));
  return pq_launch_status();
}

extern "C" pq_status pq_rope_rotate(pq_ctx* ctx, const void* x, int64_t T, int32_t H, int32_t D, int64_t ld,
                                    int64_t pos0, double theta, void* y, void* stream) {
  if (!ctx || !x || !y) return PQ_ERR_INVALID_ARG;
  if (T < 0 || H <= 0 || pos0 < 0 || !(theta > 1.0) || ld < static_cast<int64_t>(H) * 128) return PQ_ERR_INVALID_ARG;
  if (D != 128) return PQ_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(y) || ld % 8 != 0) return PQ_ERR_ALIGN;
  if (T == 0) return PQ_OK;
  rope_rotate_kernel<<<grid_for(ctx, T, 1), RP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(y), T, H, ld, pos0, log2(theta));
  return pq_launch_status();
}

extern "C" pq_status pq_rope_kv4_append(pq_ctx* ctx, const pq_kv4_cache* c, int32_t seq, void* qkv, int64_t T, int64_t ld, int64_t pos0,
                                        double theta, int32_t rotate, void* stream) {
  if (!ctx || !c || !qkv || !c->kq || !c->vq || !c->len) return PQ_ERR_INVALID_ARG;
  if (c->sk_tok || c->sv_tok) return PQ_ERR_UNSUPPORTED;  // the static setting only
  if (!c->s_k || !c->s_v) return PQ_ERR_INVALID_ARG;
  if (T < 0 || seq < 0 || seq >= c->B || c->Hkv <= 0 || c->Hq <= 0 || pos0 < 0 || !(theta > 1.0)) return PQ_ERR_INVALID_ARG;
  if (ld < static_cast<int64_t>(c->Hq + 2 * c->Hkv) * 128) return PQ_ERR_INVALID_ARG;
  if (c->D != 128) return PQ_ERR_SHAPE;
  if (!aligned16(qkv) || ld % 8 != 0 || !aligned16(c->kq) || !aligned16(c->vq)) return PQ_ERR_ALIGN;
  if (T == 0) return PQ_OK;
  const int64_t seq_off = static_cast<int64_t>(seq) * c->Hkv * c->Tmax * 64;
  rope_kv4_append_kernel<<<grid_for(ctx, T, 1), RP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<__nv_bfloat16*>(qkv), T, c->Hq, c->Hkv, ld, pos0, log2(theta), rotate, c->kq + seq_off, c->vq + seq_off, c->s_k, c->s_v,
      c->len + seq, c->Tmax, ctx->d_status, ctx->d_tickets + 1);
  return pq_launch_status();
}

extern "C" pq_status pq_silu_mul(pq_ctx* ctx, const void* gate, const void* up, int64_t M, int64_t F, int64_t ld_in,
                                 void* y, int64_t ldy, void* stream) {
  if (!ctx || !gate || !up || !y) return PQ_ERR_INVALID_ARG;
  if (M < 0 || F <= 0 || ld_in < F || ldy < F) return PQ_ERR_INVALID_ARG;
  if (F % 8 != 0 || F > (1 << 30)) return PQ_ERR_SHAPE;
  if (!aligned16(gate) || !aligned16(up) || !aligned16(y) || ld_in % 8 != 0 || ldy % 8 != 0) return PQ_ERR_ALIGN;
  if (M == 0) return PQ_OK;
  silu_mul_kernel<<<grid_for(ctx, M * (F / 8), EW_THREADS), EW_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(gate), static_cast<const __nv_bfloat16*>(up), ld_in,
      static_cast<__nv_bfloat16*>(y), ldy, M, static_cast<int>(F));
  return pq_launch_status();
}

extern "C" pq_status pq_residual_add(pq_ctx* ctx, const void* a, const void* b, void* y, int64_t n, void* stream) {
  if (!ctx || !a || !b || !y || n < 0) return PQ_ERR_INVALID_ARG;
  if (n % 8 != 0) return PQ_ERR_SHAPE;
  if (!aligned16(a) || !aligned16(b) || !aligned16(y)) return PQ_ERR_ALIGN;
  if (n == 0) return PQ_OK;
  add_kernel<<<grid_for(ctx, n / 8, EW_THREADS), EW_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(a), static_cast<const __nv_bfloat16*>(b), static_cast<__nv_bfloat16*>(y), n / 8);
  return pq_launch_status();
}

extern "C" pq_status pq_calib_kv_scale(pq_ctx* ctx, const void* x, int64_t n_tok, int32_t Hkv, int32_t D, int64_t ld_tok,
                                       float* s, void* stream) {
  if (!ctx || !x || !s) return PQ_ERR_INVALID_ARG;
  if (n_tok < 0 || Hkv <= 0 || ld_tok < static_cast<int64_t>(Hkv) * 128) return PQ_ERR_INVALID_ARG;
  if (D != 128) return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) & 7) || ld_tok % 4 != 0) return PQ_ERR_ALIGN;
  if (n_tok == 0) return PQ_OK;
  calib_kv_scale_kernel<<<grid_for(ctx, n_tok * Hkv, EW_THREADS / 32), EW_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(x), n_tok, Hkv, ld_tok, s);
  return pq_launch_status();
}

// ================================================================================= outlier tokens
// Sec. 4.1, Eq. 2: M[i] = max_c |X[i,c]|, R[i] = M[i] / median(M); an upper outlier has R > eta1, a lower one
// 1 / R > eta2. Two launches: a warp per token takes the maximum of the absolute values (the bf16 pattern
// without its sign is monotone: integer maximum), then one CTA sorts the maxima in shared memory (bitonic, on
// the fp32 bit patterns, all non-negative), takes the median (mean of the two middle values) and classifies.
namespace {
constexpr int OT_MAX_TOKENS = 8192;
constexpr int OT_THREADS = 1024;

__global__ void __launch_bounds__(256) token_absmax_kernel(const __nv_bfloat16* x, int64_t ldx, int64_t T, int64_t C, float* M) {
  const int lane = threadIdx.x & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= T) return;
  const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx);
  uint32_t mx = 0;
  for (int64_t i = lane; i < C / 8; i += 32) {
    const uint4 v = __ldg(src + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) mx = max(mx, max(w[e] & 0x7FFFu, (w[e] >> 16) & 0x7FFFu));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) M[row] = __uint_as_float(mx << 16);
}

__global__ void __launch_bounds__(OT_THREADS) outlier_classify_kernel(const float* M, int T, float eta1, float eta2, float* R,
                                                                       int32_t* flags, float* median_out) {
  __shared__ uint32_t key[OT_MAX_TOKENS];
  int n = 1;
  while (n < T) n <<= 1;
  for (int i = threadIdx.x; i < n; i += OT_THREADS) key[i] = i < T ? __float_as_uint(M[i]) : 0xFFFFFFFFu;
  __syncthreads();
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < n; i += OT_THREADS) {
        const int partner = i ^ j;
        if (partner > i) {
          const uint32_t a = key[i], b = key[partner];
          const bool up = (i & k) == 0;
          if ((a > b) == up) key[i] = b, key[partner] = a;
        }
      }
      __syncthreads();
    }
  }
  const float med = __fmul_rn(0.5f, __fadd_rn(__uint_as_float(key[(T - 1) / 2]), __uint_as_float(key[T / 2])));
  if (threadIdx.x == 0) *median_out = med;
  for (int i = threadIdx.x; i < T; i += OT_THREADS) {
    const float m = M[i];
    const float r = __fdiv_rn(m, med), inv = __fdiv_rn(med, m);
    R[i] = r;
    flags[i] = r > eta1 ? 1 : (inv > eta2 ? 2 : 0);
  }
}
}  // namespace

extern "C" pq_status pq_outlier_tokens(pq_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ldx, float eta1, float eta2,
                                       float* M, float* R, int32_t* flags, float* median, void* stream) {
  if (!ctx || !x || !M || !R || !flags || !median) return PQ_ERR_INVALID_ARG;
  if (T <= 0 || C <= 0 || ldx < C || !(eta1 > 0.0f) || !(eta2 > 0.0f)) return PQ_ERR_INVALID_ARG;
  if (T > OT_MAX_TOKENS || C % 8 != 0) return PQ_ERR_SHAPE;
  if (!aligned16(x) || ldx % 8 != 0) return PQ_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  token_absmax_kernel<<<static_cast<unsigned>((T + 7) / 8), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), ldx, T, C, M);
  outlier_classify_kernel<<<1, OT_THREADS, 0, st>>>(M, static_cast<int>(T), eta1, eta2, R, flags, median);
  return pq_launch_status();
}

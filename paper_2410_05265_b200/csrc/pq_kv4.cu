// KV4 quantize-on-write and decode attention over [full-precision prefix || INT4 cache]
// (Sec. 4.2, Eq. 3; Table 1, O2: per-head static KV scales).
#include <math.h>

#include <mutex>

#include "pq_common.cuh"

namespace {

// ================================================================================= append
constexpr int AP_THREADS = 256;

// One thread quantizes 32 consecutive head-dim elements of K and of V (64 B in, 16 B out each).
__global__ void __launch_bounds__(AP_THREADS)
    kv4_append_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, uint8_t* __restrict__ kq,
                      uint8_t* __restrict__ vq, const float* __restrict__ s_k, const float* __restrict__ s_v,
                      int32_t* __restrict__ len, int B, int T_new, int Hkv, int Tmax, int32_t* status,
                      uint32_t* ticket) {
  __shared__ int bad;
  __shared__ int last;
  if (threadIdx.x == 0) bad = 0, last = 0;
  __syncthreads();
  for (int b = threadIdx.x; b < B; b += AP_THREADS)
    if (len[b] < 0 || len[b] + T_new > Tmax) bad = 1;
  __syncthreads();
  if (bad) {  // every CTA reaches the same verdict: nothing is written, len stays
    if (blockIdx.x == 0 && threadIdx.x == 0) pq::report(status, PQ_ERR_SHAPE);
    return;
  }
  const int64_t n_units = static_cast<int64_t>(B) * T_new * Hkv * 4;
  for (int64_t unit = static_cast<int64_t>(blockIdx.x) * AP_THREADS + threadIdx.x; unit < n_units;
       unit += static_cast<int64_t>(gridDim.x) * AP_THREADS) {
    const int part = static_cast<int>(unit & 3);
    const int64_t bth = unit >> 2;
    const int h = static_cast<int>(bth % Hkv);
    const int64_t bt = bth / Hkv;
    const int t = static_cast<int>(bt % T_new), b = static_cast<int>(bt / T_new);
    const int64_t pos = len[b] + t;
    const int64_t src = bth * 128 + part * 32;
    const int64_t dst = ((static_cast<int64_t>(b) * Hkv + h) * Tmax + pos) * 64 + part * 16;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const uint4* in = reinterpret_cast<const uint4*>((which ? v : k) + src);
      const float s = __ldg((which ? s_v : s_k) + h);
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 w = __ldg(in + i);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
        uint32_t acc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float a = __uint_as_float(ww[j] << 16), c = __uint_as_float(ww[j] & 0xFFFF0000u);
          const int ca = max(-8, min(7, __float2int_rn(__fdiv_rn(a, s))));
          const int cc = max(-8, min(7, __float2int_rn(__fdiv_rn(c, s))));
          acc |= static_cast<uint32_t>((ca & 0xF) | ((cc & 0xF) << 4)) << (8 * j);
        }
        o[i] = acc;
      }
      *reinterpret_cast<uint4*>((which ? vq : kq) + dst) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  // the last CTA to finish advances the lengths (every other CTA has read them by then)
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (last) {
    for (int b = threadIdx.x; b < B; b += AP_THREADS) len[b] += T_new;
    if (threadIdx.x == 0) *ticket = 0;
  }
}

// ================================================================================= decode attention
constexpr int DA_WARPS = 4;
constexpr int DA_THREADS = DA_WARPS * 32;
constexpr int DA_MAX_SPLITS = 32;
constexpr int DA_MAX_PREFIX = 64;
constexpr int DA_ROWS = 8;  // query heads per KV head the MMA tile can carry
constexpr int DA_TICKET0 = 16;

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  const uint32_t z = 0;  // rows 8..15 of the A tile are padding
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  const uint32_t z = 0;
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
}
// (a & m) ^ c in one LOP3
__device__ __forceinline__ uint32_t and_xor(uint32_t a, uint32_t m, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(a), "r"(m), "r"(c));  // (a & b) ^ c
  return d;
}
__device__ __forceinline__ uint32_t hsub2_u32(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct AttnParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const __half* prefix_k;
  const __half* prefix_v;
  const uint8_t* kq;
  const uint8_t* vq;
  const float* s_k;
  const float* s_v;
  const int32_t* len;
  float* ws_o;   // [B*Hkv, S, G, 128]
  float* ws_ml;  // [B*Hkv, S, G, 2]
  uint32_t* tickets;
  float sm_scale;
  int B, Hq, Hkv, G, n_prefix, Tmax;
};

// Grid (splits, Hkv, B). A CTA streams its slice of one (sequence, KV head) cache row by row:
// each warp takes 16-key blocks, computes the scores of the G query heads of the group with the
// bf16 MMA (codes turned into bf16 by OR-ing them under an exponent; the resulting +136 offset
// is removed through the row sum of q), runs an online softmax and accumulates P.V with the
// fp16 MMA (codes turned into exact fp16 integers). The last CTA of a (sequence, head) merges the
// splits, adds the full-precision prefix keys/values and writes bf16.
__global__ void __launch_bounds__(DA_THREADS) decode_attn_kernel(const AttnParams p) {
  __shared__ float sm_o[DA_WARPS][DA_ROWS][128];
  __shared__ float sm_ml[DA_WARPS][DA_ROWS][2];
  __shared__ float sm_pre[DA_ROWS][DA_MAX_PREFIX];
  __shared__ int is_last;

  const int split = blockIdx.x, S = gridDim.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = p.G;
  const int bh = b * p.Hkv + h;
  int len_b = p.len[b];
  len_b = len_b < 0 ? 0 : (len_b > p.Tmax ? p.Tmax : len_b);
  const int chunk = (((len_b + S - 1) / S) + 15) & ~15;
  const int t0 = split * chunk;
  const int t1 = min(len_b, t0 + chunk);

  // ---- query fragments: register rho = 4m + k holds q[d], q[d+4] with d = 32t + 8m + k ----------
  const bool row_ok = g < G;
  const __nv_bfloat16* qrow = p.q + (static_cast<int64_t>(b) * p.Hq + h * G + (row_ok ? g : 0)) * 128;
  uint32_t qa[16];
  float qsum = 0.0f;
  {
    const uint4* q4 = reinterpret_cast<const uint4*>(qrow + 32 * t);
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      uint4 w = row_ok ? __ldg(q4 + m) : make_uint4(0, 0, 0, 0);  // 8 bf16: d = 32t + 8m + 0..7
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        // element k is in word k/2, half k%2; element k+4 in word (k+4)/2, same half
        const uint32_t lo = (k & 1) ? (ww[k >> 1] >> 16) : (ww[k >> 1] & 0xFFFFu);
        const uint32_t hi = (k & 1) ? (ww[(k + 4) >> 1] >> 16) : (ww[(k + 4) >> 1] & 0xFFFFu);
        qa[4 * m + k] = lo | (hi << 16);
        qsum += __uint_as_float(lo << 16) + __uint_as_float(hi << 16);
      }
    }
    qsum += __shfl_xor_sync(0xffffffffu, qsum, 1);
    qsum += __shfl_xor_sync(0xffffffffu, qsum, 2);
  }
  const float scale2 = __ldg(p.s_k + h) * p.sm_scale * 1.4426950408889634f;  // scores in log2 units
  const float bias = 136.0f * qsum * scale2;

  const uint8_t* kbase = p.kq + static_cast<int64_t>(bh) * p.Tmax * 64;
  const uint8_t* vbase = p.vq + static_cast<int64_t>(bh) * p.Tmax * 64;

  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f;
  float m_run = -INFINITY, l_run = 0.0f;

  const uint4 z4 = make_uint4(0, 0, 0, 0);
  const uint2 z2 = make_uint2(0, 0);
  uint4 kc[2];
  uint2 vc[4];
  auto load_block = [&](int j0, uint4 (&kk)[2], uint2 (&vv)[4]) {
#pragma unroll
    for (int ti = 0; ti < 2; ++ti) {
      const int key = j0 + 8 * ti + g;
      kk[ti] = key < t1 ? __ldg(reinterpret_cast<const uint4*>(kbase + static_cast<int64_t>(key) * 64 + 16 * t)) : z4;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int key = j0 + 2 * t + (i & 1) + 8 * (i >> 1);
      vv[i] = key < t1 ? __ldg(reinterpret_cast<const uint2*>(vbase + static_cast<int64_t>(key) * 64 + 8 * g)) : z2;
    }
  };

  int j0 = t0 + 16 * warp;
  if (j0 < t1) load_block(j0, kc, vc);
  for (; j0 < t1; j0 += 16 * DA_WARPS) {
    uint4 kn[2];
    uint2 vn[4];
    const int jn = j0 + 16 * DA_WARPS;
    if (jn < t1) load_block(jn, kn, vn);

    // ---- scores of 16 keys -----------------------------------------------------------------
    float s[2][2];
#pragma unroll
    for (int ti = 0; ti < 2; ++ti) {
      const uint32_t ww[4] = {kc[ti].x, kc[ti].y, kc[ti].z, kc[ti].w};
      float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        // registers rho = 2i, 2i+1: word m = rho / 4, shift k = rho % 4
        const uint32_t b0 = and_xor(ww[(2 * i) >> 2] >> (4 * ((2 * i) & 3)), 0x000F000Fu, 0x43084308u);
        const uint32_t b1 = and_xor(ww[(2 * i + 1) >> 2] >> (4 * ((2 * i + 1) & 3)), 0x000F000Fu, 0x43084308u);
        mma_bf16_16816(c, qa[2 * i], qa[2 * i + 1], b0, b1);
      }
      const int key = j0 + 8 * ti + 2 * t;
      s[ti][0] = key < t1 ? c[0] * scale2 - bias : -INFINITY;
      s[ti][1] = key + 1 < t1 ? c[1] * scale2 - bias : -INFINITY;
    }
    float bm = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
    const float m_new = fmaxf(m_run, bm);  // finite: key j0 of this block is valid for every row
    const float alpha = ex2(m_run - m_new);
    const float p00 = ex2(s[0][0] - m_new), p01 = ex2(s[0][1] - m_new);
    const float p10 = ex2(s[1][0] - m_new), p11 = ex2(s[1][1] - m_new);
    const uint32_t pa0 = pack_half2(p00, p01), pa2 = pack_half2(p10, p11);
    {
      // the denominator sums the same fp16-rounded probabilities the MMA multiplies with
      const __half2 h0 = *reinterpret_cast<const __half2*>(&pa0), h1 = *reinterpret_cast<const __half2*>(&pa2);
      const float2 f0 = __half22float2(h0), f1 = __half22float2(h1);
      l_run = l_run * alpha + ((f0.x + f0.y) + (f1.x + f1.y));
    }
    if (__any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
      for (int i = 0; i < 16; ++i) o[i][0] *= alpha, o[i][1] *= alpha;
    }
    m_run = m_new;

    // ---- P.V for the 16 keys -----------------------------------------------------------------
    // vc[0], vc[1]: keys 2t, 2t+1; vc[2], vc[3]: keys 2t+8, 2t+9; 16 nibbles each: d = 16g + 0..15
#pragma unroll
    for (int pair = 0; pair < 2; ++pair) {
      const uint32_t a0w = pair ? vc[0].y : vc[0].x, a1w = pair ? vc[1].y : vc[1].x;
      const uint32_t b0w = pair ? vc[2].y : vc[2].x, b1w = pair ? vc[3].y : vc[3].x;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const uint32_t wa = __byte_perm(a0w, a1w, half ? 0x7632 : 0x5410);
        const uint32_t wb = __byte_perm(b0w, b1w, half ? 0x7632 : 0x5410);
#pragma unroll
        for (int n = 0; n < 4; ++n) {
          const uint32_t f0 = hsub2_u32(and_xor(wa >> (4 * n), 0x000F000Fu, 0x64086408u), 0x64086408u);
          const uint32_t f1 = hsub2_u32(and_xor(wb >> (4 * n), 0x000F000Fu, 0x64086408u), 0x64086408u);
          mma_f16_16816(o[pair * 8 + half * 4 + n], pa0, pa2, f0, f1);
        }
      }
    }
    kc[0] = kn[0], kc[1] = kn[1];
    vc[0] = vn[0], vc[1] = vn[1], vc[2] = vn[2], vc[3] = vn[3];
  }
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);

  // ---- merge the warps of this CTA -----------------------------------------------------------
  if (row_ok) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      sm_o[warp][g][32 * t + i] = o[i][0];       // column 2t   -> d = 16*(2t)   + i
      sm_o[warp][g][32 * t + 16 + i] = o[i][1];  // column 2t+1 -> d = 16*(2t+1) + i
    }
    if (t == 0) sm_ml[warp][g][0] = m_run, sm_ml[warp][g][1] = l_run;
  }
  __syncthreads();
  {
    const int d = threadIdx.x;  // 128 threads <-> 128 head-dim elements
    for (int r = 0; r < G; ++r) {
      float m = -INFINITY;
#pragma unroll
      for (int w = 0; w < DA_WARPS; ++w) m = fmaxf(m, sm_ml[w][r][0]);
      float acc = 0.0f, l = 0.0f;
#pragma unroll
      for (int w = 0; w < DA_WARPS; ++w) {
        const float mw = sm_ml[w][r][0];
        const float e = mw == -INFINITY ? 0.0f : ex2(mw - m);
        acc += sm_o[w][r][d] * e;
        l += sm_ml[w][r][1] * e;
      }
      const int64_t slot = (static_cast<int64_t>(bh) * S + split) * G + r;
      p.ws_o[slot * 128 + d] = acc;
      if (d == 0) p.ws_ml[slot * 2] = m, p.ws_ml[slot * 2 + 1] = l;
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(p.tickets + DA_TICKET0 + bh, 1u) == static_cast<uint32_t>(S - 1));
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  // ---- last CTA of this (sequence, KV head): prefix scores, then the final merge ---------------
  const float l2e = 1.4426950408889634f;
  for (int pair = warp; pair < G * p.n_prefix; pair += DA_WARPS) {
    const int r = pair / p.n_prefix, j = pair % p.n_prefix;
    const __nv_bfloat16* qr = p.q + (static_cast<int64_t>(b) * p.Hq + h * G + r) * 128;
    const __half* kr = p.prefix_k + (static_cast<int64_t>(h) * p.n_prefix + j) * 128;
    float acc = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) acc += __bfloat162float(qr[lane + 32 * i]) * __half2float(kr[lane + 32 * i]);
    for (int o2 = 16; o2 > 0; o2 >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o2);
    if (lane == 0) sm_pre[r][j] = acc * p.sm_scale * l2e;
  }
  __syncthreads();
  {
    const int d = threadIdx.x;
    const float sv = __ldg(p.s_v + h);
    for (int r = 0; r < G; ++r) {
      float m = -INFINITY;
      for (int sp = 0; sp < S; ++sp) m = fmaxf(m, __ldcg(p.ws_ml + ((static_cast<int64_t>(bh) * S + sp) * G + r) * 2));
      for (int j = 0; j < p.n_prefix; ++j) m = fmaxf(m, sm_pre[r][j]);
      float acc = 0.0f, l = 0.0f;
      if (m != -INFINITY) {
        for (int sp = 0; sp < S; ++sp) {
          const int64_t slot = (static_cast<int64_t>(bh) * S + sp) * G + r;
          const float ms = __ldcg(p.ws_ml + slot * 2);
          if (ms == -INFINITY) continue;
          const float e = ex2(ms - m);
          acc += __ldcg(p.ws_o + slot * 128 + d) * e;
          l += __ldcg(p.ws_ml + slot * 2 + 1) * e;
        }
        acc *= sv;
        for (int j = 0; j < p.n_prefix; ++j) {
          const float e = ex2(sm_pre[r][j] - m);
          acc += e * __half2float(p.prefix_v[(static_cast<int64_t>(h) * p.n_prefix + j) * 128 + d]);
          l += e;
        }
      }
      const float res = l > 0.0f ? acc / l : 0.0f;
      p.out[(static_cast<int64_t>(b) * p.Hq + h * G + r) * 128 + d] = __float2bfloat16_rn(res);
    }
  }
  if (threadIdx.x == 0) p.tickets[DA_TICKET0 + bh] = 0;
}

int choose_splits(const pq_ctx* ctx, const pq_kv4_cache* c) {
  const int64_t bh = static_cast<int64_t>(c->B) * c->Hkv;
  int64_t s = (4LL * ctx->sm_count) / (bh > 0 ? bh : 1);
  const int64_t by_len = c->Tmax / 64;
  if (s > by_len) s = by_len;
  if (s > DA_MAX_SPLITS) s = DA_MAX_SPLITS;
  if (s < 1) s = 1;
  return static_cast<int>(s);
}

pq_status check_cache(const pq_kv4_cache* c) {
  if (!c || !c->kq || !c->vq || !c->s_k || !c->s_v || !c->len) return PQ_ERR_INVALID_ARG;
  if (c->B < 0 || c->Hkv <= 0 || c->Hq <= 0 || c->n_prefix < 0 || c->Tmax < 0) return PQ_ERR_INVALID_ARG;
  if (c->n_prefix > 0 && (!c->prefix_k || !c->prefix_v)) return PQ_ERR_INVALID_ARG;
  if (c->D != 128 || c->Hq % c->Hkv != 0 || c->Hq / c->Hkv > DA_ROWS || c->n_prefix > DA_MAX_PREFIX)
    return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(c->kq) & 15) || (reinterpret_cast<uintptr_t>(c->vq) & 15)) return PQ_ERR_ALIGN;
  return PQ_OK;
}

}  // namespace

extern "C" pq_status pq_kv4_append(pq_ctx* ctx, const pq_kv4_cache* cache, const void* k, const void* v,
                                   int32_t T_new, void* stream) {
  if (!ctx || !k || !v || T_new < 0) return PQ_ERR_INVALID_ARG;
  pq_status st = check_cache(cache);
  if (st != PQ_OK) return st;
  if ((reinterpret_cast<uintptr_t>(k) & 15) || (reinterpret_cast<uintptr_t>(v) & 15)) return PQ_ERR_ALIGN;
  if (T_new == 0 || cache->B == 0) return PQ_OK;
  const int64_t n_units = static_cast<int64_t>(cache->B) * T_new * cache->Hkv * 4;
  int64_t grid = (n_units + AP_THREADS - 1) / AP_THREADS;
  if (grid > 8LL * ctx->sm_count) grid = 8LL * ctx->sm_count;
  kv4_append_kernel<<<static_cast<int>(grid), AP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v), cache->kq, cache->vq, cache->s_k,
      cache->s_v, cache->len, cache->B, T_new, cache->Hkv, cache->Tmax, ctx->d_status, ctx->d_tickets);
  return pq_launch_status();
}

extern "C" size_t pq_decode_attn_workspace_bytes(const pq_kv4_cache* cache) {
  if (!cache || cache->B <= 0 || cache->Hkv <= 0 || cache->Hq <= 0) return 0;
  const size_t G = static_cast<size_t>(cache->Hq / cache->Hkv);
  return static_cast<size_t>(cache->B) * cache->Hkv * DA_MAX_SPLITS * G * (128 + 2) * sizeof(float);
}

extern "C" pq_status pq_decode_attn_kv4_prefix(pq_ctx* ctx, const pq_kv4_cache* cache, const void* q, void* out,
                                               float sm_scale, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || !q || !out) return PQ_ERR_INVALID_ARG;
  pq_status st = check_cache(cache);
  if (st != PQ_OK) return st;
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(out) & 1)) return PQ_ERR_ALIGN;
  if (cache->B == 0) return PQ_OK;
  if (static_cast<int64_t>(cache->B) * cache->Hkv > PQ_N_TICKETS - DA_TICKET0 || cache->B > 65535 || cache->Hkv > 65535)
    return PQ_ERR_SHAPE;
  if (!ws || ws_bytes < pq_decode_attn_workspace_bytes(cache)) return PQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 15) return PQ_ERR_ALIGN;
  const int S = choose_splits(ctx, cache);
  const int G = cache->Hq / cache->Hkv;
  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.prefix_k = static_cast<const __half*>(cache->prefix_k);
  p.prefix_v = static_cast<const __half*>(cache->prefix_v);
  p.kq = cache->kq;
  p.vq = cache->vq;
  p.s_k = cache->s_k;
  p.s_v = cache->s_v;
  p.len = cache->len;
  p.ws_o = static_cast<float*>(ws);
  p.ws_ml = p.ws_o + static_cast<size_t>(cache->B) * cache->Hkv * S * G * 128;
  p.tickets = ctx->d_tickets;
  p.sm_scale = sm_scale;
  p.B = cache->B, p.Hq = cache->Hq, p.Hkv = cache->Hkv, p.G = G, p.n_prefix = cache->n_prefix, p.Tmax = cache->Tmax;
  dim3 grid(S, cache->Hkv, cache->B);
  decode_attn_kernel<<<grid, DA_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(p);
  return pq_launch_status();
}

// ================================================================================= no-allocation variant
// Scratch of pq_decode_attn_kv4_prefix_noalloc: split partials followed by the ticket counters.
// It lives in the loaded module, so every GPU that loads this library holds it until exit.
namespace {
constexpr size_t NA_PARTIAL_BYTES = size_t(8) << 20;  // 8 MiB of split partials
constexpr int NA_MAX_BH = 4096;                       // sequences x KV heads
constexpr size_t NA_TICKET_BYTES = (NA_MAX_BH + DA_TICKET0) * sizeof(uint32_t);
}  // namespace
static __device__ __align__(256) unsigned char g_noalloc_scratch[NA_PARTIAL_BYTES + NA_TICKET_BYTES];

namespace {
struct NoAllocDevice {
  bool ready;
  unsigned char* scratch;  // device address of g_noalloc_scratch on this device
  int sm_count;
};
NoAllocDevice g_na_dev[64];
std::mutex g_na_mutex;

int choose_splits_by_sm_count(int sm_count, const pq_kv4_cache* c) {
  const int64_t bh = static_cast<int64_t>(c->B) * c->Hkv;
  int64_t s = (4LL * sm_count) / (bh > 0 ? bh : 1);
  const int64_t by_len = c->Tmax / 64;
  if (s > by_len) s = by_len;
  if (s > DA_MAX_SPLITS) s = DA_MAX_SPLITS;
  if (s < 1) s = 1;
  return static_cast<int>(s);
}
}  // namespace

extern "C" pq_status pq_decode_attn_kv4_prefix_noalloc(const pq_kv4_cache* cache, const void* q, void* out,
                                                       float sm_scale, void* stream) {
  if (!q || !out) return PQ_ERR_INVALID_ARG;
  pq_status st = check_cache(cache);
  if (st != PQ_OK) return st;
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(out) & 1)) return PQ_ERR_ALIGN;
  if (cache->B == 0) return PQ_OK;
  if (cache->B > 65535 || cache->Hkv > 65535) return PQ_ERR_SHAPE;
  const int64_t bh = static_cast<int64_t>(cache->B) * cache->Hkv;
  if (bh > NA_MAX_BH) return PQ_ERR_WORKSPACE;

  // once per device, with that device current: the array's name is only a host-side handle, the
  // kernel needs the device address the runtime resolves for it
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PQ_ERR_CUDA;
  NoAllocDevice nd;
  {
    std::lock_guard<std::mutex> lock(g_na_mutex);
    if (!g_na_dev[dev].ready) {
      void* ptr = nullptr;
      int sms = 0;
      if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return PQ_ERR_CUDA;
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return PQ_ERR_CUDA;
      g_na_dev[dev].scratch = static_cast<unsigned char*>(ptr);
      g_na_dev[dev].sm_count = sms;
      g_na_dev[dev].ready = true;
    }
    nd = g_na_dev[dev];
  }
  const int S = choose_splits_by_sm_count(nd.sm_count, cache);
  const int G = cache->Hq / cache->Hkv;
  const size_t need = static_cast<size_t>(bh) * S * G * (128 + 2) * sizeof(float);
  if (need > NA_PARTIAL_BYTES) return PQ_ERR_WORKSPACE;

  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint32_t* tickets = reinterpret_cast<uint32_t*>(nd.scratch + NA_PARTIAL_BYTES);
  // the array keeps whatever the previous call left: the counters must start at zero
  if (cudaMemsetAsync(tickets + DA_TICKET0, 0, static_cast<size_t>(bh) * sizeof(uint32_t), cs) != cudaSuccess)
    return PQ_ERR_CUDA;
  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.prefix_k = static_cast<const __half*>(cache->prefix_k);
  p.prefix_v = static_cast<const __half*>(cache->prefix_v);
  p.kq = cache->kq;
  p.vq = cache->vq;
  p.s_k = cache->s_k;
  p.s_v = cache->s_v;
  p.len = cache->len;
  p.ws_o = reinterpret_cast<float*>(nd.scratch);
  p.ws_ml = p.ws_o + static_cast<size_t>(bh) * S * G * 128;
  p.tickets = tickets;
  p.sm_scale = sm_scale;
  p.B = cache->B, p.Hq = cache->Hq, p.Hkv = cache->Hkv, p.G = G, p.n_prefix = cache->n_prefix, p.Tmax = cache->Tmax;
  dim3 grid(S, cache->Hkv, cache->B);
  decode_attn_kernel<<<grid, DA_THREADS, 0, cs>>>(p);
  return pq_launch_status();
}

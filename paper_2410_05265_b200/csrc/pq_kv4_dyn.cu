// Group-wise dynamic KV4 (Table 1, O1: the "group-wise dynamic" KV cache of the paper's comparison setting; with a
// group size of 128 and a head dimension of 128 a group is one (token, head) vector): the step of a vector is
// computed when the token is written and stored beside the codes; attention scales every key's score and every
// value row by the key's own step. Plain fp32 kernels: this is the setting the static path is compared with.
#include <math.h>

#include "pq_common.cuh"

namespace {

constexpr int DY_THREADS = 256;
constexpr int DY_WARPS = DY_THREADS / 32;
constexpr int DY_MAX_SPLITS = 32;   // the workspace of pq_decode_attn_workspace_bytes holds this many partials
constexpr int DY_ROWS = 8;          // query heads per KV head
constexpr int DY_MAX_PREFIX = 64;

// ---------------------------------------------------------------------------------------------- append
// Four consecutive threads share one 128-wide vector (32 elements each): maximum over the four, step = max / 7 in
// fp32 (1 for an all-zero vector), fp32 division + round-half-even per element, like the static append.
__global__ void __launch_bounds__(DY_THREADS)
    kv4_append_dyn_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, uint8_t* __restrict__ kq,
                          uint8_t* __restrict__ vq, float* __restrict__ sk_tok, float* __restrict__ sv_tok, int32_t* __restrict__ len,
                          int B, int T_new, int Hkv, int Tmax, int64_t ld_tok, int32_t* status, uint32_t* ticket) {
  __shared__ int bad;
  __shared__ int last;
  if (threadIdx.x == 0) bad = 0, last = 0;
  __syncthreads();
  for (int b = threadIdx.x; b < B; b += DY_THREADS)
    if (len[b] < 0 || len[b] + T_new > Tmax) bad = 1;
  __syncthreads();
  if (bad) {  // every CTA reaches the same verdict: nothing is written, len stays
    if (blockIdx.x == 0 && threadIdx.x == 0) pq::report(status, PQ_ERR_SHAPE);
    return;
  }
  const int64_t n_units = static_cast<int64_t>(B) * T_new * Hkv * 4;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * DY_THREADS;
  for (int64_t base = static_cast<int64_t>(blockIdx.x) * DY_THREADS; base < n_units; base += stride) {  // the same trip count for a warp
    const int64_t unit = base + threadIdx.x;
    const bool ok = unit < n_units;  // whole groups of four: n_units is a multiple of 4
    const int part = static_cast<int>(unit & 3);
    const int64_t bth = ok ? unit >> 2 : 0;
    const int h = static_cast<int>(bth % Hkv);
    const int64_t bt = bth / Hkv;
    const int t = static_cast<int>(bt % T_new), b = static_cast<int>(bt / T_new);
    const int64_t pos = len[b] + t;
    const int64_t src = bt * ld_tok + h * 128 + part * 32;
    const int64_t vec = (static_cast<int64_t>(b) * Hkv + h) * Tmax + pos;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const uint4* in = reinterpret_cast<const uint4*>((which ? v : k) + src);
      uint4 w[4];
      float mx = 0.0f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        w[i] = ok ? __ldg(in + i) : make_uint4(0, 0, 0, 0);
        const uint32_t ww[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) mx = fmaxf(mx, fmaxf(fabsf(__uint_as_float(ww[j] << 16)), fabsf(__uint_as_float(ww[j] & 0xFFFF0000u))));
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float s = mx == 0.0f ? 1.0f : __fdiv_rn(mx, 7.0f);
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t ww[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
        uint32_t acc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int ca = max(-8, min(7, __float2int_rn(__fdiv_rn(__uint_as_float(ww[j] << 16), s))));
          const int cc = max(-8, min(7, __float2int_rn(__fdiv_rn(__uint_as_float(ww[j] & 0xFFFF0000u), s))));
          acc |= static_cast<uint32_t>((ca & 0xF) | ((cc & 0xF) << 4)) << (8 * j);
        }
        o[i] = acc;
      }
      if (ok) {
        *reinterpret_cast<uint4*>((which ? vq : kq) + vec * 64 + part * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        if (part == 0) (which ? sv_tok : sk_tok)[vec] = s;
      }
    }
  }
  if (gridDim.x > 1) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  } else if (threadIdx.x == 0) {
    last = 1;
  }
  __syncthreads();
  if (last) {
    for (int b = threadIdx.x; b < B; b += DY_THREADS) len[b] += T_new;
    if (threadIdx.x == 0 && gridDim.x > 1) *ticket = 0;
  }
}

// ---------------------------------------------------------------------------------------------- decode attention
struct DynAttnParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const __half* prefix_k;
  const __half* prefix_v;
  const uint8_t* kq;
  const uint8_t* vq;
  const float* sk_tok;
  const float* sv_tok;
  const int32_t* len;
  float* ws_o;   // [B*Hkv, S, G, 128]
  float* ws_ml;  // [B*Hkv, S, G, 2]
  uint32_t* tickets;
  float sm_scale;
  int B, Hq, Hkv, G, n_prefix, Tmax;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Grid (splits, Hkv, B), 8 warps. A warp takes chunks of 32 keys: one key per lane for the scores (the lane's 128 codes
// against the G query rows kept in shared memory), an online softmax across the warp, then the value rows staged in
// the warp's shared memory and read with four head dims per lane. Split 0 also scores the full-precision prefix.
// Warps, then splits (workspace + ticket), are merged with the usual (maximum, denominator, weighted sum) rule.
__global__ void __launch_bounds__(DY_THREADS) decode_attn_dyn_kernel(const DynAttnParams p) {
  __shared__ __align__(16) float q_s[DY_ROWS][128];
  __shared__ __align__(16) float o_s[DY_WARPS][DY_ROWS][128];  // a warp's partial output at the end ...
  uint8_t(*v_s)[DY_ROWS * 128 * 4] = reinterpret_cast<uint8_t(*)[DY_ROWS * 128 * 4]>(o_s);  // ... and its 32 staged value rows before
  __shared__ float ml_s[DY_WARPS][DY_ROWS][2];
  __shared__ int is_last;
  const int split = blockIdx.x, S = gridDim.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.G, bh = b * p.Hkv + h;
  for (int i = threadIdx.x; i < G * 128; i += DY_THREADS)
    q_s[i >> 7][i & 127] = __bfloat162float(p.q[(static_cast<int64_t>(b) * p.Hq + h * G + (i >> 7)) * 128 + (i & 127)]);
  __syncthreads();
  int len_b = __ldg(p.len + b);
  len_b = len_b < 0 ? 0 : (len_b > p.Tmax ? p.Tmax : len_b);
  const uint8_t* kbase = p.kq + static_cast<int64_t>(bh) * p.Tmax * 64;
  const uint8_t* vbase = p.vq + static_cast<int64_t>(bh) * p.Tmax * 64;
  const float* skb = p.sk_tok + static_cast<int64_t>(bh) * p.Tmax;
  const float* svb = p.sv_tok + static_cast<int64_t>(bh) * p.Tmax;
  const float l2e_scale = p.sm_scale * 1.4426950408889634f;

  float m[DY_ROWS], l[DY_ROWS], acc[DY_ROWS][4];
#pragma unroll
  for (int g = 0; g < DY_ROWS; ++g) m[g] = -INFINITY, l[g] = 0.0f, acc[g][0] = acc[g][1] = acc[g][2] = acc[g][3] = 0.0f;

  // folds one chunk (scores s[g] of this lane's key in log2 units, -inf when the lane has no key) into the warp's state;
  // value(jj, vv) gives the four head dims 4 lane .. 4 lane + 3 of key jj of the chunk, already in value units
  auto fold = [&](const float (&s)[DY_ROWS], auto value) {
    float pj[DY_ROWS];
#pragma unroll
    for (int g = 0; g < DY_ROWS; ++g) {
      float mx = s[g];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m[g], mx);
      const float alpha = m_new == -INFINITY ? 1.0f : ex2(m[g] - m_new);
      m[g] = m_new;
      l[g] *= alpha;
      acc[g][0] *= alpha, acc[g][1] *= alpha, acc[g][2] *= alpha, acc[g][3] *= alpha;
      pj[g] = m_new == -INFINITY ? 0.0f : ex2(s[g] - m_new);
      l[g] += pj[g];  // this lane's share; the lanes are summed at the end
    }
    for (int jj = 0; jj < 32; ++jj) {
      float vv[4];
      value(jj, vv);
#pragma unroll
      for (int g = 0; g < DY_ROWS; ++g) {
        const float pg = __shfl_sync(0xffffffffu, pj[g], jj);
        acc[g][0] = fmaf(pg, vv[0], acc[g][0]), acc[g][1] = fmaf(pg, vv[1], acc[g][1]);
        acc[g][2] = fmaf(pg, vv[2], acc[g][2]), acc[g][3] = fmaf(pg, vv[3], acc[g][3]);
      }
    }
  };

  // ---- the full-precision prefix: split 0, warp 0, one prefix key per lane
  if (split == 0 && warp == 0) {
    for (int j0 = 0; j0 < p.n_prefix; j0 += 32) {
      const int j = j0 + lane;
      float s[DY_ROWS];
#pragma unroll
      for (int g = 0; g < DY_ROWS; ++g) s[g] = 0.0f;
      if (j < p.n_prefix) {
        const uint4* kr = reinterpret_cast<const uint4*>(p.prefix_k + (static_cast<int64_t>(h) * p.n_prefix + j) * 128);
        for (int c = 0; c < 16; ++c) {
          const uint4 kv = __ldg(kr + c);
          const uint32_t kw[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 kf = __half22float2(*reinterpret_cast<const __half2*>(&kw[e]));
#pragma unroll
            for (int g = 0; g < DY_ROWS; ++g)
              if (g < G) s[g] = fmaf(q_s[g][8 * c + 2 * e], kf.x, fmaf(q_s[g][8 * c + 2 * e + 1], kf.y, s[g]));
          }
        }
      }
#pragma unroll
      for (int g = 0; g < DY_ROWS; ++g) s[g] = (j < p.n_prefix && g < G) ? s[g] * l2e_scale : -INFINITY;
      fold(s, [&](int jj, float (&vv)[4]) {
        vv[0] = vv[1] = vv[2] = vv[3] = 0.0f;
        if (j0 + jj < p.n_prefix) {
          const uint2 w = __ldg(reinterpret_cast<const uint2*>(p.prefix_v + (static_cast<int64_t>(h) * p.n_prefix + j0 + jj) * 128) + lane);
          const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x)), c2 = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
          vv[0] = a.x, vv[1] = a.y, vv[2] = c2.x, vv[3] = c2.y;
        }
      });
    }
  }

  // ---- the INT4 region: chunk c of 32 keys belongs to split c % S, warp (c / S) % 8
  const int n_chunks = (len_b + 31) / 32;
  for (int c = split + S * warp; c < n_chunks; c += S * DY_WARPS) {
    const int j = c * 32 + lane;
    const bool have = j < len_b;
    float s[DY_ROWS];
#pragma unroll
    for (int g = 0; g < DY_ROWS; ++g) s[g] = 0.0f;
    const uint4* kr = reinterpret_cast<const uint4*>(kbase + static_cast<int64_t>(have ? j : 0) * 64);
    const uint4* vr = reinterpret_cast<const uint4*>(vbase + static_cast<int64_t>(have ? j : 0) * 64);
    uint4* vdst = reinterpret_cast<uint4*>(v_s[warp] + lane * 64);
#pragma unroll
    for (int i = 0; i < 4; ++i) vdst[i] = have ? __ldg(vr + i) : make_uint4(0, 0, 0, 0);
    for (int i = 0; i < 4; ++i) {
      const uint4 kv = have ? __ldg(kr + i) : make_uint4(0, 0, 0, 0);
      const uint32_t kw[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float code[8];
#pragma unroll
        for (int n = 0; n < 8; ++n) code[n] = static_cast<float>(static_cast<int>(((kw[e] >> (4 * n)) & 0xF) ^ 8) - 8);
#pragma unroll
        for (int g = 0; g < DY_ROWS; ++g) {
          if (g < G) {  // the query row's eight dims in two 16-byte reads (every lane the same address)
            const float4 qa = *reinterpret_cast<const float4*>(&q_s[g][32 * i + 8 * e]), qb = *reinterpret_cast<const float4*>(&q_s[g][32 * i + 8 * e + 4]);
            s[g] = fmaf(qa.x, code[0], fmaf(qa.y, code[1], fmaf(qa.z, code[2], fmaf(qa.w, code[3], s[g]))));
            s[g] = fmaf(qb.x, code[4], fmaf(qb.y, code[5], fmaf(qb.z, code[6], fmaf(qb.w, code[7], s[g]))));
          }
        }
      }
    }
    const float f = have ? __ldg(skb + j) * l2e_scale : 0.0f;
    const float sv_mine = have ? __ldg(svb + j) : 0.0f;
#pragma unroll
    for (int g = 0; g < DY_ROWS; ++g) s[g] = (have && g < G) ? s[g] * f : -INFINITY;
    __syncwarp();  // the warp's value rows are in place
    fold(s, [&](int jj, float (&vv)[4]) {
      const float svj = __shfl_sync(0xffffffffu, sv_mine, jj);
      const uint32_t w = *reinterpret_cast<const uint16_t*>(v_s[warp] + jj * 64 + 2 * lane);
#pragma unroll
      for (int n = 0; n < 4; ++n) vv[n] = static_cast<float>(static_cast<int>(((w >> (4 * n)) & 0xF) ^ 8) - 8) * svj;
    });
    __syncwarp();  // before the next chunk overwrites the staging rows
  }

  // ---- merge: lanes -> warp (denominators), warps -> CTA, CTA -> workspace, last CTA of the (sequence, head) -> output
#pragma unroll
  for (int g = 0; g < DY_ROWS; ++g) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l[g] += __shfl_xor_sync(0xffffffffu, l[g], o);
    if (g < G) {
      *reinterpret_cast<float4*>(&o_s[warp][g][4 * lane]) = make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
      if (lane == 0) ml_s[warp][g][0] = m[g], ml_s[warp][g][1] = l[g];
    }
  }
  __syncthreads();
  for (int item = threadIdx.x; item < G * 128; item += DY_THREADS) {
    const int g = item >> 7, d = item & 127;
    float mm = -INFINITY;
    for (int w = 0; w < DY_WARPS; ++w) mm = fmaxf(mm, ml_s[w][g][0]);
    float o = 0.0f, ll = 0.0f;
    for (int w = 0; w < DY_WARPS; ++w) {
      const float e = ml_s[w][g][0] == -INFINITY ? 0.0f : ex2(ml_s[w][g][0] - mm);
      o = fmaf(o_s[w][g][d], e, o);
      ll = fmaf(ml_s[w][g][1], e, ll);
    }
    const int64_t slot = (static_cast<int64_t>(bh) * S + split) * G + g;
    p.ws_o[slot * 128 + d] = o;
    if (d == 0) p.ws_ml[slot * 2] = mm, p.ws_ml[slot * 2 + 1] = ll;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = atomicAdd(p.tickets + bh, 1u) == static_cast<uint32_t>(S - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int item = threadIdx.x; item < G * 128; item += DY_THREADS) {
    const int g = item >> 7, d = item & 127;
    const int64_t slot0 = static_cast<int64_t>(bh) * S * G + g;
    float mm = -INFINITY;
    for (int sp = 0; sp < S; ++sp) mm = fmaxf(mm, __ldcg(p.ws_ml + (slot0 + static_cast<int64_t>(sp) * G) * 2));
    float o = 0.0f, ll = 0.0f;
    for (int sp = 0; sp < S; ++sp) {
      const int64_t slot = slot0 + static_cast<int64_t>(sp) * G;
      const float ms = __ldcg(p.ws_ml + slot * 2);
      const float e = ms == -INFINITY ? 0.0f : ex2(ms - mm);
      o = fmaf(__ldcg(p.ws_o + slot * 128 + d), e, o);
      ll = fmaf(__ldcg(p.ws_ml + slot * 2 + 1), e, ll);
    }
    p.out[(static_cast<int64_t>(b) * p.Hq + h * G + g) * 128 + d] = __float2bfloat16_rn(ll > 0.0f ? o / ll : 0.0f);
  }
  if (threadIdx.x == 0) p.tickets[bh] = 0;
}

}  // namespace

pq_status pq_kv4_append_dyn_launch(pq_ctx* ctx, const pq_kv4_cache* c, const void* k, const void* v, int32_t T_new, int64_t ld_tok,
                                   cudaStream_t st) {
  const int64_t n_units = static_cast<int64_t>(c->B) * T_new * c->Hkv * 4;
  int64_t grid = (n_units + DY_THREADS - 1) / DY_THREADS;
  if (grid > 8LL * ctx->sm_count) grid = 8LL * ctx->sm_count;
  kv4_append_dyn_kernel<<<static_cast<int>(grid), DY_THREADS, 0, st>>>(
      static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v), c->kq, c->vq, c->sk_tok, c->sv_tok, c->len, c->B, T_new,
      c->Hkv, c->Tmax, ld_tok, ctx->d_status, ctx->d_tickets);
  return pq_launch_status();
}

pq_status pq_decode_attn_dyn_launch(pq_ctx* ctx, const pq_kv4_cache* c, const void* q, void* out, float sm_scale, void* ws,
                                    cudaStream_t st, int ticket0) {
  const int64_t bh = static_cast<int64_t>(c->B) * c->Hkv;
  int64_t S = (4LL * ctx->sm_count) / (bh > 0 ? bh : 1);
  const int64_t by_len = c->Tmax / 256;  // a split's eight warps want a chunk of 32 keys each
  if (S > by_len) S = by_len;
  if (S > DY_MAX_SPLITS) S = DY_MAX_SPLITS;
  if (S < 1) S = 1;
  const int G = c->Hq / c->Hkv;
  DynAttnParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.prefix_k = static_cast<const __half*>(c->prefix_k);
  p.prefix_v = static_cast<const __half*>(c->prefix_v);
  p.kq = c->kq, p.vq = c->vq, p.sk_tok = c->sk_tok, p.sv_tok = c->sv_tok, p.len = c->len;
  p.ws_o = static_cast<float*>(ws);
  p.ws_ml = p.ws_o + static_cast<size_t>(bh) * S * G * 128;
  p.tickets = ctx->d_tickets + ticket0;
  p.sm_scale = sm_scale;
  p.B = c->B, p.Hq = c->Hq, p.Hkv = c->Hkv, p.G = G, p.n_prefix = c->n_prefix, p.Tmax = c->Tmax;
  decode_attn_dyn_kernel<<<dim3(static_cast<unsigned>(S), c->Hkv, c->B), DY_THREADS, 0, st>>>(p);
  return pq_launch_status();
}

// Causal prefill attention over [full-precision prefix || INT4 cache] (Sec. 4.2, Eq. 3): query t of a
// sequence sees every prefixed key and the cached keys 0..t of the same sequence.
//
// Grid (query tiles, KV heads, head groups). A CTA owns 16 consecutive query tokens of up to four of
// the query heads that share one KV head (four warps: two such CTAs fit an SM, which hides the
// softmax phases of one behind the MMAs of the other); warp g holds one head's 16 x 128 query tile as
// fp16 MMA fragments. Keys are
// walked in blocks of 64: the packed rows are fetched one block ahead into registers, expanded to
// exact fp16 integers (the per-head steps s_k, s_v are folded into the score scale and the final
// normalisation) and stored as swizzled [key][dim] tiles that ldmatrix turns into MMA operands.
// Scores and P.V use m16n8k16 fp16 MMAs with fp32 accumulation and the usual online softmax in
// log2 units; P is rounded to fp16 and the denominator sums the same rounded values. The prefix
// block comes first: its keys are used as stored (fp16), its scores take sm_scale alone and its
// probabilities are divided by s_v before the product so that one accumulator serves both regions.
#include <math.h>

#include "pq_common.cuh"

namespace {

constexpr int PA_TOK = 16;    // query tokens per CTA
constexpr int PA_KEYS = 64;   // keys per block
constexpr int PA_TILE_BYTES = PA_KEYS * 128 * 2;  // one fp16 [64][128] tile

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// Two codes of one packed byte (bits 0..7 of `b`, the rest ignored) as an exact fp16 pair (lo, hi).
// 0x6400 | (n ^ 8) is 1032 + code for the low nibble; the high nibble stays four bits up and reads
// 1152 + 16 * code; one fused multiply-add removes both offsets and the factor 16.
__device__ __forceinline__ uint32_t byte_to_h2(uint32_t b) {
  const uint32_t spread = __byte_perm(b, 0, 0x4040);  // byte 0 of b in bits 0..7 and 16..23
  uint32_t v;
  asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(v) : "r"(spread), "r"(0x00F0000Fu), "r"(0x64806408u));
  const __half2 scale = __halves2half2(__float2half_rn(1.0f), __float2half_rn(0.0625f));
  const __half2 off = __halves2half2(__float2half_rn(-1032.0f), __float2half_rn(-72.0f));
  const __half2 r = __hfma2(*reinterpret_cast<const __half2*>(&v), scale, off);
  return *reinterpret_cast<const uint32_t*>(&r);
}
// Byte address of 16-byte chunk `c` (0..15) of row `r` in a swizzled [rows][128] fp16 tile.
__device__ __forceinline__ uint32_t tile_off(int r, int c) { return static_cast<uint32_t>(r * 256 + ((c ^ (r & 7)) << 4)); }

struct PrefillParams {
  const __nv_bfloat16* q;   // [T, Hq, 128] with ldq elements between tokens
  int64_t ldq;
  __nv_bfloat16* out;       // [T, Hq, 128]
  const __half* prefix_k;   // [Hkv, n_prefix, 128]
  const __half* prefix_v;
  const uint8_t* kq;        // this sequence: [Hkv, Tmax, 64]
  const uint8_t* vq;
  const float* s_k;
  const float* s_v;
  float sm_scale;
  int T, Hq, Hkv, G, n_prefix, Tmax;
};

// One thread's share of a block of packed rows: 16 bytes of K and 16 bytes of V when the CTA has 256
// threads (G = 8); CTAs with fewer warps take several shares.
struct PackedShare {
  uint4 k, v;
};

template <int G>
__device__ __forceinline__ void fetch_block(const PrefillParams& p, int h, int key0, int n_keys, PackedShare (&sh)[8 / G]) {
  // share s of thread x covers key (x + s * 32G) / 4, bytes 16 * ((x + s * 32G) % 4) .. +15
#pragma unroll
  for (int s = 0; s < 8 / G; ++s) {
    const int unit = threadIdx.x + s * 32 * G, key = unit >> 2, part = unit & 3;
    if (key < n_keys) {
      const int64_t off = (static_cast<int64_t>(h) * p.Tmax + key0 + key) * 64 + part * 16;
      sh[s].k = __ldg(reinterpret_cast<const uint4*>(p.kq + off));
      sh[s].v = __ldg(reinterpret_cast<const uint4*>(p.vq + off));
    } else {
      sh[s].k = sh[s].v = make_uint4(0x88888888u, 0x88888888u, 0x88888888u, 0x88888888u);  // any finite codes
    }
  }
}

template <int G>
__device__ __forceinline__ void store_block(uint8_t* k_tile, uint8_t* v_tile, const PackedShare (&sh)[8 / G]) {
#pragma unroll
  for (int s = 0; s < 8 / G; ++s) {
    const int unit = threadIdx.x + s * 32 * G, key = unit >> 2, part = unit & 3;  // 32 dims: chunks 4*part .. 4*part+3
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const uint4 pk = which ? sh[s].v : sh[s].k;
      const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
      uint8_t* tile = which ? v_tile : k_tile;
#pragma unroll
      for (int i = 0; i < 4; ++i) {  // word i: dims 32*part + 8i .. +7 = one 16-byte fp16 chunk
        uint4 o;
        o.x = byte_to_h2(w[i]), o.y = byte_to_h2(w[i] >> 8), o.z = byte_to_h2(w[i] >> 16), o.w = byte_to_h2(w[i] >> 24);
        *reinterpret_cast<uint4*>(tile + tile_off(key, 4 * part + i)) = o;
      }
    }
  }
}

template <int G>
__global__ void __launch_bounds__(32 * G) prefill_attn_kernel(const PrefillParams p) {
  extern __shared__ __align__(1024) uint8_t pa_smem[];  // [2 buffers][K tile | V tile]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int h = blockIdx.y;
  const int tile = gridDim.x - 1 - blockIdx.x;  // long tiles first
  const int tok0 = tile * PA_TOK;
  const int head = h * p.G + blockIdx.z * G + warp;  // G = heads of this CTA, p.G = heads per KV head
  const int n_ctx = min(p.T, tok0 + PA_TOK);     // cached keys any row of this tile may see
  const int n_blocks = (n_ctx + PA_KEYS - 1) / PA_KEYS;
  const bool has_prefix = p.n_prefix > 0;

  // ---- query fragments: rows = tokens tok0 + g and tok0 + g + 8, fp16 ------------------------------
  uint32_t qa[8][4];
  {
    const int r0 = min(tok0 + g, p.T - 1), r1 = min(tok0 + g + 8, p.T - 1);
    const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + static_cast<int64_t>(r0) * p.ldq + head * 128);
    const uint32_t* q1 = reinterpret_cast<const uint32_t*>(p.q + static_cast<int64_t>(r1) * p.ldq + head * 128);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint32_t w[4] = {__ldg(q0 + ks * 8 + t), __ldg(q1 + ks * 8 + t), __ldg(q0 + ks * 8 + 4 + t), __ldg(q1 + ks * 8 + 4 + t)};
#pragma unroll
      for (int i = 0; i < 4; ++i) qa[ks][i] = pack_h2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
    }
  }
  const float l2e = 1.4426950408889634f;
  const float sk = __ldg(p.s_k + h), sv = __ldg(p.s_v + h);
  const float scale_ctx = sk * p.sm_scale * l2e, scale_pre = p.sm_scale * l2e, inv_sv = 1.0f / sv;

  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};  // rows g and g + 8

  const uint32_t smem_base = pq::smem_u32(pa_smem);
  PackedShare sh[8 / G];
  int buf = 0;

  // block -1 is the prefix (fp16 as stored), blocks 0 .. n_blocks-1 the cached keys
  const int first = has_prefix ? -1 : 0;
  if (first == 0 && n_blocks > 0) fetch_block<G>(p, h, 0, min(PA_KEYS, n_ctx), sh);
  for (int blk = first; blk < n_blocks; ++blk) {
    uint8_t* k_tile = pa_smem + buf * 2 * PA_TILE_BYTES;
    uint8_t* v_tile = k_tile + PA_TILE_BYTES;
    if (blk < 0) {
      // prefix rows copied as they are; rows past n_prefix are zero and masked below
      for (int unit = threadIdx.x; unit < PA_KEYS * 16; unit += 32 * G) {
        const int key = unit >> 4, c = unit & 15;
        uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
        if (key < p.n_prefix) {
          const int64_t off = (static_cast<int64_t>(h) * p.n_prefix + key) * 128 + c * 8;
          kv4 = __ldg(reinterpret_cast<const uint4*>(p.prefix_k + off));
          vv4 = __ldg(reinterpret_cast<const uint4*>(p.prefix_v + off));
        }
        *reinterpret_cast<uint4*>(k_tile + tile_off(key, c)) = kv4;
        *reinterpret_cast<uint4*>(v_tile + tile_off(key, c)) = vv4;
      }
    } else {
      store_block<G>(k_tile, v_tile, sh);
    }
    __syncthreads();
    // fetch the next block's packed rows while this one is multiplied
    if (blk + 1 < n_blocks) fetch_block<G>(p, h, (blk + 1) * PA_KEYS, min(PA_KEYS, n_ctx - (blk + 1) * PA_KEYS), sh);

    const int key0 = blk < 0 ? 0 : blk * PA_KEYS;
    const int n_valid = blk < 0 ? p.n_prefix : min(PA_KEYS, n_ctx - key0);
    const float scale = blk < 0 ? scale_pre : scale_ctx;
    const uint32_t k_addr = smem_base + buf * 2 * PA_TILE_BYTES, v_addr = k_addr + PA_TILE_BYTES;

    // ---- S = Q K^T: 8 key tiles of 8 x 8 dim steps of 16 ------------------------------------------
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.0f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {  // key tiles 2jp, 2jp+1
        // matrices: (tile 2jp, dims 0-7), (2jp, dims 8-15), (2jp+1, 0-7), (2jp+1, 8-15) of this dim step
        const int row = (2 * jp + (lane >> 4)) * 8 + (lane & 7), chunk = 2 * ks + ((lane >> 3) & 1);
        uint32_t b[4];
        ldsm_x4(k_addr + tile_off(row, chunk), b);
        mma_16816(s[2 * jp], qa[ks], b[0], b[1]);
        mma_16816(s[2 * jp + 1], qa[ks], b[2], b[3]);
      }
    }
    // ---- scale, mask, online softmax -------------------------------------------------------------
    const int tok_a = tok0 + g, tok_b = tok0 + g + 8;  // rows of this lane
    const bool need_mask = blk < 0 ? (n_valid < PA_KEYS) : (key0 + PA_KEYS > tok0 + 1 || n_valid < PA_KEYS);
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[j][e];  // raw: the (positive) score scale is applied with the subtraction of the maximum below
        if (need_mask) {
          const int key = 8 * j + 2 * t + (e & 1);  // within the block
          const int tok = (e & 2) ? tok_b : tok_a;
          const bool ok = blk < 0 ? key < n_valid : (key0 + key <= tok && key < n_valid);
          if (!ok) v = -INFINITY;
        }
        s[j][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float alpha[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r] * scale);
      alpha[r] = m_new == -INFINITY ? 1.0f : ex2f(m_run[r] - m_new);
      m_run[r] = m_new;
      l_run[r] *= alpha[r];
    }
    // after the first blocks the running maximum seldom moves: the rescaling is skipped when no row of the warp needs it
    if (__any_sync(0xffffffffu, alpha[0] != 1.0f || alpha[1] != 1.0f)) {
#pragma unroll
      for (int i = 0; i < 16; ++i) o[i][0] *= alpha[0], o[i][1] *= alpha[0], o[i][2] *= alpha[1], o[i][3] *= alpha[1];
    }
    const float pscale = blk < 0 ? inv_sv : 1.0f;  // prefix values are real values, the accumulator is in code units
    uint32_t pa[4][4];  // A fragments of P for the four 16-key steps
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float ma = m_run[0] == -INFINITY ? 0.0f : m_run[0], mb = m_run[1] == -INFINITY ? 0.0f : m_run[1];
      const float p0 = ex2f(fmaf(s[j][0], scale, -ma)), p1 = ex2f(fmaf(s[j][1], scale, -ma));
      const float p2 = ex2f(fmaf(s[j][2], scale, -mb)), p3 = ex2f(fmaf(s[j][3], scale, -mb));
      const uint32_t lo = pack_h2(p0 * pscale, p1 * pscale), hi = pack_h2(p2 * pscale, p3 * pscale);
      // the denominator sums what the MMA multiplies with (rounded to fp16), in probability units
      const float2 fl = __half22float2(*reinterpret_cast<const __half2*>(&lo)), fh = __half22float2(*reinterpret_cast<const __half2*>(&hi));
      const float back = blk < 0 ? sv : 1.0f;
      l_run[0] += (fl.x + fl.y) * back;
      l_run[1] += (fh.x + fh.y) * back;
      pa[j >> 1][(j & 1) * 2] = lo;      // a0 / a2: row g
      pa[j >> 1][(j & 1) * 2 + 1] = hi;  // a1 / a3: row g + 8
    }
    // ---- O += P V: 4 key steps of 16 x 16 dim tiles of 8 --------------------------------------------
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {  // dim tiles 2dp, 2dp+1
        // transposed loads: (keys 0-7, dims tile 2dp), (keys 8-15, 2dp), (keys 0-7, 2dp+1), (keys 8-15, 2dp+1)
        const int row = kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), chunk = 2 * dp + (lane >> 4);
        uint32_t b[4];
        ldsm_x4_trans(v_addr + tile_off(row, chunk), b);
        mma_16816(o[2 * dp], pa[kk], b[0], b[1]);
        mma_16816(o[2 * dp + 1], pa[kk], b[2], b[3]);
      }
    }
    buf ^= 1;
  }

  // ---- normalise and store -------------------------------------------------------------------------
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
  const float na = l_run[0] > 0.0f ? sv / l_run[0] : 0.0f, nb = l_run[1] > 0.0f ? sv / l_run[1] : 0.0f;
  const int tok_a = tok0 + g, tok_b = tok0 + g + 8;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int d = 8 * i + 2 * t;
    if (tok_a < p.T) {
      const __nv_bfloat162 v = __floats2bfloat162_rn(o[i][0] * na, o[i][1] * na);
      *reinterpret_cast<__nv_bfloat162*>(p.out + (static_cast<int64_t>(tok_a) * p.Hq + head) * 128 + d) = v;
    }
    if (tok_b < p.T) {
      const __nv_bfloat162 v = __floats2bfloat162_rn(o[i][2] * nb, o[i][3] * nb);
      *reinterpret_cast<__nv_bfloat162*>(p.out + (static_cast<int64_t>(tok_b) * p.Hq + head) * 128 + d) = v;
    }
  }
}

template <int G>
pq_status launch_prefill(const PrefillParams& p, cudaStream_t st) {
  constexpr int smem = 4 * PA_TILE_BYTES;
  static bool attr_set[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PQ_ERR_CUDA;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(prefill_attn_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return PQ_ERR_CUDA;
    attr_set[dev] = true;
  }
  dim3 grid((p.T + PA_TOK - 1) / PA_TOK, p.Hkv, p.G / G);
  prefill_attn_kernel<G><<<grid, 32 * G, smem, st>>>(p);
  return pq_launch_status();
}

}  // namespace

extern "C" pq_status pq_prefill_attn_kv4_prefix(pq_ctx* ctx, const pq_kv4_cache* c, int32_t seq, const void* q, int64_t ldq,
                                                int32_t T, void* out, float sm_scale, void* stream) {
  if (!ctx || !c || !q || !out || !c->kq || !c->vq || !c->s_k || !c->s_v) return PQ_ERR_INVALID_ARG;
  if (ldq < static_cast<int64_t>(c->Hq) * 128 || (ldq & 1)) return PQ_ERR_INVALID_ARG;
  if (T < 0 || seq < 0 || seq >= c->B || c->Hkv <= 0 || c->Hq <= 0 || c->n_prefix < 0) return PQ_ERR_INVALID_ARG;
  if (c->n_prefix > 0 && (!c->prefix_k || !c->prefix_v)) return PQ_ERR_INVALID_ARG;
  if (c->D != 128 || c->Hq % c->Hkv != 0 || T > c->Tmax || c->n_prefix > PA_KEYS || c->Hkv > 65535) return PQ_ERR_SHAPE;
  const int G = c->Hq / c->Hkv;
  if (G != 1 && G != 2 && G != 4 && G != 8) return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(c->kq) & 15) || (reinterpret_cast<uintptr_t>(c->vq) & 15) ||
      (reinterpret_cast<uintptr_t>(q) & 3) || (reinterpret_cast<uintptr_t>(out) & 3) ||
      (c->n_prefix > 0 && ((reinterpret_cast<uintptr_t>(c->prefix_k) & 15) || (reinterpret_cast<uintptr_t>(c->prefix_v) & 15))))
    return PQ_ERR_ALIGN;
  if (T == 0) return PQ_OK;
  PrefillParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.ldq = ldq;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.prefix_k = static_cast<const __half*>(c->prefix_k);
  p.prefix_v = static_cast<const __half*>(c->prefix_v);
  const int64_t seq_off = static_cast<int64_t>(seq) * c->Hkv * c->Tmax * 64;
  p.kq = c->kq + seq_off;
  p.vq = c->vq + seq_off;
  p.s_k = c->s_k;
  p.s_v = c->s_v;
  p.sm_scale = sm_scale;
  p.T = T, p.Hq = c->Hq, p.Hkv = c->Hkv, p.G = G, p.n_prefix = c->n_prefix, p.Tmax = c->Tmax;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  switch (G) {
    case 1: return launch_prefill<1>(p, st);
    case 2: return launch_prefill<2>(p, st);
    case 4: return launch_prefill<4>(p, st);
    default: return launch_prefill<4>(p, st);  // eight heads per KV head: two CTAs of four warps, two CTAs per SM
  }
}

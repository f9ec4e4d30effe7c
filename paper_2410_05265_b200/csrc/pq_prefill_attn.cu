// Causal prefill attention over [full-precision prefix || INT4 cache] (Sec. 4.2, Eq. 3): query t of a
// sequence sees every prefixed key and the cached keys 0..t of the same sequence.
//
// Both products run on the 5th-generation tensor cores (tcgen05.mma kind::f16, fp16 operands, fp32
// accumulators in tensor memory). A CTA owns one KV head and 256 query rows = 256/G consecutive tokens x the
// G query heads that share the KV head, as two 128-row tiles, so a key tile is expanded once for all of them.
// Keys are walked in tiles of 128 (the prefix, up to 64 full-precision keys, is a first tile of its own):
//   loader warp      1-D bulk copies of the packed K and V rows of a key tile (8 KB each) into a landing ring.
//   expansion warps  codes -> exact fp16 integers (the per-head steps s_k, s_v are folded into the score scale and
//                    the final normalisation), written as [key][dim] tiles in the 128-byte-swizzled layout that
//                    serves as the K-major B operand of S = Q K^T and as the MN-major B operand of O = P V.
//   MMA warp         S_i = Q_i K^T into tensor memory; once the softmax warps have put P_i back (fp16, over the
//                    columns of S_i) O_i += P_i V with P as the tensor-memory A operand; S of the next key tile
//                    is issued right behind, so one tile's softmax runs under the other tile's MMAs.
//   softmax warps    one thread per query row (tcgen05.ld 32x32b): running maximum in log2 units that is moved only
//                    when a score exceeds it by more than 8 (then O_i is rescaled in tensor memory), P = 2^(s - m)
//                    rounded to fp16, denominator in fp32; at the end O_i / l * s_v -> bf16.
// Inside every group of eight head dims the expansion leaves the order 0,4,1,5,2,6,3,7 (two codes per
// instruction); Q and the prefix rows are stored in the same order (the contraction does not care) and the
// output columns are put back when they are written. Every wait is bounded.
#include <math.h>

#include "pq_common.cuh"

namespace {

constexpr int PA_ROWS = 128;          // query rows per tile (MMA M)
constexpr int PA_KEYS = 128;          // keys per tile
constexpr int PA_MAX_PREFIX = 64;     // the prefix tile has 64 key rows
constexpr int PA_HALF = 128 * 128;    // bytes of one half tile: 128 rows x 64 fp16 (128 bytes, swizzled)
constexpr int PA_TILE = 2 * PA_HALF;  // a [128][128] fp16 tile: dims 0..63, then dims 64..127
constexpr int PA_LAND = 2 * PA_KEYS * 64;  // packed K rows, then packed V rows of one key tile
constexpr int PA_STAGES = 2;
constexpr int PA_SOFTMAX_WARPS = 8, PA_EXPAND_WARPS = 4;
constexpr int PA_WARP_EXPAND0 = PA_SOFTMAX_WARPS, PA_WARP_MMA = PA_WARP_EXPAND0 + PA_EXPAND_WARPS, PA_WARP_LOAD = PA_WARP_MMA + 1;
constexpr int PA_THREADS = (PA_WARP_LOAD + 1) * 32;  // 448
constexpr int PA_TMEM_COLS = 512;     // S0 | S1 | O0 | O1, 128 columns each; P_i lies over the first 64 columns of S_i
constexpr float PA_LAZY = 8.0f;       // log2 units a score may exceed the running reference before it is moved

struct PaBarriers {
  uint64_t land_full[PA_STAGES], land_empty[PA_STAGES];
  uint64_t kv_full[PA_STAGES], kv_empty[PA_STAGES];
  uint64_t s_full[2], p_full[2], o_final[2];
  uint64_t q_ready, drain;
  uint32_t tmem_base;
  volatile int abort_flag;
};

constexpr size_t PA_SMEM_BYTES = 1024 /*alignment slack*/ + 2 * PA_TILE /*Q*/ + PA_STAGES * 2 * PA_TILE /*K, V*/ +
                                 PA_STAGES * PA_LAND + sizeof(PaBarriers);
static_assert(PA_SMEM_BYTES <= 227 * 1024, "shared memory budget");

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
  const float* sk_tok;      // group-wise dynamic setting: this sequence's per-key steps [Hkv, Tmax]
  const float* sv_tok;
  int32_t* status;
  long long wait_clocks;
  float sm_scale;
  int T, Hq, Hkv, G, n_prefix, Tmax;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3f(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
template <uint32_t M, uint32_t C>
__device__ __forceinline__ uint32_t and_xor(uint32_t a) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(a), "n"(M), "n"(C));  // (a & b) ^ c
  return d;
}
__device__ __forceinline__ uint32_t hfma2_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// Eight codes of one packed word (nibble i = head dim i of the group) as exact fp16 integers in the order
// (0,4) (1,5) (2,6) (3,7): nibbles 0 and 4 under the exponent of 1024 read 1032 + code, nibbles 1 and 5 stay four
// bits up and read 1152 + 16 * code; one fused multiply-add each removes the offset (and the factor 16).
__device__ __forceinline__ uint4 expand8(uint32_t w) {
  const uint32_t w8 = w >> 8;
  const uint32_t ONE = 0x3C003C00u, SIXTEENTH = 0x2C002C00u;       // half2(1, 1), half2(1/16, 1/16)
  const uint32_t M1032 = 0xE408E408u, M72 = 0xD480D480u;           // half2(-1032, -1032), half2(-72, -72)
  uint4 o;
  o.x = hfma2_u32(and_xor<0x000F000Fu, 0x64086408u>(w), ONE, M1032);
  o.y = hfma2_u32(and_xor<0x00F000F0u, 0x64806480u>(w), SIXTEENTH, M72);
  o.z = hfma2_u32(and_xor<0x000F000Fu, 0x64086408u>(w8), ONE, M1032);
  o.w = hfma2_u32(and_xor<0x00F000F0u, 0x64806480u>(w8), SIXTEENTH, M72);
  return o;
}
// Eight fp16 values (d0 .. d7 in four words) in the same order (0,4) (1,5) (2,6) (3,7).
__device__ __forceinline__ uint4 permute8_h(const uint4& v) {
  return make_uint4(__byte_perm(v.x, v.z, 0x5410), __byte_perm(v.x, v.z, 0x7632), __byte_perm(v.y, v.w, 0x5410),
                    __byte_perm(v.y, v.w, 0x7632));
}
// Byte offset of 16-byte chunk c16 (eight dims; 0..15) of row r inside a [rows][128] fp16 tile.
__device__ __forceinline__ uint32_t tile_off(int r, int c16) {
  return static_cast<uint32_t>((c16 >> 3) * PA_HALF + r * 128 + (((c16 & 7) ^ (r & 7)) << 4));
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
               "l"(src), "r"(bytes), "r"(pq::smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, const uint4& v) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---- tcgen05 forms used here (cta_group::1, kind::f16) ----------------------------------------------------
// Instruction descriptor: fp16 x fp16 -> fp32, A K-major (or in tensor memory), B K-major or MN-major.
__host__ __device__ constexpr uint32_t idesc_f16(int M, int N, bool b_mn_major) {
  return (1u << 4) /*D = f32*/ | (0u << 7) /*A = f16*/ | (0u << 10) /*B = f16*/ | (b_mn_major ? (1u << 16) : 0u) |
         (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}
// Shared-memory descriptor of a 128-byte-swizzled operand whose rows are 128 bytes and whose 8-row groups are
// 1024 bytes apart. K-major use: rows = M/N index, the row's bytes = 64 K elements (lbo unused). MN-major use:
// rows = K index, the row's bytes = 64 M/N elements, lbo = distance to the next 64 M/N elements.
__device__ __forceinline__ uint64_t desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr >> 4) & 0x3FFF);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
__device__ __forceinline__ void mma_f16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 16 / 32 consecutive 32-bit columns: thread i of the warp owns lane (base + i).
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// DYN (group-wise dynamic KV, Table 1 O1): every key's score and value row take the key's own step, read by the
// softmax warps (all lanes the same address); the reference exponent is then the exact running maximum, so that
// P * step stays inside fp16 for any step, and O is accumulated in value units.
template <bool DYN>
__global__ void __launch_bounds__(PA_THREADS, 1) prefill_attn_kernel(const PrefillParams p) {
  extern __shared__ uint8_t pa_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(pa_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_buf = smem;                                // two Q tiles
  uint8_t* kv_buf = q_buf + 2 * PA_TILE;                // stage s: K tile, then V tile
  uint8_t* land = kv_buf + PA_STAGES * 2 * PA_TILE;     // stage s: packed K rows, then packed V rows
  PaBarriers* bars = reinterpret_cast<PaBarriers*>(land + PA_STAGES * PA_LAND);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y, G = p.G;
  const int R = 256 / G;                                   // query tokens of this CTA
  const int t0 = (static_cast<int>(gridDim.x) - 1 - static_cast<int>(blockIdx.x)) * R;  // long tiles first
  const int n_ctx = min(p.T, t0 + R);                      // cached keys any row of this CTA may see
  const int n_kt = (n_ctx + PA_KEYS - 1) / PA_KEYS;
  const int has_prefix = p.n_prefix > 0 ? 1 : 0;
  const int n_tiles = has_prefix + n_kt;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < PA_STAGES; ++i) {
      pq::mbar_init(&bars->land_full[i], 1);
      pq::mbar_init(&bars->land_empty[i], PA_EXPAND_WARPS);
      pq::mbar_init(&bars->kv_full[i], PA_EXPAND_WARPS);
      pq::mbar_init(&bars->kv_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      pq::mbar_init(&bars->s_full[i], 1);
      pq::mbar_init(&bars->p_full[i], 4);
      pq::mbar_init(&bars->o_final[i], 1);
    }
    pq::mbar_init(&bars->q_ready, PA_SOFTMAX_WARPS);
    pq::mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    pq::mbar_fence_init();
  }
  if (warp == PA_WARP_MMA) {
    pq::tmem_alloc(&bars->tmem_base, PA_TMEM_COLS);
    pq::tmem_relinquish();
  }
  pq::tc_fence_before();
  __syncthreads();
  pq::tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  // Bounded wait; also gives up when another role of the CTA has raised the abort flag.
  auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
    if (pq::mbar_try_wait(bar, parity)) return true;
    const long long c0 = clock64();
    for (;;) {
      if (pq::mbar_try_wait(bar, parity)) return true;
      if (*abort_flag) return false;
      if (clock64() - c0 > p.wait_clocks) return false;
    }
  };
  auto give_up = [&]() {
    bars->abort_flag = 1;
    pq::report(p.status, PQ_ERR_TIMEOUT);
  };

  const float l2e = 1.4426950408889634f;
  int loads_issued = 0;  // loader lane only

  if (warp < PA_SOFTMAX_WARPS) {
    // ================================================================== softmax warps: one thread per query row
    const int i = warp >> 2, row = (warp & 3) * 32 + lane;      // Q tile and row inside it
    const int r_cta = i * PA_ROWS + row;
    const int tok_raw = t0 + r_cta / G, head = h * G + r_cta % G;
    const int tok = min(tok_raw, p.T - 1);
    {
      // Q staging: the warp brings its 32 rows in, two rows (512 contiguous bytes) per load instruction; a thread per
      // row with 16-byte loads 256 bytes apart costs 32 tag look-ups per instruction and ~8000 clocks before the first MMA.
      const uint32_t dst = pq::smem_u32(q_buf + i * PA_TILE);
      const int c16 = lane & 15, lg = __ffs(G) - 1;
      uint4 qv[16];
#pragma unroll
      for (int it = 0; it < 16; ++it) {
        const int rq = i * PA_ROWS + (warp & 3) * 32 + it * 2 + (lane >> 4);
        const int tq = min(t0 + (rq >> lg), p.T - 1), hq = h * G + (rq & (G - 1));  // G is a power of two
        const uint4* src = reinterpret_cast<const uint4*>(p.q + static_cast<int64_t>(tq) * p.ldq + hq * 128) + c16;  // eight bf16: dims 8 c16 .. +7
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"  // volatile: the sixteen requests go out before the first use
                     : "=r"(qv[it].x), "=r"(qv[it].y), "=r"(qv[it].z), "=r"(qv[it].w)
                     : "l"(src));
      }
#pragma unroll
      for (int it = 0; it < 16; ++it) {
        const uint32_t w[4] = {qv[it].x, qv[it].y, qv[it].z, qv[it].w};
        float f[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = __uint_as_float((e & 1) ? (w[e >> 1] & 0xFFFF0000u) : (w[e >> 1] << 16));
        sts128(dst + tile_off((warp & 3) * 32 + it * 2 + (lane >> 4), c16),
               make_uint4(pack_h2(f[0], f[4]), pack_h2(f[1], f[5]), pack_h2(f[2], f[6]), pack_h2(f[3], f[7])));
      }
      pq::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) pq::mbar_arrive(&bars->q_ready);
    }
    const float sk = DYN ? 1.0f : __ldg(p.s_k + h), sv = DYN ? 1.0f : __ldg(p.s_v + h);
    const float scale_ctx = sk * p.sm_scale * l2e, scale_pre = p.sm_scale * l2e, log2_sv = log2f(sv);
    const float* skb = DYN ? p.sk_tok + static_cast<int64_t>(h) * p.Tmax : nullptr;
    const float* svb = DYN ? p.sv_tok + static_cast<int64_t>(h) * p.Tmax : nullptr;
    constexpr float LAZY = DYN ? 0.0f : PA_LAZY;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_base + i * 128, o_addr = tmem_base + lane_base + 256 + i * 128;
    const int tile_min_tok = t0 + (i * PA_ROWS) / G;
    float m_ref = -INFINITY, l = 0.0f;
    bool ok = true;
    for (int jt = 0; jt < n_tiles; ++jt) {
      const bool is_pre = has_prefix && jt == 0;
      const int key0 = (jt - has_prefix) * PA_KEYS;
      if (__any_sync(0xffffffffu, !wait(&bars->s_full[i], jt & 1))) {
        ok = false;
        break;
      }
      pq::tc_fence_after();
      const int n_chunks = is_pre ? PA_MAX_PREFIX / 32 : PA_KEYS / 32;
      const float scale = is_pre ? scale_pre : scale_ctx;
      const bool need_mask = is_pre ? (p.n_prefix < PA_MAX_PREFIX) : (key0 + PA_KEYS - 1 > tile_min_tok || key0 + PA_KEYS > n_ctx);
      const int limit = is_pre ? p.n_prefix : min(n_ctx - key0, tok - key0 + 1);  // columns below it are visible
      // ---- pass 1: the row's maximum over the visible keys of this tile. The next 32 columns are requested before
      // the current ones are worked on (the last request is pass 2's first), and four partial maxima keep the
      // comparisons from forming one chain.
      uint32_t rr[2][32];
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      pq::tmem_ld_32x32(s_addr, rr[0]);
#pragma unroll
      for (int c = 0; c < PA_KEYS / 32; ++c) {
        if (c < n_chunks) {
          pq::tmem_ld_wait_for(rr[c & 1]);
          pq::tmem_ld_32x32(s_addr + (c + 1 < n_chunks ? (c + 1) * 32 : 0), rr[(c + 1) & 1]);
          const uint32_t(&r)[32] = rr[c & 1];
          if (DYN && !is_pre) {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int col = c * 32 + e;
              const float v = __uint_as_float(r[e]) * __ldg(skb + min(key0 + col, p.Tmax - 1));
              mx4[e & 3] = fmaxf(mx4[e & 3], col < limit ? v : -INFINITY);
            }
          } else if (need_mask) {
#pragma unroll
            for (int e = 0; e < 32; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], c * 32 + e < limit ? __uint_as_float(r[e]) : -INFINITY);
          } else {
#pragma unroll
            for (int e = 0; e < 32; e += 2) mx4[(e >> 1) & 3] = max3f(mx4[(e >> 1) & 3], __uint_as_float(r[e]), __uint_as_float(r[e + 1]));
          }
        }
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float mx_s = mx * scale;
      const bool grow = mx_s > m_ref + LAZY;  // also the first visible key of a row (m_ref = -inf)
      if (__any_sync(0xffffffffu, grow)) {
        const float m_new = grow ? mx_s : m_ref;
        const float alpha = grow ? ex2f(m_ref - m_new) : 1.0f;  // 2^(-inf) = 0 for a row that had seen nothing
        l *= alpha;
        if (jt > 0) {  // S_i of this tile is complete, so O_i += P V of the tile before is, too
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            pq::tmem_ld_32x32(o_addr + c * 32, r);
            pq::tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
            tmem_st_32x32(o_addr + c * 32, r);
          }
        }
        m_ref = m_new;
      }
      // ---- pass 2: P = 2^(s * scale - m), fp16, written over the first columns of S_i. Prefix values are real
      // values while O is kept in code units: their P carries 1 / s_v, as an offset of the exponent, and the tile's
      // part of the denominator is multiplied back by s_v.
      const float m_use = m_ref == -INFINITY ? 0.0f : m_ref;  // such a row has every column masked
      const float m_off = (!DYN && is_pre) ? m_use + log2_sv : m_use;
      const float2 scale2 = make_float2(scale, scale), moff2 = make_float2(-m_off, -m_off);
      float2 l4[4] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
#pragma unroll
      for (int c = 0; c < PA_KEYS / 32; ++c) {  // n_chunks is even: pass 1 left the request for columns 0..31 in rr[0]
        if (c < n_chunks) {
          pq::tmem_ld_wait_for(rr[c & 1]);
          if (c + 1 < n_chunks) pq::tmem_ld_32x32(s_addr + (c + 1) * 32, rr[(c + 1) & 1]);
          const uint32_t(&r)[32] = rr[c & 1];
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float2 sc = make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1]));
            float w0 = 1.0f, w1 = 1.0f;
            if (DYN && !is_pre) {
              const int j0 = min(key0 + c * 32 + e, p.Tmax - 1), j1 = min(key0 + c * 32 + e + 1, p.Tmax - 1);
              sc.x *= __ldg(skb + j0), sc.y *= __ldg(skb + j1);
              w0 = __ldg(svb + j0), w1 = __ldg(svb + j1);
            }
            const float2 x = __ffma2_rn(sc, scale2, moff2);
            float2 pp = make_float2(ex2f(x.x), ex2f(x.y));
            if (need_mask || DYN) {
              pp.x = c * 32 + e < limit ? pp.x : 0.0f;
              pp.y = c * 32 + e + 1 < limit ? pp.y : 0.0f;
            }
            l4[(e >> 1) & 3] = __fadd2_rn(l4[(e >> 1) & 3], pp);
            pk[e >> 1] = DYN ? pack_h2(pp.x * w0, pp.y * w1) : pack_h2(pp.x, pp.y);
          }
          tmem_st_32x16(s_addr + c * 16, pk);
        }
      }
      {
        const float lt = ((l4[0].x + l4[0].y) + (l4[1].x + l4[1].y)) + ((l4[2].x + l4[2].y) + (l4[3].x + l4[3].y));
        l += (!DYN && is_pre) ? lt * sv : lt;
      }
      tmem_st_wait();
      pq::tc_fence_before();
      __syncwarp();
      if (lane == 0) pq::mbar_arrive(&bars->p_full[i]);
    }
    if (ok && __any_sync(0xffffffffu, !wait(&bars->o_final[i], 0))) ok = false;
    if (ok) {
      pq::tc_fence_after();
      const float norm = l > 0.0f ? sv / l : 0.0f;
      __nv_bfloat16* dst = p.out + (static_cast<int64_t>(tok) * p.Hq + head) * 128;
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        pq::tmem_ld_32x32(o_addr + c * 32, r);
        pq::tmem_ld_wait();
        if (tok_raw < p.T) {
#pragma unroll
          for (int a = 0; a < 4; ++a) {  // columns 8a .. 8a+7 hold dims 0,4,1,5,2,6,3,7 of the group
            float v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[8 * a + e]) * norm;
            const __nv_bfloat162 d01 = __floats2bfloat162_rn(v[0], v[2]), d23 = __floats2bfloat162_rn(v[4], v[6]);
            const __nv_bfloat162 d45 = __floats2bfloat162_rn(v[1], v[3]), d67 = __floats2bfloat162_rn(v[5], v[7]);
            *reinterpret_cast<uint4*>(dst + c * 32 + a * 8) =
                make_uint4(*reinterpret_cast<const uint32_t*>(&d01), *reinterpret_cast<const uint32_t*>(&d23),
                           *reinterpret_cast<const uint32_t*>(&d45), *reinterpret_cast<const uint32_t*>(&d67));
          }
        }
      }
    } else if (lane == 0) {
      give_up();
    }
  } else if (warp < PA_WARP_MMA) {
    // ================================================================== expansion warps
    const int tid_e = (warp - PA_WARP_EXPAND0) * 32 + lane;
    bool ok = true;
    for (int jt = 0; jt < n_tiles && ok; ++jt) {
      const int stage = jt % PA_STAGES;
      const bool is_pre = has_prefix && jt == 0;
      if (__any_sync(0xffffffffu, !wait(&bars->kv_empty[stage], ((jt / PA_STAGES) & 1) ^ 1))) {
        ok = false;
        break;
      }
      const uint32_t k_tile = pq::smem_u32(kv_buf + stage * 2 * PA_TILE), v_tile = k_tile + PA_TILE;
      if (is_pre) {
        // full-precision rows as they are stored (reordered inside groups of eight dims); rows past n_prefix are zero
        for (int unit = tid_e; unit < PA_MAX_PREFIX * 16; unit += PA_EXPAND_WARPS * 32) {
          const int row = unit >> 4, c16 = unit & 15;
          uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
          if (row < p.n_prefix) {
            const int64_t off = (static_cast<int64_t>(h) * p.n_prefix + row) * 128 + c16 * 8;
            kv4 = permute8_h(__ldg(reinterpret_cast<const uint4*>(p.prefix_k + off)));
            vv4 = permute8_h(__ldg(reinterpret_cast<const uint4*>(p.prefix_v + off)));
          }
          sts128(k_tile + tile_off(row, c16), kv4);
          sts128(v_tile + tile_off(row, c16), vv4);
        }
      } else {
        const int kt = jt - has_prefix, slot = kt % PA_STAGES;
        if (__any_sync(0xffffffffu, !wait(&bars->land_full[slot], (kt / PA_STAGES) & 1))) {
          ok = false;
          break;
        }
        const uint32_t src = pq::smem_u32(land + slot * PA_LAND);
#pragma unroll 2
        for (int it = 0; it < PA_KEYS * 4 / (PA_EXPAND_WARPS * 32); ++it) {  // 128 keys x 4 chunks of 16 packed bytes
          const int unit = it * (PA_EXPAND_WARPS * 32) + tid_e, row = unit >> 2, part = unit & 3;  // 32 dims: chunks 4 part .. +3
          const uint4 kw = lds128(src + unit * 16), vw = lds128(src + PA_KEYS * 64 + unit * 16);
          const uint32_t kk[4] = {kw.x, kw.y, kw.z, kw.w}, vv[4] = {vw.x, vw.y, vw.z, vw.w};
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            sts128(k_tile + tile_off(row, 4 * part + w), expand8(kk[w]));
            sts128(v_tile + tile_off(row, 4 * part + w), expand8(vv[w]));
          }
        }
        __syncwarp();
        if (lane == 0) pq::mbar_arrive(&bars->land_empty[slot]);
      }
      pq::fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's async proxy
      __syncwarp();
      if (lane == 0) pq::mbar_arrive(&bars->kv_full[stage]);
    }
    if (!ok && lane == 0) give_up();
  } else if (warp == PA_WARP_LOAD) {
    // ================================================================== loader
    if (lane == 0) {
      bool ok = true;
      for (int kt = 0; kt < n_kt; ++kt) {
        const int slot = kt % PA_STAGES;
        if (!wait(&bars->land_empty[slot], ((kt / PA_STAGES) & 1) ^ 1)) {
          ok = false;
          break;
        }
        const uint32_t bytes = static_cast<uint32_t>(min(PA_KEYS, n_ctx - kt * PA_KEYS)) * 64u;
        const int64_t off = (static_cast<int64_t>(h) * p.Tmax + static_cast<int64_t>(kt) * PA_KEYS) * 64;
        const uint32_t dst = pq::smem_u32(land + slot * PA_LAND);
        pq::mbar_arrive_expect_tx(&bars->land_full[slot], 2 * bytes);
        bulk_load(dst, p.kq + off, bytes, &bars->land_full[slot]);
        bulk_load(dst + PA_KEYS * 64, p.vq + off, bytes, &bars->land_full[slot]);
        loads_issued = kt + 1;
      }
      if (!ok) give_up();
    }
  } else {
    // ================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC_S = idesc_f16(PA_ROWS, PA_KEYS, false), IDESC_S_PRE = idesc_f16(PA_ROWS, PA_MAX_PREFIX, false);
      constexpr uint32_t IDESC_O = idesc_f16(PA_ROWS, 128, true);
      auto issue_s = [&](int i, int jt) {
        const bool is_pre = has_prefix && jt == 0;
        const uint32_t q_addr = pq::smem_u32(q_buf + i * PA_TILE), k_addr = pq::smem_u32(kv_buf + (jt % PA_STAGES) * 2 * PA_TILE);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {  // 16 head dims per instruction
          const uint32_t off = (kk >> 2) * PA_HALF + (kk & 3) * 32;
          mma_f16_ss(tmem_base + i * 128, desc_sw128(q_addr + off, 16), desc_sw128(k_addr + off, 16), is_pre ? IDESC_S_PRE : IDESC_S,
                     kk ? 1u : 0u);
        }
        pq::mma_commit(&bars->s_full[i]);
      };
      auto issue_pv = [&](int i, int jt) {
        const bool is_pre = has_prefix && jt == 0;
        const uint32_t v_addr = pq::smem_u32(kv_buf + (jt % PA_STAGES) * 2 * PA_TILE + PA_TILE);
        const int n_steps = is_pre ? PA_MAX_PREFIX / 16 : PA_KEYS / 16;  // 16 keys per instruction
        for (int kk = 0; kk < n_steps; ++kk)
          mma_f16_ts(tmem_base + 256 + i * 128, tmem_base + i * 128 + kk * 8, desc_sw128(v_addr + kk * 2048, PA_HALF), IDESC_O,
                     (jt > 0 || kk > 0) ? 1u : 0u);
      };
      bool ok = wait(&bars->q_ready, 0) && wait(&bars->kv_full[0], 0);
      if (ok) {
        pq::tc_fence_after();
        issue_s(0, 0);
        issue_s(1, 0);
      }
      for (int jt = 0; jt < n_tiles && ok; ++jt) {
        for (int i = 0; i < 2 && ok; ++i) {
          if (!wait(&bars->p_full[i], jt & 1)) {
            ok = false;
            break;
          }
          pq::tc_fence_after();
          issue_pv(i, jt);
          if (i == 1) pq::mma_commit(&bars->kv_empty[jt % PA_STAGES]);  // both tiles' S and P V of this stage are issued
          if (jt + 1 < n_tiles) {
            if (i == 0 && !wait(&bars->kv_full[(jt + 1) % PA_STAGES], ((jt + 1) / PA_STAGES) & 1)) {
              ok = false;
              break;
            }
            pq::tc_fence_after();
            issue_s(i, jt + 1);
          } else {
            pq::mma_commit(&bars->o_final[i]);
          }
        }
      }
      if (!ok) give_up();
      // whatever was issued has finished before tensor memory is released or shared memory given back
      pq::mma_commit(&bars->drain);
      pq::mbar_wait(&bars->drain, 0);
    }
  }

  pq::tc_fence_before();
  __syncthreads();
  if (warp == PA_WARP_LOAD && lane == 0 && bars->abort_flag) {
    // copies that nobody consumed must have landed before the CTA may exit
    for (int kt = max(0, loads_issued - PA_STAGES); kt < loads_issued; ++kt) pq::mbar_wait(&bars->land_full[kt % PA_STAGES], (kt / PA_STAGES) & 1);
  }
  __syncthreads();
  if (warp == PA_WARP_MMA) {
    pq::tc_fence_after();
    pq::tmem_dealloc(tmem_base, PA_TMEM_COLS);
  }
}

}  // namespace

extern "C" pq_status pq_prefill_attn_kv4_prefix(pq_ctx* ctx, const pq_kv4_cache* c, int32_t seq, const void* q, int64_t ldq,
                                                int32_t T, void* out, float sm_scale, void* stream) {
  if (!ctx || !c || !q || !out || !c->kq || !c->vq) return PQ_ERR_INVALID_ARG;
  if ((c->sk_tok != nullptr) != (c->sv_tok != nullptr)) return PQ_ERR_INVALID_ARG;
  const bool dyn = c->sk_tok != nullptr;
  if (!dyn && (!c->s_k || !c->s_v)) return PQ_ERR_INVALID_ARG;
  if (ldq < static_cast<int64_t>(c->Hq) * 128) return PQ_ERR_INVALID_ARG;
  if (T < 0 || seq < 0 || seq >= c->B || c->Hkv <= 0 || c->Hq <= 0 || c->n_prefix < 0 || !(sm_scale > 0.0f)) return PQ_ERR_INVALID_ARG;
  if (c->n_prefix > 0 && (!c->prefix_k || !c->prefix_v)) return PQ_ERR_INVALID_ARG;
  if (c->D != 128 || c->Hq % c->Hkv != 0 || T > c->Tmax || c->n_prefix > PA_MAX_PREFIX || c->Hkv > 65535) return PQ_ERR_SHAPE;
  const int G = c->Hq / c->Hkv;
  if (G != 1 && G != 2 && G != 4 && G != 8) return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(c->kq) & 15) || (reinterpret_cast<uintptr_t>(c->vq) & 15) ||
      (reinterpret_cast<uintptr_t>(q) & 15) || (ldq & 7) || (reinterpret_cast<uintptr_t>(out) & 15) ||
      (c->n_prefix > 0 && ((reinterpret_cast<uintptr_t>(c->prefix_k) & 15) || (reinterpret_cast<uintptr_t>(c->prefix_v) & 15))))
    return PQ_ERR_ALIGN;
  if (T == 0) return PQ_OK;
  PrefillParams p{};
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
  p.sk_tok = dyn ? c->sk_tok + static_cast<int64_t>(seq) * c->Hkv * c->Tmax : nullptr;
  p.sv_tok = dyn ? c->sv_tok + static_cast<int64_t>(seq) * c->Hkv * c->Tmax : nullptr;
  p.status = ctx->d_status;
  p.wait_clocks = ctx->wait_clocks;
  p.sm_scale = sm_scale;
  p.T = T, p.Hq = c->Hq, p.Hkv = c->Hkv, p.G = G, p.n_prefix = c->n_prefix, p.Tmax = c->Tmax;
  static bool attr_set[64] = {};
  if (ctx->device < 0 || ctx->device >= 64) return PQ_ERR_UNSUPPORTED;
  if (!attr_set[ctx->device]) {
    if (cudaFuncSetAttribute(prefill_attn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(PA_SMEM_BYTES)) != cudaSuccess ||
        cudaFuncSetAttribute(prefill_attn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(PA_SMEM_BYTES)) != cudaSuccess)
      return PQ_ERR_CUDA;
    attr_set[ctx->device] = true;
  }
  const int R = 256 / G;
  dim3 grid((T + R - 1) / R, c->Hkv);
  if (dyn)
    prefill_attn_kernel<true><<<grid, PA_THREADS, PA_SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(p);
  else
    prefill_attn_kernel<false><<<grid, PA_THREADS, PA_SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(p);
  return pq_launch_status();
}

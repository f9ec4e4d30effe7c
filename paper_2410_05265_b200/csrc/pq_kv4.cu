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
                      int32_t* __restrict__ len, int B, int T_new, int Hkv, int Tmax, int64_t ld_tok, int32_t* status,
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
    const int64_t src = bt * ld_tok + h * 128 + part * 32;
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
  // the last CTA to finish advances the lengths (every other CTA has read them by then); a lone
  // CTA, the usual case at decode, needs no ticket
  if (gridDim.x > 1) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  } else if (threadIdx.x == 0) {
    last = 1;
  }
  __syncthreads();
  if (last) {
    for (int b = threadIdx.x; b < B; b += AP_THREADS) len[b] += T_new;
    if (threadIdx.x == 0 && gridDim.x > 1) *ticket = 0;
  }
}

// ================================================================================= decode attention
constexpr int DA_WARPS = 4;
constexpr int DA_THREADS = DA_WARPS * 32;
constexpr int DA_MAX_SPLITS = 32;
constexpr int DA_MAX_PREFIX = 64;
constexpr int DA_ROWS = 8;  // query heads per KV head the MMA tile can carry
constexpr int DA_TICKET0 = 16;
constexpr float DA_HEADROOM = 15.0f;  // log2 units a score may exceed the reference exponent before it is moved
constexpr int DA_ROUND = 128;                     // keys staged per round (one half of the staging buffer)
constexpr int DA_CHUNK = 64;                      // keys per bulk copy and per barrier
constexpr int DA_CHUNKS = DA_ROUND / DA_CHUNK;
#ifndef PQ_DA_SLOTS
#define PQ_DA_SLOTS 2
#endif
#ifndef PQ_DA_EARLY
#define PQ_DA_EARLY 1
#endif
constexpr int DA_SLOTS = PQ_DA_SLOTS;             // rounds of staging per CTA
constexpr int DA_EARLY = PQ_DA_EARLY;             // rounds requested at kernel entry
constexpr int DA_HALF_BYTES = DA_ROUND * 64 * 2;  // one slot: packed K rows, then packed V rows
constexpr int DA_SMEM_BYTES = DA_SLOTS * DA_HALF_BYTES;  // 32 KB
static_assert(DA_CHUNK == 16 * DA_WARPS, "one 16-key block per warp per chunk");
constexpr int DA_SO_STRIDE = 136;                 // floats per (warp, head) row of the per-warp partial outputs
static_assert(DA_SMEM_BYTES >= (DA_WARPS * DA_SO_STRIDE + 128) * DA_ROWS * 4, "the staging area is reused for the partials");

// D (+)= A * B, m16n8k16, fp16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_f16_16816_full(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                   uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// (a & M) ^ C in one LOP3; the constants are immediates of the instruction stream, so the compiler is
// free to keep them wherever it likes instead of re-creating register copies next to every use
template <uint32_t M, uint32_t C>
__device__ __forceinline__ uint32_t and_xor(uint32_t a) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(a), "n"(M), "n"(C));  // (a & b) ^ c
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
// 8x8 transpose of 16-bit elements across the warp: lane (g, t) gives row g, columns 2t, 2t+1 and
// receives row g, columns 2t, 2t+1 of the transposed matrix.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier.
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
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}

// ---- thread-block cluster helpers (distributed shared memory) --------------------------------------
__device__ __forceinline__ void cluster_arrive_wait() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_cta(uint32_t smem_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t a) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t a) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
  return v;
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
  float* ws_o;   // [B*Hkv, S, G, 128] partial outputs, already in value units
  float* ws_ml;  // [B*Hkv, S, G, 2]   running maximum (log2 units) and denominator
  uint32_t* tickets;
  int32_t* status;  // device status word; null for the entry point that has no context
  long long wait_clocks;  // bound of the waits for staged cache rows, in SM clocks
  float sm_scale;
  int B, Hq, Hkv, G, n_prefix, Tmax;
  // fused append (decode_attn_kernel<.., true>): the new token's k, v [B, Hkv, 128], the writable lengths and one
  // grid-wide counter
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  int32_t* len_rw;
  uint32_t* len_tickets;
};

// Grid (splits, Hkv, B). The cache of one (sequence, KV head) is cut into rounds of 128 keys; split s
// takes the rounds s, s + S, s + 2S, ... so that where its first rounds lie does not depend on the
// sequence length: their bulk copies into shared memory start with the first instructions, before
// len[b] has come back from memory (a round past the end is copied all the same when it lies inside
// the cache allocation, and is then ignored). Three rounds are in flight ahead of the warps, 64 keys
// per copy and barrier, issued by one lane of the warp that owns the barrier.
// Each warp takes one 16-key block of every 64-key chunk:
//   scores   S^T[key, head] with the fp16 MMA, keys on the 16-row side (every operand register is
//            useful). Codes become fp16 in place under an exponent (one LOP3 for two codes: nibbles
//            0 and 2 of a 16-bit half give 1032 + code, nibbles 1 and 3 give 1152 + 16 * code with
//            no shift); the factor 16 is folded into q and the offsets into a per-head constant.
//   softmax  in log2 units against a per-head reference exponent that moves only when a score
//            exceeds it by more than DA_HEADROOM; the reference and the offset constant are one
//            FFMA operand. P is rounded to fp16 and transposed to the operand layout of the next
//            MMA by movmatrix.
//   output   O^T = V^T P^T with the fp16 MMA, head dims on the 16-row side, codes made exact fp16
//            integers; one more MMA with a matrix of ones sums the same rounded P into the
//            denominator.
// The CTA of the last split also scores the full-precision prefix keys and folds them into its partial.
// CLUSTER: the splits of a (sequence, head) form one thread-block cluster and merge their partials
// through distributed shared memory (no workspace, no ticket); otherwise the partials go through the
// caller's workspace and the last CTA to finish merges them.
// FUSED: the call also appends one token per sequence (what pq_kv4_append does for T_new = 1). The attention
// streams the cache as it was; the CTA of the last split quantizes the new k and v of its head, writes their codes
// to row len[b] and folds the new key into its partial like one more full-precision key whose key and value are
// the dequantized codes. The last CTA of the grid to finish (every CTA has read the lengths by then) advances
// every len[b]. As with the two calls, nothing is appended anywhere when any sequence is full.
// MULTI (with CLUSTER): a (sequence, head) has several clusters of eight splits.
template <bool CLUSTER, bool FUSED, bool MULTI = false>
__global__ void __launch_bounds__(DA_THREADS, 4) decode_attn_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t da_stage[];  // DA_SLOTS slots of [K rows | V rows] of one round
  // the per-warp partial outputs reuse the staging area once the key loop is over
  // [warp][head][DA_SO_STRIDE]; head dim d = 16a + 2b + c sits at 16b + 2a + c and the rows are padded so
  // that the 32 lanes of a store cover all banks (a lane holds dims 16g + 2m, +1 of the heads 2t, 2t+1)
  float* sm_o = reinterpret_cast<float*>(da_stage);
  float* cl_o = reinterpret_cast<float*>(da_stage + DA_WARPS * DA_ROWS * DA_SO_STRIDE * 4);  // [G][128]: this CTA's partial (cluster mode)
  __shared__ float2 cl_ml[DA_ROWS];
  __shared__ __align__(8) uint64_t full[DA_SLOTS][DA_CHUNKS];
  __shared__ float sm_ml[DA_WARPS][DA_ROWS][2];
  __shared__ float sm_pre[DA_ROWS][DA_MAX_PREFIX + 1];  // the last column: the key appended by this call
  __shared__ float sm_newv[FUSED ? 128 : 1];             // its dequantized value
  __shared__ float sm_red[DA_WARPS][DA_ROWS];
  __shared__ int sm_full;
  __shared__ int is_last;
  __shared__ volatile int sm_abort;  // a warp's wait for staged rows ran out: every warp leaves the key loop at the same round

  const int split = blockIdx.x, S = gridDim.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = p.G;
  const int bh = b * p.Hkv + h;
  const uint8_t* kbase = p.kq + static_cast<int64_t>(bh) * p.Tmax * 64;
  const uint8_t* vbase = p.vq + static_cast<int64_t>(bh) * p.Tmax * 64;
  const uint32_t stage_addr = pq::smem_u32(da_stage);

  // Programmatic dependent launch: the next kernel of the stream may be placed as this one's CTAs retire. What this
  // kernel reads that its predecessor may have written (everything for the plain call; the query and the new token
  // for the one-launch decode step, whose cache rows and lengths are older than that by its contract) is read after
  // griddepcontrol.wait; the one-launch form requests its first cache rows ahead of the wait.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!FUSED) asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- every small load of the set-up goes out before the first bulk copy: behind the copies of all
  // the CTAs it would wait for megabytes of cache to be served first
  const bool row_ok = g < G;
  const bool has_prefix = split == S - 1 && p.n_prefix > 0;
  uint4 q_raw[4];  // 32 bf16 of query head g: dims 32t .. 32t+31
  auto load_q = [&]() {
    const uint4* q4 = reinterpret_cast<const uint4*>(p.q + (static_cast<int64_t>(b) * p.Hq + h * G + (row_ok ? g : 0)) * 128 + 32 * t);
#pragma unroll
    for (int w = 0; w < 4; ++w) q_raw[w] = row_ok ? __ldg(q4 + w) : make_uint4(0, 0, 0, 0);
  };
  if (!FUSED) load_q();
  // the fused kernel writes the lengths at its end: it reads them past the read-only path
  int len_b = FUSED ? __ldcg(p.len + b) : __ldg(p.len + b);
  const float s_k_h = __ldg(p.s_k + h), s_v_h = __ldg(p.s_v + h);
  // prefix values of the four head dims this thread merges after the key loop, so that the merge does
  // not wait for them (keys past the fourth are read there)
  uint2 pv_early[4];
#pragma unroll
  for (int j = 0; j < 4; ++j)
    pv_early[j] = (has_prefix && j < p.n_prefix)
                      ? __ldg(reinterpret_cast<const uint2*>(p.prefix_v + (static_cast<int64_t>(h) * p.n_prefix + j) * 128) + lane)
                      : make_uint2(0u, 0u);

  const bool has_extra = FUSED && split == S - 1;
  float k_new_d = 0.0f, v_new_d = 0.0f;  // this thread's head dim of the token being appended
  if (FUSED && threadIdx.x == 0) sm_full = 0;
  if (threadIdx.x == 0) sm_abort = 0;
  // the operands of the first 16 (head, prefix key) pairs (all of them for a 4-token prefix under 4 heads)
  uint4 pre_q[2] = {}, pre_k[2] = {};
  auto load_pre = [&](bool want_q, bool want_k) {
    if (!has_prefix) return;
    const int pair = threadIdx.x >> 3, sub = threadIdx.x & 7;
    const bool ok = pair < G * p.n_prefix;
    const int r = ok ? pair / p.n_prefix : 0, j = ok ? pair % p.n_prefix : 0;
    const uint4* qr = reinterpret_cast<const uint4*>(p.q + (static_cast<int64_t>(b) * p.Hq + h * G + r) * 128 + 16 * sub);
    const uint4* kr = reinterpret_cast<const uint4*>(p.prefix_k + (static_cast<int64_t>(h) * p.n_prefix + j) * 128 + 16 * sub);
    if (want_q) pre_q[0] = __ldg(qr), pre_q[1] = __ldg(qr + 1);
    if (want_k) pre_k[0] = __ldg(kr), pre_k[1] = __ldg(kr + 1);
  };
  load_pre(!FUSED, true);

  // ---- staging. Barrier n = 2 * slot + chunk belongs to warp n % 4: its lane 0 initialises it and
  // issues every copy that completes on it. Local round i of this split is the global round
  // split + i * S and uses slot i % DA_SLOTS; the first DA_EARLY rounds are requested before the length
  // is known when they lie inside the allocation as a whole.
  auto round_key0 = [&](int i) { return (split + i * S) * DA_ROUND; };
  auto speculated = [&](int i) { return round_key0(i) + DA_ROUND <= p.Tmax; };  // i < DA_EARLY only
  // copies started on the barriers this warp owns (barrier n belongs to warp n % DA_WARPS; lane 0 of the warp counts)
  constexpr int DA_OWNED = (DA_SLOTS * DA_CHUNKS + DA_WARPS - 1) / DA_WARPS;
  int n_issued[DA_OWNED] = {};
  auto issue_chunk = [&](int i, int c, int n_keys) {  // lane 0 of the owning warp
    ++n_issued[((i % DA_SLOTS) * DA_CHUNKS + c) / DA_WARPS];
    const uint32_t slot = stage_addr + (i % DA_SLOTS) * DA_HALF_BYTES;
    const int k0 = round_key0(i) + c * DA_CHUNK;
    const uint32_t bytes = static_cast<uint32_t>(n_keys) * 64u;
    uint64_t* bar = &full[i % DA_SLOTS][c];
    pq::mbar_arrive_expect_tx(bar, 2 * bytes);
    bulk_load(slot + c * (DA_CHUNK * 64), kbase + static_cast<int64_t>(k0) * 64, bytes, bar);
    bulk_load(slot + DA_ROUND * 64 + c * (DA_CHUNK * 64), vbase + static_cast<int64_t>(k0) * 64, bytes, bar);
  };
  if (lane == 0) {
    for (int n = warp; n < DA_SLOTS * DA_CHUNKS; n += DA_WARPS) pq::mbar_init(&full[0][0] + n, 1);
    pq::mbar_fence_init();
    for (int n = warp; n < DA_EARLY * DA_CHUNKS; n += DA_WARPS)
      if (speculated(n / DA_CHUNKS)) issue_chunk(n / DA_CHUNKS, n % DA_CHUNKS, DA_CHUNK);
  }
  if (FUSED) {
    // the first cache rows are on their way: now the predecessor's results (query, new token) may be read
    asm volatile("griddepcontrol.wait;" ::: "memory");
    load_q();
    load_pre(true, false);
    if (has_extra) {
      const int64_t off = (static_cast<int64_t>(b) * p.Hkv + h) * 128 + threadIdx.x;
      k_new_d = __bfloat162float(p.k_new[off]), v_new_d = __bfloat162float(p.v_new[off]);
    }
  }
  __syncthreads();  // every barrier is initialised (all warps are still together here: this costs nothing)
  if (FUSED) {  // one verdict for the whole batch, as the append call gives it
    for (int i = threadIdx.x; i < p.B; i += DA_THREADS) {
      const int l = __ldcg(p.len + i);
      if (l < 0 || l + 1 > p.Tmax) sm_full = 1;
    }
    __syncthreads();
  }
  const bool append_ok = FUSED && !sm_full;
  const int len_raw = len_b;
  // Called by every thread of every CTA when the CTA is done. The last CTA of the whole grid advances every length:
  // by then each CTA has read the lengths it needs (its own sequence's, and all of them for the verdict above),
  // so no CTA can ever see a length this launch has already moved.
  auto finish_append = [&]() {
    if (!FUSED) return;
    if (!append_ok) {
      if (threadIdx.x == 0 && p.status && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) pq::report(p.status, PQ_ERR_SHAPE);
      return;
    }
    __syncthreads();  // is_last is free again, and this CTA's cache writes precede the ticket
    if (threadIdx.x == 0) {
      __threadfence();
      const uint32_t n_ctas = gridDim.x * gridDim.y * gridDim.z;
      is_last = atomicAdd(p.len_tickets, 1u) == n_ctas - 1;
    }
    __syncthreads();
    if (is_last) {
      for (int i = threadIdx.x; i < p.B; i += DA_THREADS) p.len_rw[i] = __ldcg(p.len_rw + i) + 1;
      if (threadIdx.x == 0) *p.len_tickets = 0;
    }
  };
  len_b = len_b < 0 ? 0 : (len_b > p.Tmax ? p.Tmax : len_b);
  const int t1 = len_b;
  const int n_rounds_all = (len_b + DA_ROUND - 1) / DA_ROUND;
  const int n_rounds = n_rounds_all > split ? (n_rounds_all - split + S - 1) / S : 0;  // of this split
  if (lane == 0) {
    for (int n = warp; n < DA_EARLY * DA_CHUNKS; n += DA_WARPS) {
      const int i = n / DA_CHUNKS, k0 = round_key0(i) + (n % DA_CHUNKS) * DA_CHUNK;
      if (!speculated(i) && i < n_rounds && k0 < t1) issue_chunk(i, n % DA_CHUNKS, min(DA_CHUNK, t1 - k0));
    }
  }
  // ---- the last split (it never has more rounds than the others) scores the full-precision prefix keys in fp32, in
  // log2 units: eight lanes per (head, prefix key) pair, 16 dims each, every load issued at once
  if (has_prefix) {
    const int n_pairs = G * p.n_prefix, sub = threadIdx.x & 7;
    for (int pair0 = 0; pair0 < n_pairs; pair0 += DA_THREADS / 8) {
      const int pair = pair0 + (threadIdx.x >> 3);
      const bool ok = pair < n_pairs;
      const int r = ok ? pair / p.n_prefix : 0, j = ok ? pair % p.n_prefix : 0;
      const uint4* qr = reinterpret_cast<const uint4*>(p.q + (static_cast<int64_t>(b) * p.Hq + h * G + r) * 128 + 16 * sub);
      const uint4* kr = reinterpret_cast<const uint4*>(p.prefix_k + (static_cast<int64_t>(h) * p.n_prefix + j) * 128 + 16 * sub);
      const bool early = pair0 == 0;
      const uint4 qv[2] = {early ? pre_q[0] : __ldg(qr), early ? pre_q[1] : __ldg(qr + 1)};
      const uint4 kv[2] = {early ? pre_k[0] : __ldg(kr), early ? pre_k[1] : __ldg(kr + 1)};
      float acc = 0.0f;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint32_t qw[4] = {qv[i].x, qv[i].y, qv[i].z, qv[i].w}, kw[4] = {kv[i].x, kv[i].y, kv[i].z, kv[i].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 kf = __half22float2(*reinterpret_cast<const __half2*>(&kw[e]));
          acc = fmaf(__uint_as_float(qw[e] << 16), kf.x, acc);
          acc = fmaf(__uint_as_float(qw[e] & 0xFFFF0000u), kf.y, acc);
        }
      }
      acc += __shfl_xor_sync(0xffffffffu, acc, 1);
      acc += __shfl_xor_sync(0xffffffffu, acc, 2);
      acc += __shfl_xor_sync(0xffffffffu, acc, 4);
      if (ok && sub == 0) sm_pre[r][j] = acc * p.sm_scale * 1.4426950408889634f;
    }
  }

  // ---- the appended token: codes to the cache, score and value of the new key for this CTA's partial ----------
  if (has_extra && append_ok) {
    const float sk_h = s_k_h;
    const int kc = max(-8, min(7, __float2int_rn(__fdiv_rn(k_new_d, sk_h))));
    const int vc = max(-8, min(7, __float2int_rn(__fdiv_rn(v_new_d, s_v_h))));
    // two head dims per byte, low nibble first: the even thread of a pair writes
    const int kc_hi = __shfl_down_sync(0xffffffffu, kc, 1), vc_hi = __shfl_down_sync(0xffffffffu, vc, 1);
    if ((threadIdx.x & 1) == 0) {
      const int64_t row = (static_cast<int64_t>(bh) * p.Tmax + len_raw) * 64 + (threadIdx.x >> 1);
      const_cast<uint8_t*>(p.kq)[row] = static_cast<uint8_t>((kc & 0xF) | ((kc_hi & 0xF) << 4));
      const_cast<uint8_t*>(p.vq)[row] = static_cast<uint8_t>((vc & 0xF) | ((vc_hi & 0xF) << 4));
    }
    sm_newv[FUSED ? threadIdx.x : 0] = static_cast<float>(vc) * s_v_h;
    for (int r = 0; r < G; ++r) {  // q[r] . k_code over the 128 threads
      float part = __bfloat162float(p.q[(static_cast<int64_t>(b) * p.Hq + h * G + r) * 128 + threadIdx.x]) * static_cast<float>(kc);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      if (lane == 0) sm_red[warp][r] = part;
    }
    __syncthreads();
    if (threadIdx.x < G) {
      float dot = 0.0f;
#pragma unroll
      for (int w = 0; w < DA_WARPS; ++w) dot += sm_red[w][threadIdx.x];
      sm_pre[threadIdx.x][p.n_prefix] = dot * sk_h * p.sm_scale * 1.4426950408889634f;
    }
  }

  // ---- query fragments (fp16 B operand of the score MMA: k = head dims, n = query heads) ----------
  // A 32-bit word of a packed key row holds the codes of dims 8W..8W+7; nibble i of its low half is
  // dim 8W+i, nibble i of its high half dim 8W+4+i. Fragment j of a lane holds (q[D], q[D+4]) in its first and
  // (q[D+1], q[D+5]) / 16 in its second register with D = 32t + 8(j>>1) + 2(j&1), of head g: the k rows
  // 2t, 2t+1 and 2t+8, 2t+9 of score MMA j.
  uint32_t qb[8][2];
  float q_even = 0.0f, q_odd = 0.0f;
  {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const uint4 v = q_raw[w];  // 8 bf16: d = 32t + 8w + 0..7
      const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
      float f[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = __uint_as_float((e & 1) ? (ww[e >> 1] & 0xFFFF0000u) : (ww[e >> 1] << 16));
#pragma unroll
      for (int jj = 0; jj < 2; ++jj) {  // score MMA j = 2w + jj uses nibbles 2jj and 2jj + 1
        const int i0 = 2 * jj;
        const __half2 a0 = __floats2half2_rn(f[i0], f[i0 + 4]);
        const __half2 a2 = __floats2half2_rn(f[i0 + 1] * 0.0625f, f[i0 + 5] * 0.0625f);
        qb[2 * w + jj][0] = *reinterpret_cast<const uint32_t*>(&a0);
        qb[2 * w + jj][1] = *reinterpret_cast<const uint32_t*>(&a2);
        // the offsets are removed with the values the MMA really multiplies
        const float2 e0 = __half22float2(a0), e1 = __half22float2(a2);
        q_even += e0.x + e0.y;
        q_odd += e1.x + e1.y;
      }
    }
    q_even += __shfl_xor_sync(0xffffffffu, q_even, 1);
    q_even += __shfl_xor_sync(0xffffffffu, q_even, 2);
    q_odd += __shfl_xor_sync(0xffffffffu, q_odd, 1);
    q_odd += __shfl_xor_sync(0xffffffffu, q_odd, 2);
  }
  const float scale2 = s_k_h * p.sm_scale * 1.4426950408889634f;  // scores in log2 units
  // The score tile of a lane is (keys g, g + 8) x (heads 2t, 2t + 1): it needs the offset constants of
  // those two heads, which the lanes 8t and 8t + 4 hold.
  const float bias_g = (1032.0f * q_even + 1152.0f * q_odd) * scale2;
  const float bias0 = __shfl_sync(0xffffffffu, bias_g, 8 * t), bias1 = __shfl_sync(0xffffffffu, bias_g, 8 * t + 4);
  // Reference exponents of heads 2t and 2t + 1 (the same in all lanes of equal t). A head that does not
  // exist keeps a huge one: its probabilities are zero and it never asks for a move.
  float m0 = 2 * t < G ? -INFINITY : 1e30f, m1 = 2 * t + 1 < G ? -INFINITY : 1e30f;
  float bm0 = bias0 + m0, bm1 = bias1 + m1;  // what is subtracted from a raw score

  // Output accumulators of the transposed product: tile m holds, for this lane, o[m][0], o[m][1] =
  // dim 16g+2m of heads 2t, 2t+1 and o[m][2], o[m][3] = 16 x dim 16g+2m+1 of the same heads.
  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f;
  float lacc[4] = {0.0f, 0.0f, 0.0f, 0.0f};  // [0], [1]: denominators of heads 2t, 2t+1

  // byte offsets of this lane's loads inside a staged 16-key block
  const uint32_t k_off = g * 64 + 16 * t;             // key g (and g + 8): 32 codes at dims 32t..32t+31
  const uint32_t v_off = (2 * t) * 64 + 8 * g;        // keys 2t, 2t+1, 2t+8, 2t+9: 16 codes at dims 16g..16g+15
  bool timed_out = false;
  for (int r = 0; r < n_rounds && !timed_out; ++r) {
    const uint32_t ks = stage_addr + (r % DA_SLOTS) * DA_HALF_BYTES;
    const int r0 = round_key0(r);
    const uint32_t parity = (r / DA_SLOTS) & 1;
    // A warp takes one 16-key block of each of the two chunks of a round, in one pass: two independent
    // instruction streams to interleave. A block past the end of the sequence is computed all the
    // same on whatever the buffer holds (any code pattern is a finite fp16 value) with all its
    // probabilities forced to zero.
    const bool round_ok = !__any_sync(0xffffffffu, !pq::mbar_wait_for(&full[r % DA_SLOTS][0], parity, p.wait_clocks) ||
                                                        (r0 + DA_CHUNK < t1 && !pq::mbar_wait_for(&full[r % DA_SLOTS][1], parity, p.wait_clocks)));
    if (!round_ok) {
      sm_abort = 1;
      timed_out = true;
      if (r + DA_SLOTS >= n_rounds) break;  // no CTA barrier is left in the loop: this warp may leave on its own
    }
    if (round_ok) {
    if (r == 0 && lane == 0) {  // the remaining slots are requested once the first data is here
      for (int n = warp; n < DA_SLOTS * DA_CHUNKS; n += DA_WARPS) {  // by the barrier's owner, like every other request
        const int i = n / DA_CHUNKS, k0 = round_key0(i) + (n % DA_CHUNKS) * DA_CHUNK;
        if (n >= DA_EARLY * DA_CHUNKS && i < n_rounds && k0 < t1) issue_chunk(i, n % DA_CHUNKS, min(DA_CHUNK, t1 - k0));
      }
    }
    float c[2][4];  // raw scores: [0], [1] = key g x heads 2t, 2t+1; [2], [3] = key g + 8 x the same heads
    bool dead_lo[2], dead_hi[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int j0 = r0 + u * DA_CHUNK + 16 * warp;
      const uint32_t kb = ks + (j0 - r0) * 64;
      dead_lo[u] = j0 + g >= t1, dead_hi[u] = j0 + 8 + g >= t1;
      const uint4 kc0 = lds128(kb + k_off), kc1 = lds128(kb + k_off + 8 * 64);
      // ---- scores of 16 keys x 8 heads: two accumulation chains over the eight 16-dim steps -------
      float ca[4] = {0.0f, 0.0f, 0.0f, 0.0f}, cb[4] = {0.0f, 0.0f, 0.0f, 0.0f};
      const uint32_t wl[4] = {kc0.x, kc0.y, kc0.z, kc0.w}, wh[4] = {kc1.x, kc1.y, kc1.z, kc1.w};
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const uint32_t wl8 = wl[w] >> 8, wh8 = wh[w] >> 8;
        mma_f16_16816_full(ca, and_xor<0x000F000Fu, 0x64086408u>(wl[w]), and_xor<0x000F000Fu, 0x64086408u>(wh[w]),
                           and_xor<0x00F000F0u, 0x64806480u>(wl[w]), and_xor<0x00F000F0u, 0x64806480u>(wh[w]),
                           qb[2 * w][0], qb[2 * w][1]);
        mma_f16_16816_full(cb, and_xor<0x000F000Fu, 0x64086408u>(wl8), and_xor<0x000F000Fu, 0x64086408u>(wh8),
                           and_xor<0x00F000F0u, 0x64806480u>(wl8), and_xor<0x00F000F0u, 0x64806480u>(wh8),
                           qb[2 * w + 1][0], qb[2 * w + 1][1]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) c[u][i] = ca[i] + cb[i];
    }
    // ---- softmax against the reference exponents: e = log2 of the probability ----------------------
    float e[2][4];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      e[u][0] = dead_lo[u] ? -INFINITY : fmaf(c[u][0], scale2, -bm0);
      e[u][1] = dead_lo[u] ? -INFINITY : fmaf(c[u][1], scale2, -bm1);
      e[u][2] = dead_hi[u] ? -INFINITY : fmaf(c[u][2], scale2, -bm0);
      e[u][3] = dead_hi[u] ? -INFINITY : fmaf(c[u][3], scale2, -bm1);
    }
    // A reference moves only when a score exceeds it by more than DA_HEADROOM (probabilities then stay
    // below 2^15, well inside fp16 and fp32 range; the reference is just a common exponent, the
    // merges below rescale by it). The first pass of a warp always takes this path (e = +inf).
    const float e_max = fmaxf(fmaxf(fmaxf(e[0][0], e[0][1]), fmaxf(e[0][2], e[0][3])), fmaxf(fmaxf(e[1][0], e[1][1]), fmaxf(e[1][2], e[1][3])));
    if (__any_sync(0xffffffffu, e_max > DA_HEADROOM)) {
      float s[2][4];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        s[u][0] = dead_lo[u] ? -INFINITY : fmaf(c[u][0], scale2, -bias0);
        s[u][1] = dead_lo[u] ? -INFINITY : fmaf(c[u][1], scale2, -bias1);
        s[u][2] = dead_hi[u] ? -INFINITY : fmaf(c[u][2], scale2, -bias0);
        s[u][3] = dead_hi[u] ? -INFINITY : fmaf(c[u][3], scale2, -bias1);
      }
      // maxima of heads 2t, 2t+1 over the 32 keys of this pass: over the eight lanes of equal t
      float x0 = fmaxf(fmaxf(s[0][0], s[0][2]), fmaxf(s[1][0], s[1][2])), x1 = fmaxf(fmaxf(s[0][1], s[0][3]), fmaxf(s[1][1], s[1][3]));
#pragma unroll
      for (int d = 4; d < 32; d <<= 1) {
        x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, d));
        x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, d));
      }
      // a warp whose 32 keys all lie past the end keeps its reference (-inf - -inf would not be a number)
      const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);
      const float a_lo = n0 == -INFINITY ? 1.0f : ex2(m0 - n0), a_hi = n1 == -INFINITY ? 1.0f : ex2(m1 - n1);
      m0 = n0, m1 = n1;
      bm0 = bias0 + m0, bm1 = bias1 + m1;
      lacc[0] *= a_lo, lacc[1] *= a_hi, lacc[2] *= a_lo, lacc[3] *= a_hi;
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i][0] *= a_lo, o[i][1] *= a_hi, o[i][2] *= a_lo, o[i][3] *= a_hi;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        e[u][0] = n0 == -INFINITY ? -INFINITY : s[u][0] - m0, e[u][1] = n1 == -INFINITY ? -INFINITY : s[u][1] - m1;
        e[u][2] = n0 == -INFINITY ? -INFINITY : s[u][2] - m0, e[u][3] = n1 == -INFINITY ? -INFINITY : s[u][3] - m1;
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int j0 = r0 + u * DA_CHUNK + 16 * warp;
      const uint32_t vb = ks + (j0 - r0) * 64 + DA_ROUND * 64;
      const uint2 vc0 = lds64(vb + v_off), vc1 = lds64(vb + v_off + 64);
      const uint2 vc2 = lds64(vb + v_off + 8 * 64), vc3 = lds64(vb + v_off + 9 * 64);
      // P in fp16, transposed from (key, head pair) to the (key pair, head) layout of an MMA B operand
      const uint32_t pb0 = movmatrix_trans(pack_half2(ex2(e[u][0]), ex2(e[u][1])));
      const uint32_t pb1 = movmatrix_trans(pack_half2(ex2(e[u][2]), ex2(e[u][3])));
      // the denominator sums the same fp16-rounded probabilities the output MMA multiplies with
      mma_f16_16816_full(lacc, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, pb0, pb1);
      // ---- O^T += V^T P^T: rows = head dims, columns = query heads ------------------------------
      // A merged word pairs the same four dims of two neighbouring keys; its nibbles 0 and 2 give
      // exact codes, nibbles 1 and 3 give 16 * code (rows g+8 of the tile, rescaled at the end).
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const uint32_t sel = (q4 & 1) ? 0x7632u : 0x5410u;
        const uint32_t ya = __byte_perm(q4 < 2 ? vc0.x : vc0.y, q4 < 2 ? vc1.x : vc1.y, sel);
        const uint32_t yb = __byte_perm(q4 < 2 ? vc2.x : vc2.y, q4 < 2 ? vc3.x : vc3.y, sel);
        const uint32_t ya8 = ya >> 8, yb8 = yb >> 8;
        mma_f16_16816_full(o[2 * q4], hsub2_u32(and_xor<0x000F000Fu, 0x64086408u>(ya), 0x64086408u),
                           hsub2_u32(and_xor<0x00F000F0u, 0x64806480u>(ya), 0x64806480u),
                           hsub2_u32(and_xor<0x000F000Fu, 0x64086408u>(yb), 0x64086408u),
                           hsub2_u32(and_xor<0x00F000F0u, 0x64806480u>(yb), 0x64806480u), pb0, pb1);
        mma_f16_16816_full(o[2 * q4 + 1], hsub2_u32(and_xor<0x000F000Fu, 0x64086408u>(ya8), 0x64086408u),
                           hsub2_u32(and_xor<0x00F000F0u, 0x64806480u>(ya8), 0x64806480u),
                           hsub2_u32(and_xor<0x000F000Fu, 0x64086408u>(yb8), 0x64086408u),
                           hsub2_u32(and_xor<0x00F000F0u, 0x64806480u>(yb8), 0x64806480u), pb0, pb1);
      }
    }
    }  // round_ok
    if (r + DA_SLOTS < n_rounds) {  // the slot is free once every warp is past it
      __syncthreads();
      if (sm_abort) {  // the same verdict in every warp: nothing more is requested, the loop ends here
        timed_out = true;
        break;
      }
      for (int c = 0; c < DA_CHUNKS; ++c) {
        const int k0 = round_key0(r + DA_SLOTS) + c * DA_CHUNK;
        if (lane == 0 && warp == ((r % DA_SLOTS) * DA_CHUNKS + c) % DA_WARPS && k0 < t1)
          issue_chunk(r + DA_SLOTS, c, min(DA_CHUNK, t1 - k0));
      }
    }
  }
  // every copy that was started must have landed before the staging area is reused: a round requested ahead of the
  // length and then not needed, and whatever was in flight when a wait ran out (these only wait for memory, hence
  // the generous bound)
  if (lane == 0) {
#pragma unroll
    for (int o = 0; o < DA_OWNED; ++o)
      if (n_issued[o] > 0 && !pq::mbar_wait(&full[0][0] + o * DA_WARPS + warp, (n_issued[o] - 1) & 1)) timed_out = true;
  }
  if (timed_out && lane == 0 && p.status) pq::report(p.status, PQ_ERR_TIMEOUT);
  __syncthreads();  // the staging area becomes the per-warp partial outputs

  // ---- merge the warps of this CTA (and, in the last split, the prefix keys) into one partial ------------
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    const int head = 2 * t + hh;
    if (head < G) {
#pragma unroll
      for (int m = 0; m < 8; ++m)
        *reinterpret_cast<float2*>(sm_o + (warp * DA_ROWS + head) * DA_SO_STRIDE + 16 * m + 2 * g) =
            make_float2(o[m][hh], o[m][2 + hh] * 0.0625f);
    }
  }
  if (g == 0) {
    if (2 * t < G) sm_ml[warp][2 * t][0] = m0, sm_ml[warp][2 * t][1] = lacc[0];
    if (2 * t + 1 < G) sm_ml[warp][2 * t + 1][0] = m1, sm_ml[warp][2 * t + 1][1] = lacc[1];
  }
  __syncthreads();
  {
    // warp w takes the heads w, w + 4; lane c4 of it the head dims 4 c4 .. 4 c4 + 3
    const int n_pre = has_prefix ? p.n_prefix : 0;
    const bool extra = has_extra && append_ok;  // the appended key sits in column n_prefix of sm_pre
    const int c4 = lane;
    const int qpos = 16 * ((2 * c4) & 7) + 2 * (c4 >> 2);  // dims 4 c4, +1 here, dims 4 c4 + 2, +3 sixteen floats on
    for (int r = warp; r < G; r += DA_WARPS) {
      float m = -INFINITY;
#pragma unroll
      for (int w = 0; w < DA_WARPS; ++w) m = fmaxf(m, sm_ml[w][r][0]);
      for (int j = 0; j < n_pre; ++j) m = fmaxf(m, sm_pre[r][j]);
      if (extra) m = fmaxf(m, sm_pre[r][p.n_prefix]);
      float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      float l = 0.0f;
#pragma unroll
      for (int w = 0; w < DA_WARPS; ++w) {
        const float mw = sm_ml[w][r][0];
        const float e = mw == -INFINITY ? 0.0f : ex2(mw - m);
        const float* src = sm_o + (w * DA_ROWS + r) * DA_SO_STRIDE + qpos;
        const float2 lo = *reinterpret_cast<const float2*>(src), hi = *reinterpret_cast<const float2*>(src + 16);
        acc.x = fmaf(lo.x, e, acc.x), acc.y = fmaf(lo.y, e, acc.y), acc.z = fmaf(hi.x, e, acc.z), acc.w = fmaf(hi.y, e, acc.w);
        l = fmaf(sm_ml[w][r][1], e, l);
      }
      // codes -> values; the prefix values below are already in value units
      acc.x *= s_v_h, acc.y *= s_v_h, acc.z *= s_v_h, acc.w *= s_v_h;
      for (int j = 0; j < n_pre; ++j) {
        const float e = ex2(sm_pre[r][j] - m);
        uint2 pv = make_uint2(0u, 0u);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
          if (j == jj) pv = pv_early[jj];
        if (j >= 4) pv = __ldg(reinterpret_cast<const uint2*>(p.prefix_v + (static_cast<int64_t>(h) * p.n_prefix + j) * 128) + c4);
        const float2 v01 = __half22float2(*reinterpret_cast<const __half2*>(&pv.x));
        const float2 v23 = __half22float2(*reinterpret_cast<const __half2*>(&pv.y));
        acc.x = fmaf(e, v01.x, acc.x), acc.y = fmaf(e, v01.y, acc.y), acc.z = fmaf(e, v23.x, acc.z), acc.w = fmaf(e, v23.y, acc.w);
        l += e;
      }
      if (extra) {
        const float e = ex2(sm_pre[r][p.n_prefix] - m);
        const float4 nv = *reinterpret_cast<const float4*>(sm_newv + (FUSED ? 4 * c4 : 0));
        acc.x = fmaf(e, nv.x, acc.x), acc.y = fmaf(e, nv.y, acc.y), acc.z = fmaf(e, nv.z, acc.z), acc.w = fmaf(e, nv.w, acc.w);
        l += e;
      }
      if (CLUSTER) {
        *reinterpret_cast<float4*>(cl_o + r * 128 + 4 * c4) = acc;
        if (c4 == 0) cl_ml[r] = make_float2(m, l);
      } else {
        const int64_t slot = (static_cast<int64_t>(bh) * S + split) * G + r;
        *reinterpret_cast<float4*>(p.ws_o + slot * 128 + 4 * c4) = acc;
        if (c4 == 0) *reinterpret_cast<float2*>(p.ws_ml + slot * 2) = make_float2(m, l);
      }
    }
  }
  // Clusters hold up to eight consecutive splits. One cluster per (sequence, head) writes the result itself;
  // several (few sequences, long caches) each leave one merged partial in the workspace and the last cluster to
  // finish merges those few.
  const int csize = S < 8 ? S : 8, n_clusters = MULTI ? S / csize : 1;
  const int n_parts = CLUSTER ? n_clusters : S;  // partials per (sequence, head) that meet in the workspace
  if (CLUSTER) {
    // every split's partial is in its CTA's shared memory; thread i of the cluster takes (head, four
    // dims) item i and reads the cluster's partials through distributed shared memory, all loads at once
    cluster_arrive_wait();
    const int rank = split % csize, ci = split / csize;
    const int item = rank * DA_THREADS + threadIdx.x;
    if (item < G * 32) {
      const int r = item >> 5, c4 = item & 31;
      const uint32_t o_addr = pq::smem_u32(cl_o + r * 128 + 4 * c4), ml_addr = pq::smem_u32(cl_ml + r);
      float4 v[8];
      float2 ml[8];
#pragma unroll
      for (int sp = 0; sp < 8; ++sp) {
        if (sp < csize) {
          v[sp] = ld_cluster_f4(map_cta(o_addr, sp));
          ml[sp] = ld_cluster_f2(map_cta(ml_addr, sp));
        } else {
          v[sp] = make_float4(0.f, 0.f, 0.f, 0.f);
          ml[sp] = make_float2(-INFINITY, 0.f);
        }
      }
      float m = -INFINITY;
#pragma unroll
      for (int sp = 0; sp < 8; ++sp) m = fmaxf(m, ml[sp].x);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float l = 0.0f;
#pragma unroll
      for (int sp = 0; sp < 8; ++sp) {
        const float w = ml[sp].x == -INFINITY ? 0.0f : ex2(ml[sp].x - m);
        acc.x = fmaf(v[sp].x, w, acc.x), acc.y = fmaf(v[sp].y, w, acc.y), acc.z = fmaf(v[sp].z, w, acc.z), acc.w = fmaf(v[sp].w, w, acc.w);
        l = fmaf(ml[sp].y, w, l);
      }
      if (n_clusters == 1) {
        const float inv = l > 0.0f ? 1.0f / l : 0.0f;
        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 packed;
        packed.x = *reinterpret_cast<const uint32_t*>(&lo), packed.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(p.out + (static_cast<int64_t>(b) * p.Hq + h * G + r) * 128 + 4 * c4) = packed;
      } else {  // this cluster's partial, in the layout of a split's partial
        const int64_t slot = (static_cast<int64_t>(bh) * n_clusters + ci) * G + r;
        *reinterpret_cast<float4*>(p.ws_o + slot * 128 + 4 * c4) = acc;
        if (c4 == 0) *reinterpret_cast<float2*>(p.ws_ml + slot * 2) = make_float2(m, l);
        __threadfence();
      }
    }
    cluster_arrive_wait();  // no CTA leaves while a peer may still read its shared memory
    if (n_clusters == 1 || rank != 0) {
      finish_append();
      return;
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(p.tickets + DA_TICKET0 + bh, 1u) == static_cast<uint32_t>(n_parts - 1));
  __syncthreads();
  if (!is_last) {
    finish_append();
    return;
  }
  __threadfence();

  // ---- last CTA of this (sequence, KV head): merge the partials --------------------------------
  // One L2 round trip: every (m, l) pair and the first eight partial columns of each thread are
  // requested together; the weights are computed while the columns are in flight.
  float* part_m = reinterpret_cast<float*>(da_stage);  // [S][G]; the staging area is free again
  float* part_l = part_m + DA_MAX_SPLITS * DA_ROWS;
  float* part_w = part_l + DA_MAX_SPLITS * DA_ROWS;
  float* head_l = part_w + DA_MAX_SPLITS * DA_ROWS;    // [G]
  for (int i = threadIdx.x; i < n_parts * G; i += DA_THREADS) {
    const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.ws_ml) + static_cast<int64_t>(bh) * n_parts * G + i);
    part_m[i] = ml.x, part_l[i] = ml.y;
  }
  const float4* wo = reinterpret_cast<const float4*>(p.ws_o) + static_cast<int64_t>(bh) * n_parts * G * 32;
  const int n_items = G * 32;  // (head, group of four dims)
  float4 pre[8];
  {
    const int item = threadIdx.x, r = item >> 5, c4 = item & 31;
#pragma unroll
    for (int sp = 0; sp < 8; ++sp)
      pre[sp] = (item < n_items && sp < n_parts) ? __ldcg(wo + (sp * G + r) * 32 + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  __syncthreads();
  if (threadIdx.x < G) {
    const int r = threadIdx.x;
    float m = -INFINITY;
    for (int sp = 0; sp < n_parts; ++sp) m = fmaxf(m, part_m[sp * G + r]);
    float l = 0.0f;
    for (int sp = 0; sp < n_parts; ++sp) {
      const float ms = part_m[sp * G + r];
      const float e = ms == -INFINITY ? 0.0f : ex2(ms - m);  // also covers m == -inf (nothing cached, no prefix)
      part_w[sp * G + r] = e;
      l += part_l[sp * G + r] * e;
    }
    head_l[r] = l;
  }
  __syncthreads();
  for (int item = threadIdx.x; item < n_items; item += DA_THREADS) {
    const int r = item >> 5, c4 = item & 31;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sp0 = 0; sp0 < n_parts; sp0 += 8) {
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int sp = sp0 + u;
        if (sp < n_parts) {
          const float4 v = (sp0 == 0 && item == static_cast<int>(threadIdx.x)) ? pre[u] : __ldcg(wo + (sp * G + r) * 32 + c4);
          const float w = part_w[sp * G + r];
          acc.x = fmaf(v.x, w, acc.x), acc.y = fmaf(v.y, w, acc.y), acc.z = fmaf(v.z, w, acc.z), acc.w = fmaf(v.w, w, acc.w);
        }
      }
    }
    const float l = head_l[r];
    const float inv = l > 0.0f ? 1.0f / l : 0.0f;
    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<const uint32_t*>(&lo), packed.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p.out + (static_cast<int64_t>(b) * p.Hq + h * G + r) * 128 + 4 * c4) = packed;
  }
  if (threadIdx.x == 0) p.tickets[DA_TICKET0 + bh] = 0;
  finish_append();
}

// The kernel needs the dynamic shared-memory attribute set once per device (this allocates nothing).
bool set_attn_smem() {
  static bool done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  if (!done[dev]) {
    if (cudaFuncSetAttribute(decode_attn_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, DA_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(decode_attn_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, DA_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(decode_attn_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DA_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(decode_attn_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DA_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(decode_attn_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             DA_SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(decode_attn_kernel<true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             DA_SMEM_BYTES) != cudaSuccess)
      return false;
    done[dev] = true;
  }
  return true;
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

bool is_dynamic(const pq_kv4_cache* c) { return c->sk_tok != nullptr && c->sv_tok != nullptr; }

pq_status check_cache(const pq_kv4_cache* c) {
  if (!c || !c->kq || !c->vq || !c->len) return PQ_ERR_INVALID_ARG;
  if ((c->sk_tok != nullptr) != (c->sv_tok != nullptr)) return PQ_ERR_INVALID_ARG;
  if (!is_dynamic(c) && (!c->s_k || !c->s_v)) return PQ_ERR_INVALID_ARG;
  if (c->B < 0 || c->Hkv <= 0 || c->Hq <= 0 || c->n_prefix < 0 || c->Tmax < 0) return PQ_ERR_INVALID_ARG;
  if (c->n_prefix > 0 && (!c->prefix_k || !c->prefix_v)) return PQ_ERR_INVALID_ARG;
  if (c->D != 128 || c->Hq % c->Hkv != 0 || c->Hq / c->Hkv > DA_ROWS || c->n_prefix > DA_MAX_PREFIX)
    return PQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(c->kq) & 15) || (reinterpret_cast<uintptr_t>(c->vq) & 15)) return PQ_ERR_ALIGN;
  if (c->n_prefix > 0 && ((reinterpret_cast<uintptr_t>(c->prefix_k) & 15) || (reinterpret_cast<uintptr_t>(c->prefix_v) & 15)))
    return PQ_ERR_ALIGN;
  return PQ_OK;
}

}  // namespace

pq_status pq_kv4_append_dyn_launch(pq_ctx* ctx, const pq_kv4_cache* c, const void* k, const void* v, int32_t T_new, int64_t ld_tok,
                                   cudaStream_t st);
pq_status pq_decode_attn_dyn_launch(pq_ctx* ctx, const pq_kv4_cache* c, const void* q, void* out, float sm_scale, void* ws,
                                    cudaStream_t st, int ticket0);

extern "C" pq_status pq_kv4_append_strided(pq_ctx* ctx, const pq_kv4_cache* cache, const void* k, const void* v,
                                           int32_t T_new, int64_t ld_tok, void* stream) {
  if (!ctx || !k || !v || T_new < 0) return PQ_ERR_INVALID_ARG;
  pq_status st = check_cache(cache);
  if (st != PQ_OK) return st;
  if (ld_tok < static_cast<int64_t>(cache->Hkv) * 128) return PQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k) & 15) || (reinterpret_cast<uintptr_t>(v) & 15) || ld_tok % 8 != 0) return PQ_ERR_ALIGN;
  if (T_new == 0 || cache->B == 0) return PQ_OK;
  if (is_dynamic(cache)) return pq_kv4_append_dyn_launch(ctx, cache, k, v, T_new, ld_tok, static_cast<cudaStream_t>(stream));
  const int64_t n_units = static_cast<int64_t>(cache->B) * T_new * cache->Hkv * 4;
  int64_t grid = (n_units + AP_THREADS - 1) / AP_THREADS;
  if (grid > 8LL * ctx->sm_count) grid = 8LL * ctx->sm_count;
  kv4_append_kernel<<<static_cast<int>(grid), AP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v), cache->kq, cache->vq, cache->s_k,
      cache->s_v, cache->len, cache->B, T_new, cache->Hkv, cache->Tmax, ld_tok, ctx->d_status, ctx->d_tickets);
  return pq_launch_status();
}

extern "C" pq_status pq_kv4_append(pq_ctx* ctx, const pq_kv4_cache* cache, const void* k, const void* v,
                                   int32_t T_new, void* stream) {
  if (!cache) return PQ_ERR_INVALID_ARG;
  return pq_kv4_append_strided(ctx, cache, k, v, T_new, static_cast<int64_t>(cache->Hkv) * 128, stream);
}

extern "C" size_t pq_decode_attn_workspace_bytes(const pq_kv4_cache* cache) {
  if (!cache || cache->B <= 0 || cache->Hkv <= 0 || cache->Hq <= 0) return 0;
  const size_t G = static_cast<size_t>(cache->Hq / cache->Hkv);
  return static_cast<size_t>(cache->B) * cache->Hkv * DA_MAX_SPLITS * G * (128 + 2) * sizeof(float);
}

namespace {
constexpr int DA_LEN_TICKET0 = PQ_N_TICKETS / 2;  // the grid-wide counter of the fused append

// k_new, v_new: null for the plain attention; else the token appended by the same launch.
pq_status decode_attn_launch(pq_ctx* ctx, const pq_kv4_cache* cache, const void* q, void* out, float sm_scale, void* ws,
                             size_t ws_bytes, void* stream, const void* k_new, const void* v_new) {
  if (!ctx || !q || !out) return PQ_ERR_INVALID_ARG;
  pq_status st = check_cache(cache);
  if (st != PQ_OK) return st;
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(out) & 7)) return PQ_ERR_ALIGN;
  if (cache->B == 0) return PQ_OK;
  if (static_cast<int64_t>(cache->B) * cache->Hkv > DA_LEN_TICKET0 - DA_TICKET0 || cache->B > DA_LEN_TICKET0 ||
      cache->Hkv > 65535)
    return PQ_ERR_SHAPE;
  if (!ws || ws_bytes < pq_decode_attn_workspace_bytes(cache)) return PQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 15) return PQ_ERR_ALIGN;
  if (is_dynamic(cache)) {
    if (k_new) return PQ_ERR_UNSUPPORTED;  // the one-launch decode step serves the static setting
    return pq_decode_attn_dyn_launch(ctx, cache, q, out, sm_scale, ws, static_cast<cudaStream_t>(stream), DA_TICKET0);
  }
  int S = choose_splits(ctx, cache);
  // With enough (sequence, head) pairs, eight splits already fill the GPU: the splits then form one
  // cluster and merge through distributed shared memory (the workspace and the tickets stay unused).
  bool cluster = static_cast<int64_t>(cache->B) * cache->Hkv * 8 >= 2LL * ctx->sm_count;
  if (cluster && S > 8) S = 8;
  // Few (sequence, head) pairs with long caches: several clusters of eight splits per pair; each merges its eight
  // partials on chip, the workspace sees one partial per cluster.
  if (!cluster && S >= 16) {
    S = S / 8 * 8;
    cluster = true;
  }
  const int n_parts = cluster ? (S < 8 ? 1 : S / 8) : S;
  const bool multi = cluster && n_parts > 1;
  const int G = cache->Hq / cache->Hkv;
  AttnParams p{};
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
  p.ws_ml = p.ws_o + static_cast<size_t>(cache->B) * cache->Hkv * n_parts * G * 128;
  p.tickets = ctx->d_tickets;
  p.status = ctx->d_status;
  p.wait_clocks = ctx->wait_clocks;
  p.sm_scale = sm_scale;
  p.B = cache->B, p.Hq = cache->Hq, p.Hkv = cache->Hkv, p.G = G, p.n_prefix = cache->n_prefix, p.Tmax = cache->Tmax;
  const bool fused = k_new != nullptr;
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.len_rw = cache->len;
  p.len_tickets = ctx->d_tickets + DA_LEN_TICKET0;
  dim3 grid(S, cache->Hkv, cache->B);
  if (!set_attn_smem()) return PQ_ERR_CUDA;
  if (cluster) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(DA_THREADS);
    cfg.dynamicSmemBytes = DA_SMEM_BYTES;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S < 8 ? S : 8;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = fused ? 2 : 1;  // the plain call gains nothing from an early placement (measured), the one-launch step does
    cudaError_t e;
    if (multi)
      e = fused ? cudaLaunchKernelEx(&cfg, decode_attn_kernel<true, true, true>, p)
                : cudaLaunchKernelEx(&cfg, decode_attn_kernel<true, false, true>, p);
    else
      e = fused ? cudaLaunchKernelEx(&cfg, decode_attn_kernel<true, true, false>, p)
                : cudaLaunchKernelEx(&cfg, decode_attn_kernel<true, false, false>, p);
    if (e != cudaSuccess) return PQ_ERR_CUDA;
    return pq_launch_status();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(DA_THREADS);
  cfg.dynamicSmemBytes = DA_SMEM_BYTES;
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = fused ? 1 : 0;
  if ((fused ? cudaLaunchKernelEx(&cfg, decode_attn_kernel<false, true, false>, p)
             : cudaLaunchKernelEx(&cfg, decode_attn_kernel<false, false, false>, p)) != cudaSuccess)
    return PQ_ERR_CUDA;
  return pq_launch_status();
}
}  // namespace

extern "C" pq_status pq_decode_attn_kv4_prefix(pq_ctx* ctx, const pq_kv4_cache* cache, const void* q, void* out,
                                               float sm_scale, void* ws, size_t ws_bytes, void* stream) {
  return decode_attn_launch(ctx, cache, q, out, sm_scale, ws, ws_bytes, stream, nullptr, nullptr);
}

extern "C" pq_status pq_kv4_append_decode_attn(pq_ctx* ctx, const pq_kv4_cache* cache, const void* k, const void* v,
                                               const void* q, void* out, float sm_scale, void* ws, size_t ws_bytes,
                                               void* stream) {
  if (!k || !v) return PQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k) & 1) || (reinterpret_cast<uintptr_t>(v) & 1)) return PQ_ERR_ALIGN;
  return decode_attn_launch(ctx, cache, q, out, sm_scale, ws, ws_bytes, stream, k, v);
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
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(out) & 7)) return PQ_ERR_ALIGN;
  if (is_dynamic(cache)) return PQ_ERR_UNSUPPORTED;
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
  AttnParams p{};
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
  p.status = nullptr;
  p.wait_clocks = PQ_DEFAULT_WAIT_CLOCKS;
  p.sm_scale = sm_scale;
  p.B = cache->B, p.Hq = cache->Hq, p.Hkv = cache->Hkv, p.G = G, p.n_prefix = cache->n_prefix, p.Tmax = cache->Tmax;
  dim3 grid(S, cache->Hkv, cache->B);
  if (!set_attn_smem()) return PQ_ERR_CUDA;
  decode_attn_kernel<false, false><<<grid, DA_THREADS, DA_SMEM_BYTES, cs>>>(p);
  return pq_launch_status();
}

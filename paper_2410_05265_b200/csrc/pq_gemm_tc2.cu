// W4A4 GEMM for prefill-shaped problems: CTA pairs on the 5th-generation tensor cores.
//
//   acc[t,n] = sum_k xq[t,k] * wq[n,k]   (exact int32),   out = bf16(acc * s_a * s_w[n])
//
// sm_100a has no 4-bit integer MMA, so packed nibbles are expanded to s8 between the TMA landing
// buffer and the operand buffer that tcgen05.mma (kind::i8) reads. The expansion is shared-memory
// store traffic, and that traffic, not the tensor pipe, is what a single CTA runs out of. Two CTAs
// of a cluster therefore share one 256 x 256 tile (cta_group::2): each CTA expands its own 128
// token rows (A) and only half of the 256 weight rows (B); the tensor cores of the pair exchange
// the B halves themselves.
//
// Roles inside each CTA (24 warps):
//   warp 0        TMA producer: packed A [128 x 64 B] and packed B half [128 x 64 B] per 128-wide
//                 K block into a ring of landing buffers (own shared memory, own barriers).
//   warps 8..23   unpack, in four groups that take K blocks in turn so that one group's barrier
//                 hops and fence latency overlap the other groups' stores. A 16-byte packed chunk
//                 (32 codes) becomes two 16-byte s8 chunks holding 16*code: `w & 0xF0F0F0F0` is
//                 16*hi, `(w << 4) & 0xF0F0F0F0` is 16*lo. Even-position codes go to one chunk,
//                 odd-position codes to the next; A and B use the same permutation of k inside a
//                 32-element group, so the dot product is unchanged. Chunks land in the
//                 128-byte-swizzled K-major layout of the MMA descriptors. When a group is done
//                 with a stage, every warp arrives on the stage's "full" barrier of the leader CTA.
//   warp 1        (leader CTA only) MMA issuer: four 256x256x32 MMAs per K block into one of two
//                 256-column TMEM accumulators; tcgen05.commit multicasts "stage free" and
//                 "accumulator ready" to both CTAs. Warp 1 of each CTA owns its TMEM allocation.
//   warps 4..7    epilogue: tcgen05.ld the CTA's 128 x 256 accumulator half, shift out the 16*16
//                 factor exactly, scale, round to bf16, stage 32 x 64 blocks in swizzled shared
//                 memory and write them with TMA stores (clipped at the matrix edge).
//
// A8 (the W4A8 precision, Sec. 5.1): the token operand already is s8. A second producer lane
// (warp 2) copies its 128 x 128-byte box straight into the operand stage with a 128-byte-swizzling
// tensor map; only the weight rows go through the landing ring and the unpack warps, which then
// write the codes in their natural order (low nibble first) to match the untouched token bytes.
// The accumulator carries one factor 16 instead of two.
//
// Every mbarrier wait is bounded; when one runs out the CTA raises an abort flag, every role of
// the CTA drains, the peer's waits run out in turn, and PQ_ERR_TIMEOUT is reported.
#include "pq_gemm_pair.cuh"

namespace {

using namespace pq_pair;

constexpr int ROWS = BM_CTA + BN_CTA;       // operand rows per CTA per stage
#ifndef PQ_GEMM_N_PK
#define PQ_GEMM_N_PK 4
#endif
#ifndef PQ_GEMM_N_S8
#define PQ_GEMM_N_S8 4
#endif
#ifndef PQ_GEMM_EPI_BUFS
#define PQ_GEMM_EPI_BUFS 1
#endif
#ifndef PQ_GEMM_UNPACK_WARPS
#define PQ_GEMM_UNPACK_WARPS 16
#endif
#ifndef PQ_GEMM_GROUPS
#define PQ_GEMM_GROUPS 4
#endif
constexpr int N_PK = PQ_GEMM_N_PK;          // landing-buffer stages
constexpr int N_S8 = PQ_GEMM_N_S8;          // operand-buffer stages
constexpr int EPI_BUFS = PQ_GEMM_EPI_BUFS;  // staging buffers per epilogue warp
constexpr int PK_STAGE = ROWS * PK_ROW;     // 16 KB
constexpr int S8_STAGE = ROWS * BK;         // 32 KB
constexpr int S8_A = BM_CTA * BK;           // the A part of an operand stage
constexpr int N_UNPACK_WARPS = PQ_GEMM_UNPACK_WARPS;
constexpr int N_GROUPS = PQ_GEMM_GROUPS;
constexpr int GROUP_WARPS = N_UNPACK_WARPS / N_GROUPS;
// A ring slot is always served by the same group, so no group can get a whole phase ahead of a
// barrier it waits on (a parity wait cannot tell phase k from phase k+2).
static_assert(N_PK % N_GROUPS == 0 && N_S8 % N_GROUPS == 0, "ring depths must be multiples of the group count");
static_assert(N_UNPACK_WARPS % N_GROUPS == 0, "equal groups");
constexpr int GROUP_THREADS = GROUP_WARPS * 32;
constexpr int UNPACK_WARP0 = 8, EPI_WARP0 = 4;
constexpr int N_THREADS = (UNPACK_WARP0 + N_UNPACK_WARPS) * 32;
constexpr int TMEM_COLS = 512;              // two 256-column accumulators
constexpr int EPI_BYTES = 4 * EPI_BUFS * EPI_BUF;
constexpr int SCALE_BYTES = 4 * BN * 4;     // per-warp copy of s_a * s_w[n0 .. n0+255]
constexpr int ZW_BYTES = 4 * BN * 4;        // per-warp copy of (z - 8) * wsum[n0 .. n0+255] (zero-point correction)

struct __align__(8) Barriers {
  uint64_t pk_full[N_PK], pk_empty[N_PK];
  uint64_t s8_full[N_S8];   // waited on in the leader CTA only: 2 * GROUP_WARPS arrivals
  uint64_t s8_empty[N_S8];  // one arrival per phase from the multicast tcgen05.commit
  uint64_t acc_full[2];     // likewise
  uint64_t acc_empty[2];    // leader CTA only: 4 epilogue warps of each CTA
  uint64_t drain;
  uint64_t a_full[N_S8];    // A8 only: the token box of an operand stage has landed (own CTA)
  uint32_t tmem_base;
  volatile int abort_flag;
};

constexpr size_t SMEM_BYTES =
    1024 /*alignment slack*/ + N_S8 * S8_STAGE + N_PK * PK_STAGE + EPI_BYTES + SCALE_BYTES + ZW_BYTES + sizeof(Barriers);
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

// D[tmem of both CTAs] (+)= A[smem of both CTAs] * B[smem halves of both CTAs], issued by one thread
// of the leader CTA.
__device__ __forceinline__ void mma2_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
template <bool A8, bool ZP>
__global__ void __launch_bounds__(N_THREADS, 1)
    gemm_w4a4_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                          const __grid_constant__ CUtensorMap tmap_out, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* s8_buf = smem;                                   // N_S8 stages: A rows then B rows, 1024-aligned
  uint8_t* pk_buf = s8_buf + N_S8 * S8_STAGE;               // N_PK stages: packed A rows then packed B rows
  uint8_t* epi_buf = pk_buf + N_PK * PK_STAGE;              // 4 warps x 2 buffers, 1024-aligned
  float* scale_buf = reinterpret_cast<float*>(epi_buf + EPI_BYTES);
  int32_t* zw_buf = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(scale_buf) + SCALE_BYTES);
  Barriers* bars = reinterpret_cast<Barriers*>(reinterpret_cast<uint8_t*>(zw_buf) + ZW_BYTES);

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // operands and output may belong to the previous kernel
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_tiles = p.tiles_m * p.tiles_n;
  const int n_kb = (p.K + BK - 1) / BK;
  const int my_tiles = pair < n_tiles ? (n_tiles - pair + n_pairs - 1) / n_pairs : 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < N_PK; ++i) {
      pq::mbar_init(&bars->pk_full[i], 1);
      pq::mbar_init(&bars->pk_empty[i], GROUP_WARPS);
    }
    for (int i = 0; i < N_S8; ++i) {
      pq::mbar_init(&bars->s8_full[i], 2 * GROUP_WARPS);
      pq::mbar_init(&bars->s8_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      pq::mbar_init(&bars->acc_full[i], 1);
      pq::mbar_init(&bars->acc_empty[i], 8);
    }
    for (int i = 0; i < N_S8; ++i) pq::mbar_init(&bars->a_full[i], 1);
    pq::mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    pq::mbar_fence_init();
    pq::fence_proxy_async_smem();
    pq::tma_prefetch_desc(&tmap_a);
    pq::tma_prefetch_desc(&tmap_b);
    pq::tma_prefetch_desc(&tmap_out);
  }
  if (warp == 1) {
    tmem_alloc2(&bars->tmem_base, TMEM_COLS);
    tmem_relinquish2();
  }
  pq::tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything arrives on them
  pq::tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  uint32_t loads_issued = 0;  // producer lanes: stages whose copies were started

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
        const int m_row = (tile % p.tiles_m) * (2 * BM_CTA) + rank * BM_CTA;
        const int n_row = (tile / p.tiles_m) * BN + rank * BN_CTA;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % N_PK, ph = (it / N_PK) & 1;
          if (!wait_bar(&bars->pk_empty[s], ph ^ 1, abort_flag, p.wait_clocks)) {
            ok = false;
            break;
          }
          if (A8) {
            pq::mbar_arrive_expect_tx(&bars->pk_full[s], BN_CTA * PK_ROW);
            pq::tma_load_2d(pk_buf + s * PK_STAGE, &tmap_b, kb * PK_ROW, n_row, &bars->pk_full[s]);
          } else {
            pq::mbar_arrive_expect_tx(&bars->pk_full[s], PK_STAGE);
            pq::tma_load_2d(pk_buf + s * PK_STAGE, &tmap_a, kb * PK_ROW, m_row, &bars->pk_full[s]);
            pq::tma_load_2d(pk_buf + s * PK_STAGE + BM_CTA * PK_ROW, &tmap_b, kb * PK_ROW, n_row, &bars->pk_full[s]);
          }
        }
      }
      loads_issued = it;
      if (!ok) {
        bars->abort_flag = 1;
        pq::report(p.status, PQ_ERR_TIMEOUT);
        // let the copies this thread started land before the CTA can exit
        const uint32_t first = it > N_PK ? it - N_PK : 0;
        for (uint32_t j = first; j < it; ++j) pq::mbar_wait(&bars->pk_full[j % N_PK], (j / N_PK) & 1);
      }
    }
  } else if (A8 && warp == 2) {
    // ------------------------------------------------------------------ token-operand producer (A8)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
        const int m_row = (tile % p.tiles_m) * (2 * BM_CTA) + rank * BM_CTA;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % N_S8, ph = (it / N_S8) & 1;
          if (!wait_bar(&bars->s8_empty[s], ph ^ 1, abort_flag, p.wait_clocks)) {
            ok = false;
            break;
          }
          pq::mbar_arrive_expect_tx(&bars->a_full[s], S8_A);
          pq::tma_load_2d(s8_buf + s * S8_STAGE, &tmap_a, kb * BK, m_row, &bars->a_full[s]);
        }
      }
      loads_issued = it;
      if (!ok) {
        bars->abort_flag = 1;
        pq::report(p.status, PQ_ERR_TIMEOUT);
        const uint32_t first = it > N_S8 ? it - N_S8 : 0;
        for (uint32_t j = first; j < it; ++j) pq::mbar_wait(&bars->a_full[j % N_S8], (j / N_S8) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = pq::umma_idesc_s8(2 * BM_CTA, BN);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++tcount) {
        const uint32_t ab = tcount & 1, aph = (tcount >> 1) & 1;
        if (!wait_bar(&bars->acc_empty[ab], aph ^ 1, abort_flag, p.wait_clocks)) {
          ok = false;
          break;
        }
        pq::tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * BN;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % N_S8, ph = (it / N_S8) & 1;
          if (!wait_bar(&bars->s8_full[s], ph, abort_flag, p.wait_clocks)) {
            ok = false;
            break;
          }
          pq::tc_fence_after();
          const uint32_t a_addr = pq::smem_u32(s8_buf + s * S8_STAGE);
          const uint32_t b_addr = a_addr + S8_A;
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            mma2_i8_ss(d_tmem, pq::umma_desc_sw128(a_addr + kk * 32), pq::umma_desc_sw128(b_addr + kk * 32), idesc,
                       (kb | kk) != 0 ? 1u : 0u);
          }
          mma2_commit_both(&bars->s8_empty[s]);  // both CTAs may refill the stage once these MMAs have read it
        }
        if (ok) mma2_commit_both(&bars->acc_full[ab]);
      }
      if (!ok) {
        bars->abort_flag = 1;
        pq::report(p.status, PQ_ERR_TIMEOUT);
      }
      // whatever was issued has finished before either CTA releases its tensor memory
      mma2_commit_both(&bars->drain);
    }
    if (lane == 0) pq::mbar_wait(&bars->drain, 0);
  } else if (warp >= UNPACK_WARP0) {
    // ------------------------------------------------------------------ unpack warps
    const int group = (warp - UNPACK_WARP0) / GROUP_WARPS;
    const int gt = (warp - UNPACK_WARP0) % GROUP_WARPS * 32 + lane;
    const uint32_t total = static_cast<uint32_t>(my_tiles) * n_kb;
    bool ok = true;
    for (uint32_t it = group; it < total; it += N_GROUPS) {
      const uint32_t ps = it % N_PK, pph = (it / N_PK) & 1;
      const uint32_t ss = it % N_S8, sph = (it / N_S8) & 1;
      const bool stuck =
          !wait_bar(&bars->pk_full[ps], pph, abort_flag, p.wait_clocks) || !wait_bar(&bars->s8_empty[ss], sph ^ 1, abort_flag, p.wait_clocks);
      if (__any_sync(0xffffffffu, stuck)) {  // warp-uniform decision
        ok = false;
        break;
      }
      const uint8_t* src = pk_buf + ps * PK_STAGE;
      uint8_t* dst = s8_buf + ss * S8_STAGE + (A8 ? S8_A : 0);  // A8: only the weight rows are expanded
      constexpr int UNITS = (A8 ? BN_CTA : ROWS) * 4;  // one unit = one 16-byte packed chunk
#pragma unroll
      for (int i = 0; i < UNITS / GROUP_THREADS; ++i) {
        const int unit = i * GROUP_THREADS + gt;
        const int row = unit >> 2, j = unit & 3;
        const uint4 w = *reinterpret_cast<const uint4*>(src + row * PK_ROW + j * 16);
        uint4 lo, hi;
        lo.x = pq::nib_lo_x16(w.x), lo.y = pq::nib_lo_x16(w.y), lo.z = pq::nib_lo_x16(w.z), lo.w = pq::nib_lo_x16(w.w);
        hi.x = pq::nib_hi_x16(w.x), hi.y = pq::nib_hi_x16(w.y), hi.z = pq::nib_hi_x16(w.z), hi.w = pq::nib_hi_x16(w.w);
        if (A8) {
          // natural order: byte 2i of a word pair is the low nibble of packed byte i, byte 2i+1 its high nibble
          const uint4 c0 = make_uint4(__byte_perm(lo.x, hi.x, 0x5140), __byte_perm(lo.x, hi.x, 0x7362),
                                      __byte_perm(lo.y, hi.y, 0x5140), __byte_perm(lo.y, hi.y, 0x7362));
          const uint4 c1 = make_uint4(__byte_perm(lo.z, hi.z, 0x5140), __byte_perm(lo.z, hi.z, 0x7362),
                                      __byte_perm(lo.w, hi.w, 0x5140), __byte_perm(lo.w, hi.w, 0x7362));
          lo = c0, hi = c1;
        }
        uint8_t* drow = dst + row * BK;
        const int sw = row & 7;
        *reinterpret_cast<uint4*>(drow + (((2 * j) ^ sw) << 4)) = lo;
        *reinterpret_cast<uint4*>(drow + (((2 * j + 1) ^ sw) << 4)) = hi;
      }
      pq::fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's async proxy
      if (A8) {  // the stage is complete only with this CTA's token box in place
        const bool late = !wait_bar(&bars->a_full[ss], sph, abort_flag, p.wait_clocks);
        if (__any_sync(0xffffffffu, late)) {
          ok = false;
          break;
        }
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive_cluster(map_to_cta(&bars->s8_full[ss], 0));
        pq::mbar_arrive(&bars->pk_empty[ps]);
      }
    }
    if (!ok && lane == 0) {
      bars->abort_flag = 1;
      pq::report(p.status, PQ_ERR_TIMEOUT);
    }
  } else if (warp >= EPI_WARP0) {
    // ------------------------------------------------------------------ epilogue warps
    constexpr int SHIFT = A8 ? 4 : 8;  // the factors 16 the expanded codes carry
    const int q = warp & 3;  // TMEM lane quarter this warp may access
    const float s_a = p.s_row ? 1.0f : __ldg(p.s_a);
    uint8_t* my_buf = epi_buf + q * EPI_BUFS * EPI_BUF;
    float* my_scale = scale_buf + q * BN;
    int32_t* my_zw = zw_buf + q * BN;
    const int zp8 = ZP ? __ldg(p.zp) - 8 : 0;
    uint32_t tcount = 0, n_store = 0;
    bool ok = true;
    for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++tcount) {
      const int m0 = (tile % p.tiles_m) * (2 * BM_CTA) + rank * BM_CTA + q * 32;
      const int n0 = (tile / p.tiles_m) * BN;
      const uint32_t ab = tcount & 1, aph = (tcount >> 1) & 1;
      fill_tile_scales<ZP>(p, n0, lane, s_a, zp8, my_scale, my_zw);
      const bool stuck = !wait_bar(&bars->acc_full[ab], aph, abort_flag, p.wait_clocks);
      if (__any_sync(0xffffffffu, stuck)) {  // warp-uniform: the TMEM loads below are warp-collective
        ok = false;
        break;
      }
      pq::tc_fence_after();
      const float rs = p.s_row ? (m0 + lane < p.M ? __ldg(p.s_row + m0 + lane) : 0.0f) : 1.0f;  // this lane's token step
      const uint32_t taddr = tmem_base + ab * BN + (static_cast<uint32_t>(q * 32) << 16);
      epilogue_tile<SHIFT, ZP, EPI_BUFS>(p, &tmap_out, taddr, m0, n0, lane, rs, my_scale, my_zw, my_buf, n_store,
                                         map_to_cta(&bars->acc_empty[ab], 0));
    }
    if (lane == 0) bulk_wait_all();
    if (!ok && lane == 0) {
      bars->abort_flag = 1;
      pq::report(p.status, PQ_ERR_TIMEOUT);
    }
  }

  pq::tc_fence_before();
  __syncthreads();
  if (bars->abort_flag) {
    // a role gave up: copies that nobody consumed must still have landed before the CTA may exit (they only wait
    // for memory, hence the generous bound)
    if (warp == 0 && lane == 0)
      for (uint32_t j = loads_issued > N_PK ? loads_issued - N_PK : 0; j < loads_issued; ++j) pq::mbar_wait(&bars->pk_full[j % N_PK], (j / N_PK) & 1);
    if (A8 && warp == 2 && lane == 0)
      for (uint32_t j = loads_issued > N_S8 ? loads_issued - N_S8 : 0; j < loads_issued; ++j) pq::mbar_wait(&bars->a_full[j % N_S8], (j / N_S8) & 1);
    __syncthreads();
  }
  cluster_sync_all();  // neither CTA frees tensor memory or exits while the pair may still touch it
  if (warp == 1) {
    pq::tc_fence_after();
    tmem_dealloc2(tmem_base, TMEM_COLS);
  }
}

}  // namespace

// Launches the CTA-pair kernel on rows [0, M) of xq/out (the caller has already applied row_begin).
// a8: xq holds one s8 code per element ([M, K] bytes) instead of packed nibbles.
// s_row: per-token steps (then s_a is ignored), or null.
pq_status pq_gemm_pair_launch(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w,
                              void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg,
                              cudaStream_t st, bool a8, const float* s_row, const int32_t* zp, const int32_t* wsum) {
  CUtensorMap ta, tb, to;
  if (!(a8 ? make_s8_map(ctx, &ta, xq, M, K) : make_packed_map(ctx, &ta, xq, M, K / 2, BM_CTA)) ||
      !make_packed_map(ctx, &tb, wq, N, K / 2, BN_CTA))
    return PQ_ERR_CUDA;
  GemmParams p;
  p.tma_store = (ldo % 8 == 0) && ((reinterpret_cast<uintptr_t>(out) & 15) == 0);
  if (p.tma_store) {
    if (!make_out_map(ctx, &to, out, M, N, ldo)) return PQ_ERR_CUDA;
  } else {
    to = ta;  // never dereferenced
  }
  p.s_row = s_row;
  p.zp = zp;
  p.wsum = wsum;
  p.s_a = s_a;
  p.s_w = s_w;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.acc_dbg = acc_dbg;
  p.status = ctx->d_status;
  p.wait_clocks = ctx->wait_clocks;
  p.ldo = ldo;
  p.M = static_cast<int>(M);
  p.N = static_cast<int>(N);
  p.K = static_cast<int>(K);
  p.tiles_m = static_cast<int>((M + 2 * BM_CTA - 1) / (2 * BM_CTA));
  p.tiles_n = static_cast<int>((N + BN - 1) / BN);
  static bool attr_set[64] = {};  // the attribute belongs to the device's copy of the kernel: once per device
  if (ctx->device < 0 || ctx->device >= 64) return PQ_ERR_UNSUPPORTED;
  if (!attr_set[ctx->device]) {
    if (cudaFuncSetAttribute(gemm_w4a4_pair_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(SMEM_BYTES)) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w4a4_pair_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(SMEM_BYTES)) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w4a4_pair_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(SMEM_BYTES)) != cudaSuccess)
      return PQ_ERR_CUDA;
    attr_set[ctx->device] = true;
  }
  const int n_tiles = p.tiles_m * p.tiles_n;
  const int max_pairs = ctx->sm_count / 2;
  const int pairs = n_tiles < max_pairs ? n_tiles : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(N_THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // the kernel may be launched while its predecessor drains; it waits for it on the device before it
  // reads or writes anything (griddepcontrol.wait at its top), which hides the launch itself
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (zp && (a8 || !wsum)) return PQ_ERR_INVALID_ARG;
  if ((zp   ? cudaLaunchKernelEx(&cfg, gemm_w4a4_pair_kernel<false, true>, ta, tb, to, p)
       : a8 ? cudaLaunchKernelEx(&cfg, gemm_w4a4_pair_kernel<true, false>, ta, tb, to, p)
            : cudaLaunchKernelEx(&cfg, gemm_w4a4_pair_kernel<false, false>, ta, tb, to, p)) != cudaSuccess)
    return PQ_ERR_CUDA;
  return pq_launch_status();
}

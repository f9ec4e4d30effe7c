// W4A4 GEMM for prefill-shaped problems: CTA pairs, token operand fed from tensor memory.
//
//   acc[t,n] = sum_k xq[t,k] * wq[n,k]   (exact int32),   out = bf16(acc * s_a * s_w[n])
//
// Same pair design as pq_gemm_tc2.cu (cta_group::2, 256 x 256 tile, packed nibbles expanded to
// 16*code as s8 on the way to the MMA), with one change that removes a third of the shared-memory
// traffic and halves the operand ring: the A operand (token rows) never goes back to shared
// memory. Each unpack thread owns one token row, reads its 64 packed bytes of a K block from the
// landing buffer (64-byte-swizzled by TMA, so the row-per-thread reads are conflict-free), expands
// them in registers and writes the 128 s8 bytes to its lane of tensor memory with tcgen05.st; the
// MMA takes A from TMEM ([d], [a], b_desc form). Only the weight rows (B) are expanded into the
// 128-byte-swizzled shared-memory layout.
//
// Tensor memory (512 columns): columns 0..255 the accumulator (one buffer: the epilogue of a tile
// runs while the unpack warps fill up to eight K blocks of the next tile), columns 256..511 a ring
// of eight A slots of 32 columns (128 K bytes per lane).
//
// Roles inside each CTA (24 warps):
//   warp 0        TMA producer: packed A [128 x 64 B, 64-byte swizzle] and packed B half [128 x 64 B].
//   warps 8..23   unpack, four groups of four warps (one warp per TMEM lane quarter); group g serves
//                 ring slots g and g+4, so it can work one K block ahead of the MMA's release of its
//                 other slot. A 16-byte packed chunk (32 codes) becomes 32 s8 bytes: even-position
//                 codes then odd-position codes, the same order for A (registers -> TMEM columns) and
//                 B (two 16-byte chunks in shared memory), so the dot product is unchanged.
//   warp 1        (leader CTA only) MMA issuer; warp 1 of each CTA owns its TMEM allocation.
//   warps 4..7    epilogue (as in pq_gemm_tc2.cu).
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
#define PQ_GEMM_N_S8 8
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
constexpr int S8_STAGE = BN_CTA * BK;       // 16 KB: weight rows only
constexpr int A_COL0 = 256;                 // first TMEM column of the A ring
constexpr int A_SLOT_COLS = BK / 4;         // 32 columns = 128 K bytes per lane
constexpr int N_UNPACK_WARPS = PQ_GEMM_UNPACK_WARPS;
constexpr int N_GROUPS = PQ_GEMM_GROUPS;
constexpr int GROUP_WARPS = N_UNPACK_WARPS / N_GROUPS;
// A ring slot is always served by the same group, so no group can get a whole phase ahead of a
// barrier it waits on (a parity wait cannot tell phase k from phase k+2).
static_assert(N_PK % N_GROUPS == 0 && N_S8 % N_GROUPS == 0, "ring depths must be multiples of the group count");
static_assert(N_UNPACK_WARPS % N_GROUPS == 0, "equal groups");
static_assert(N_UNPACK_WARPS / N_GROUPS == 4, "one warp per TMEM lane quarter in every group");
static_assert(A_COL0 + N_S8 * A_SLOT_COLS <= 512, "tensor memory budget");
constexpr int GROUP_THREADS = GROUP_WARPS * 32;
constexpr int UNPACK_WARP0 = 8, EPI_WARP0 = 4;
constexpr int N_THREADS = (UNPACK_WARP0 + N_UNPACK_WARPS) * 32;
constexpr int TMEM_COLS = 512;              // one 256-column accumulator + the A ring
constexpr int EPI_BYTES = 4 * EPI_BUFS * EPI_BUF;
constexpr int SCALE_BYTES = 4 * BN * 4;     // per-warp copy of s_a * s_w[n0 .. n0+255]
constexpr int ZW_BYTES = 4 * BN * 4;        // per-warp copy of (z - 8) * wsum[n0 .. n0+255] (zero-point correction)

struct __align__(8) Barriers {
  uint64_t pk_full[N_PK], pk_empty[N_PK];
  uint64_t s8_full[N_S8];   // waited on in the leader CTA only: 2 * GROUP_WARPS arrivals
  uint64_t s8_empty[N_S8];  // one arrival per phase from the multicast tcgen05.commit
  uint64_t acc_full[1];     // likewise
  uint64_t acc_empty[1];    // leader CTA only: 4 epilogue warps of each CTA
  uint64_t drain;
  uint32_t tmem_base;
  volatile int abort_flag;
};

constexpr size_t SMEM_BYTES =
    1024 /*alignment slack*/ + N_S8 * S8_STAGE + N_PK * PK_STAGE + EPI_BYTES + SCALE_BYTES + ZW_BYTES + sizeof(Barriers);
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

// D[tmem of both CTAs] (+)= A[tmem of both CTAs] * B[smem halves of both CTAs], issued by one thread
// of the leader CTA.
__device__ __forceinline__ void mma2_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp writes lane (base+i).
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
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <bool ZP>
__global__ void __launch_bounds__(N_THREADS, 1)
    gemm_w4a4_pair_ts_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                          const __grid_constant__ CUtensorMap tmap_out, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* s8_buf = smem;                                   // N_S8 stages of expanded weight rows, 1024-aligned
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
    pq::mbar_init(&bars->acc_full[0], 1);
    pq::mbar_init(&bars->acc_empty[0], 8);
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
          pq::mbar_arrive_expect_tx(&bars->pk_full[s], PK_STAGE);
          pq::tma_load_2d(pk_buf + s * PK_STAGE, &tmap_a, kb * PK_ROW, m_row, &bars->pk_full[s]);
          pq::tma_load_2d(pk_buf + s * PK_STAGE + BM_CTA * PK_ROW, &tmap_b, kb * PK_ROW, n_row, &bars->pk_full[s]);
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
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = pq::umma_idesc_s8(2 * BM_CTA, BN);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++tcount) {
        if (!wait_bar(&bars->acc_empty[0], (tcount & 1) ^ 1, abort_flag, p.wait_clocks)) {  // the epilogue has read the last tile
          ok = false;
          break;
        }
        pq::tc_fence_after();
        const uint32_t d_tmem = tmem_base;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % N_S8, ph = (it / N_S8) & 1;
          if (!wait_bar(&bars->s8_full[s], ph, abort_flag, p.wait_clocks)) {
            ok = false;
            break;
          }
          pq::tc_fence_after();
          const uint32_t a_tmem = tmem_base + A_COL0 + s * A_SLOT_COLS;
          const uint32_t b_addr = pq::smem_u32(s8_buf + s * S8_STAGE);
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            mma2_i8_ts(d_tmem, a_tmem + kk * 8, pq::umma_desc_sw128(b_addr + kk * 32), idesc, (kb | kk) != 0 ? 1u : 0u);
          }
          mma2_commit_both(&bars->s8_empty[s]);  // both CTAs may refill the stage once these MMAs have read it
        }
        if (ok) mma2_commit_both(&bars->acc_full[0]);
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
      // ---- A: this thread's token row, 64 packed bytes -> 128 s8 bytes -> its TMEM lane ------------
      {
        const int q = warp & 3, arow = q * 32 + lane;
        const uint8_t* arow_p = src + arow * PK_ROW;
        const int sx = (arow >> 1) & 3;  // 64-byte swizzle of the landing buffer
        uint32_t ar[32];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 w = *reinterpret_cast<const uint4*>(arow_p + ((j ^ sx) << 4));
          ar[8 * j + 0] = pq::nib_lo_x16(w.x), ar[8 * j + 1] = pq::nib_lo_x16(w.y);
          ar[8 * j + 2] = pq::nib_lo_x16(w.z), ar[8 * j + 3] = pq::nib_lo_x16(w.w);
          ar[8 * j + 4] = pq::nib_hi_x16(w.x), ar[8 * j + 5] = pq::nib_hi_x16(w.y);
          ar[8 * j + 6] = pq::nib_hi_x16(w.z), ar[8 * j + 7] = pq::nib_hi_x16(w.w);
        }
        tmem_st_32x32(tmem_base + A_COL0 + ss * A_SLOT_COLS + (static_cast<uint32_t>(q * 32) << 16), ar);
      }
      // ---- B: the CTA's 128 weight rows into the swizzled operand stage -------------------------------
      const uint8_t* bsrc = src + BM_CTA * PK_ROW;
      uint8_t* dst = s8_buf + ss * S8_STAGE;
      constexpr int UNITS = BN_CTA * 4;  // one unit = one 16-byte packed chunk
#pragma unroll
      for (int i = 0; i < UNITS / GROUP_THREADS; ++i) {
        const int unit = i * GROUP_THREADS + gt;
        const int row = unit >> 2, j = unit & 3;
        const uint4 w = *reinterpret_cast<const uint4*>(bsrc + row * PK_ROW + j * 16);
        uint4 lo, hi;
        lo.x = pq::nib_lo_x16(w.x), lo.y = pq::nib_lo_x16(w.y), lo.z = pq::nib_lo_x16(w.z), lo.w = pq::nib_lo_x16(w.w);
        hi.x = pq::nib_hi_x16(w.x), hi.y = pq::nib_hi_x16(w.y), hi.z = pq::nib_hi_x16(w.z), hi.w = pq::nib_hi_x16(w.w);
        uint8_t* drow = dst + row * BK;
        const int sw = row & 7;
        *reinterpret_cast<uint4*>(drow + (((2 * j) ^ sw) << 4)) = lo;
        *reinterpret_cast<uint4*>(drow + (((2 * j + 1) ^ sw) << 4)) = hi;
      }
      tmem_st_wait();         // the TMEM lane is written ...
      pq::tc_fence_before();  // ... and ordered before the arrival below
      pq::fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's async proxy
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
      const uint32_t aph = tcount & 1;
      fill_tile_scales<ZP>(p, n0, lane, s_a, zp8, my_scale, my_zw);
      const bool stuck = !wait_bar(&bars->acc_full[0], aph, abort_flag, p.wait_clocks);
      if (__any_sync(0xffffffffu, stuck)) {  // warp-uniform: the TMEM loads below are warp-collective
        ok = false;
        break;
      }
      pq::tc_fence_after();
      const float rs = p.s_row ? (m0 + lane < p.M ? __ldg(p.s_row + m0 + lane) : 0.0f) : 1.0f;  // this lane's token step
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
      epilogue_tile<8, ZP, EPI_BUFS>(p, &tmap_out, taddr, m0, n0, lane, rs, my_scale, my_zw, my_buf, n_store,
                                     map_to_cta(&bars->acc_empty[0], 0));
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
    __syncthreads();
  }
  cluster_sync_all();  // neither CTA frees tensor memory or exits while the pair may still touch it
  if (warp == 1) {
    pq::tc_fence_after();
    tmem_dealloc2(tmem_base, TMEM_COLS);
  }
}

}  // namespace

// Launches the CTA-pair kernel with the token operand in tensor memory on rows [0, M) of xq/out (the caller has already
// applied row_begin). s_row: per-token steps (then s_a is ignored), or null. zp, wsum: the zero point of Eq. 1 and the
// weight code sums, or null.
pq_status pq_gemm_pair_ts_launch(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w,
                                 void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg,
                                 cudaStream_t st, const float* s_row, const int32_t* zp, const int32_t* wsum) {
  if (zp && !wsum) return PQ_ERR_INVALID_ARG;
  CUtensorMap ta, tb, to;
  if (!make_packed_map(ctx, &ta, xq, M, K / 2, BM_CTA, CU_TENSOR_MAP_SWIZZLE_64B) ||
      !make_packed_map(ctx, &tb, wq, N, K / 2, BN_CTA, CU_TENSOR_MAP_SWIZZLE_NONE))
    return PQ_ERR_CUDA;
  GemmParams p;
  p.tma_store = (ldo % 8 == 0) && ((reinterpret_cast<uintptr_t>(out) & 15) == 0);
  if (p.tma_store) {
    if (!make_out_map(ctx, &to, out, M, N, ldo)) return PQ_ERR_CUDA;
  } else {
    to = ta;  // never dereferenced
  }
  p.s_a = s_a;
  p.s_w = s_w;
  p.s_row = s_row;
  p.zp = zp;
  p.wsum = wsum;
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
    if (cudaFuncSetAttribute(gemm_w4a4_pair_ts_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(SMEM_BYTES)) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w4a4_pair_ts_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
  if ((zp ? cudaLaunchKernelEx(&cfg, gemm_w4a4_pair_ts_kernel<true>, ta, tb, to, p)
          : cudaLaunchKernelEx(&cfg, gemm_w4a4_pair_ts_kernel<false>, ta, tb, to, p)) != cudaSuccess)
    return PQ_ERR_CUDA;
  return pq_launch_status();
}

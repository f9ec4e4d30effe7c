// W4A4 GEMM for prefill-shaped problems on the 5th-generation tensor cores.
//
//   acc[t,n] = sum_k xq[t,k] * wq[n,k]   (exact int32),   out = bf16(acc * s_a * s_w[n])
//
// sm_100a has no 4-bit integer MMA, so the packed nibbles are expanded to s8 on the way from the
// TMA landing buffer to the operand buffer that tcgen05.mma (kind::i8) reads:
//
//   warp 0        TMA producer: packed A tile [128 x 64 B] and B tile [256 x 64 B] per 128-wide
//                 K block into a ring of landing buffers.
//   warps 8..15   unpack: each 16-byte packed chunk (32 codes) becomes two 16-byte chunks of s8
//                 holding 16*code (the high nibble of a byte already is 16*hi as an s8, the low
//                 nibble shifted left by 4 is 16*lo). Even-position codes go to one chunk and
//                 odd-position codes to the next; A and B use the same permutation of k inside a
//                 32-element group, so the dot product is unchanged. Chunks are written in the
//                 128-byte-swizzled K-major layout the MMA descriptors expect.
//   warp 1        MMA issuer: four 128x256x32 MMAs per K block, accumulating in TMEM; owns TMEM.
//   warps 4..7    epilogue: tcgen05.ld the accumulator (two buffers, so the next tile's main loop
//                 overlaps), shift out the 16*16 factor exactly, scale, round to bf16, store.
//
// Persistent CTAs walk the tile list with a fixed stride. Every mbarrier wait is bounded: when
// one runs out the CTA raises an abort flag, every role drains and the kernel reports
// PQ_ERR_TIMEOUT through the status word instead of hanging.
#include "pq_common.cuh"

namespace {

constexpr int BM = 128;          // tile rows (tokens)
constexpr int BN = 256;          // tile columns (output channels)
constexpr int BK = 128;          // K elements per pipeline stage (64 packed bytes per row)
constexpr int PK_ROW = BK / 2;   // packed bytes per row per stage
constexpr int N_PK = 3;          // landing-buffer stages
constexpr int N_S8 = 3;          // operand-buffer stages
constexpr int PK_A = BM * PK_ROW, PK_B = BN * PK_ROW, PK_STAGE = PK_A + PK_B;  // 24 KB
constexpr int S8_A = BM * BK, S8_B = BN * BK, S8_STAGE = S8_A + S8_B;          // 48 KB
constexpr int N_UNPACK_WARPS = 8;
constexpr int N_THREADS = 512;
constexpr int UNPACK_WARP0 = 8, EPI_WARP0 = 4;
constexpr int TMEM_COLS = 512;   // two 256-column accumulators

struct __align__(8) Barriers {
  uint64_t pk_full[N_PK], pk_empty[N_PK];
  uint64_t s8_full[N_S8], s8_empty[N_S8];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  volatile int abort_flag;
};

constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + N_S8 * S8_STAGE + N_PK * PK_STAGE + sizeof(Barriers);

struct GemmParams {
  const float* s_a;
  const float* s_w;
  __nv_bfloat16* out;
  int32_t* acc_dbg;
  int32_t* status;
  int64_t ldo;
  int M, N, K;
  int tiles_m, tiles_n;
};

__global__ void __launch_bounds__(N_THREADS, 1)
    gemm_w4a4_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                        const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* s8_buf = smem;                         // N_S8 stages, each 1024-aligned: A tile then B tile
  uint8_t* pk_buf = smem + N_S8 * S8_STAGE;       // N_PK stages: packed A rows then packed B rows
  Barriers* bars = reinterpret_cast<Barriers*>(pk_buf + N_PK * PK_STAGE);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = p.tiles_m * p.tiles_n;
  const int n_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < N_PK; ++i) {
      pq::mbar_init(&bars->pk_full[i], 1);
      pq::mbar_init(&bars->pk_empty[i], N_UNPACK_WARPS);
    }
    for (int i = 0; i < N_S8; ++i) {
      pq::mbar_init(&bars->s8_full[i], N_UNPACK_WARPS);
      pq::mbar_init(&bars->s8_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      pq::mbar_init(&bars->acc_full[i], 1);
      pq::mbar_init(&bars->acc_empty[i], 4);
    }
    pq::mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    pq::mbar_fence_init();
    pq::fence_proxy_async_smem();
    pq::tma_prefetch_desc(&tmap_a);
    pq::tma_prefetch_desc(&tmap_b);
  }
  if (warp == 1) {
    pq::tmem_alloc(&bars->tmem_base, TMEM_COLS);
    pq::tmem_relinquish();
  }
  pq::tc_fence_before();
  __syncthreads();
  pq::tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % p.tiles_m) * BM, n0 = (tile / p.tiles_m) * BN;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % N_PK, ph = (it / N_PK) & 1;
          if (bars->abort_flag || !pq::mbar_wait(&bars->pk_empty[s], ph ^ 1)) {
            ok = false;
            break;
          }
          pq::mbar_arrive_expect_tx(&bars->pk_full[s], PK_STAGE);
          pq::tma_load_2d(pk_buf + s * PK_STAGE, &tmap_a, kb * PK_ROW, m0, &bars->pk_full[s]);
          pq::tma_load_2d(pk_buf + s * PK_STAGE + PK_A, &tmap_b, kb * PK_ROW, n0, &bars->pk_full[s]);
        }
      }
      if (!ok) {
        bars->abort_flag = 1;
        pq::report(p.status, PQ_ERR_TIMEOUT);
        // let the copies this thread started land before the CTA can exit
        const uint32_t first = it > N_PK ? it - N_PK : 0;
        for (uint32_t j = first; j < it; ++j) pq::mbar_wait(&bars->pk_full[j % N_PK], (j / N_PK) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = pq::umma_idesc_s8(BM, BN);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tcount) {
        const uint32_t ab = tcount & 1, aph = (tcount >> 1) & 1;
        if (bars->abort_flag || !pq::mbar_wait(&bars->acc_empty[ab], aph ^ 1)) {
          ok = false;
          break;
        }
        pq::tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * BN;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % N_S8, ph = (it / N_S8) & 1;
          if (bars->abort_flag || !pq::mbar_wait(&bars->s8_full[s], ph)) {
            ok = false;
            break;
          }
          pq::tc_fence_after();
          const uint32_t a_addr = pq::smem_u32(s8_buf + s * S8_STAGE);
          const uint32_t b_addr = a_addr + S8_A;
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            pq::mma_i8_ss(d_tmem, pq::umma_desc_sw128(a_addr + kk * 32), pq::umma_desc_sw128(b_addr + kk * 32), idesc,
                          (kb | kk) != 0 ? 1u : 0u);
          }
          pq::mma_commit(&bars->s8_empty[s]);  // frees the operand stage once these MMAs have read it
        }
        if (ok) pq::mma_commit(&bars->acc_full[ab]);
      }
      if (!ok) {
        bars->abort_flag = 1;
        pq::report(p.status, PQ_ERR_TIMEOUT);
        pq::mma_commit(&bars->drain);  // wait for whatever was issued before TMEM is released
        pq::mbar_wait(&bars->drain, 0);
      }
    }
  } else if (warp >= UNPACK_WARP0) {
    // ------------------------------------------------------------------ unpack warps
    const int ut = threadIdx.x - UNPACK_WARP0 * 32;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      for (int kb = 0; kb < n_kb; ++kb, ++it) {
        const uint32_t ps = it % N_PK, pph = (it / N_PK) & 1;
        const uint32_t ss = it % N_S8, sph = (it / N_S8) & 1;
        const bool stuck = bars->abort_flag || !pq::mbar_wait(&bars->pk_full[ps], pph) ||
                           !pq::mbar_wait(&bars->s8_empty[ss], sph ^ 1);
        if (__any_sync(0xffffffffu, stuck)) {  // warp-uniform decision
          ok = false;
          break;
        }
        const uint8_t* src = pk_buf + ps * PK_STAGE;
        uint8_t* dst = s8_buf + ss * S8_STAGE;
        constexpr int UNITS = (BM + BN) * 4;  // one unit = one 16-byte packed chunk
#pragma unroll
        for (int i = 0; i < UNITS / (N_UNPACK_WARPS * 32); ++i) {
          const int unit = i * (N_UNPACK_WARPS * 32) + ut;
          const int row = unit >> 2, j = unit & 3;
          const uint4 w = *reinterpret_cast<const uint4*>(src + row * PK_ROW + j * 16);
          uint4 lo, hi;
          lo.x = pq::nib_lo_x16(w.x), lo.y = pq::nib_lo_x16(w.y), lo.z = pq::nib_lo_x16(w.z), lo.w = pq::nib_lo_x16(w.w);
          hi.x = pq::nib_hi_x16(w.x), hi.y = pq::nib_hi_x16(w.y), hi.z = pq::nib_hi_x16(w.z), hi.w = pq::nib_hi_x16(w.w);
          uint8_t* drow = dst + row * BK;
          const int sw = row & 7;
          *reinterpret_cast<uint4*>(drow + (((2 * j) ^ sw) << 4)) = lo;
          *reinterpret_cast<uint4*>(drow + (((2 * j + 1) ^ sw) << 4)) = hi;
        }
        pq::fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's async proxy
        __syncwarp();
        if (lane == 0) {
          pq::mbar_arrive(&bars->s8_full[ss]);
          pq::mbar_arrive(&bars->pk_empty[ps]);
        }
      }
    }
    if (!ok && lane == 0) {
      bars->abort_flag = 1;
      pq::report(p.status, PQ_ERR_TIMEOUT);
    }
  } else if (warp >= EPI_WARP0) {
    // ------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;  // TMEM lane quarter this warp may access
    const float s_a = __ldg(p.s_a);
    uint32_t tcount = 0;
    bool ok = true;
    const bool vec_ok = (p.ldo % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                        ((reinterpret_cast<uintptr_t>(p.s_w) & 15) == 0);
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tcount) {
      const int m0 = (tile % p.tiles_m) * BM, n0 = (tile / p.tiles_m) * BN;
      const uint32_t ab = tcount & 1, aph = (tcount >> 1) & 1;
      const bool stuck = bars->abort_flag || !pq::mbar_wait(&bars->acc_full[ab], aph);
      if (__any_sync(0xffffffffu, stuck)) {  // warp-uniform: the TMEM loads below are warp-collective
        ok = false;
        break;
      }
      pq::tc_fence_after();
      const int row = m0 + q * 32 + lane;
      const uint32_t taddr = tmem_base + ab * BN + (static_cast<uint32_t>(q * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        pq::tmem_ld_32x32(taddr + c * 32, r);
        pq::tmem_ld_wait();
        if (c == BN / 32 - 1) {  // accumulator fully read: hand the buffer back to the MMA warp
          pq::tc_fence_before();
          __syncwarp();
          if (lane == 0) pq::mbar_arrive(&bars->acc_empty[ab]);
        }
        const int col0 = n0 + c * 32;
        if (row < p.M && col0 < p.N) {
          if (vec_ok && col0 + 32 <= p.N) {
            __nv_bfloat16* orow = p.out + static_cast<int64_t>(row) * p.ldo + col0;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint32_t packed[4];
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const float4 sw = __ldg(reinterpret_cast<const float4*>(p.s_w + col0 + g * 8 + h * 4));
                const int b = g * 8 + h * 4;
                float f0 = static_cast<float>(static_cast<int32_t>(r[b + 0]) >> 8) * (s_a * sw.x);
                float f1 = static_cast<float>(static_cast<int32_t>(r[b + 1]) >> 8) * (s_a * sw.y);
                float f2 = static_cast<float>(static_cast<int32_t>(r[b + 2]) >> 8) * (s_a * sw.z);
                float f3 = static_cast<float>(static_cast<int32_t>(r[b + 3]) >> 8) * (s_a * sw.w);
                __nv_bfloat162 p01 = __floats2bfloat162_rn(f0, f1);
                __nv_bfloat162 p23 = __floats2bfloat162_rn(f2, f3);
                packed[h * 2 + 0] = *reinterpret_cast<uint32_t*>(&p01);
                packed[h * 2 + 1] = *reinterpret_cast<uint32_t*>(&p23);
              }
              *reinterpret_cast<uint4*>(orow + g * 8) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            }
          } else {
            for (int i = 0; i < 32; ++i) {
              const int col = col0 + i;
              if (col < p.N) {
                float f = static_cast<float>(static_cast<int32_t>(r[i]) >> 8) * (s_a * __ldg(p.s_w + col));
                p.out[static_cast<int64_t>(row) * p.ldo + col] = __float2bfloat16_rn(f);
              }
            }
          }
          if (p.acc_dbg) {
            for (int i = 0; i < 32; ++i) {
              const int col = col0 + i;
              if (col < p.N) p.acc_dbg[static_cast<int64_t>(row) * p.N + col] = static_cast<int32_t>(r[i]) >> 8;
            }
          }
        }
      }
    }
    if (!ok && lane == 0) {
      bars->abort_flag = 1;
      pq::report(p.status, PQ_ERR_TIMEOUT);
    }
  }

  pq::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    pq::tc_fence_after();
    pq::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map over a dense packed matrix [rows, kbytes] of bytes; box = [box_rows, 64 bytes].
bool make_packed_map(pq_ctx* ctx, CUtensorMap* map, const uint8_t* base, int64_t rows, int64_t kbytes, int box_rows) {
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(kbytes), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstride[1] = {static_cast<cuuint64_t>(kbytes)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(PK_ROW), static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), gdim, gstride, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

// Launches the tensor-core kernel on rows [0, M) of xq/out (the caller has already applied row_begin).
pq_status pq_gemm_tc_launch(pq_ctx* ctx, const uint8_t* xq, const uint8_t* wq, const float* s_a, const float* s_w,
                            void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t* acc_dbg,
                            cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_packed_map(ctx, &ta, xq, M, K / 2, BM) || !make_packed_map(ctx, &tb, wq, N, K / 2, BN)) return PQ_ERR_CUDA;
  GemmParams p;
  p.s_a = s_a;
  p.s_w = s_w;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.acc_dbg = acc_dbg;
  p.status = ctx->d_status;
  p.ldo = ldo;
  p.M = static_cast<int>(M);
  p.N = static_cast<int>(N);
  p.K = static_cast<int>(K);
  p.tiles_m = static_cast<int>((M + BM - 1) / BM);
  p.tiles_n = static_cast<int>((N + BN - 1) / BN);
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_w4a4_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(SMEM_BYTES)) != cudaSuccess)
      return PQ_ERR_CUDA;
    attr_set = true;
  }
  const int n_tiles = p.tiles_m * p.tiles_n;
  const int grid = n_tiles < ctx->sm_count ? n_tiles : ctx->sm_count;
  gemm_w4a4_tc_kernel<<<grid, N_THREADS, SMEM_BYTES, st>>>(ta, tb, p);
  return pq_launch_status();
}

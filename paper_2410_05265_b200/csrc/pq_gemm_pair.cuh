// What the two CTA-pair GEMM kernels share: the cluster / tensor-memory / bulk-store wrappers, the launch parameters,
// the epilogue of a tile (tensor memory -> exact shift -> optional zero-point term -> scale -> bf16 -> swizzled
// staging -> TMA store) and the host-side tensor maps. The kernels differ in how the token operand reaches the MMA
// (shared memory in pq_gemm_tc2.cu, tensor memory in pq_gemm_tc3.cu) and in their accumulator buffering.
#pragma once

#include "pq_common.cuh"

namespace pq_pair {

constexpr int BM_CTA = 128;                 // token rows per CTA (256 per pair)
constexpr int BN = 256;                     // output channels per pair tile
constexpr int BN_CTA = 128;                 // weight rows expanded by each CTA
constexpr int BK = 128;                     // K elements per stage
constexpr int PK_ROW = BK / 2;              // packed bytes per row per stage
constexpr int EPI_COLS = 64;                // columns per TMA store (128 bytes of bf16)
constexpr int EPI_BUF = 32 * EPI_COLS * 2;  // 4 KB: one warp's 32 rows x 64 columns

struct GemmParams {
  const int32_t* zp;    // ZP kernels: the activation zero point z (device scalar) ...
  const int32_t* wsum;  // ... and the sum of every output channel's weight codes [N]
  const float* s_row;  // per-token steps [M] (dynamic setting) or null: the scalar s_a applies
  const float* s_a;
  const float* s_w;
  __nv_bfloat16* out;
  int32_t* acc_dbg;
  int32_t* status;
  int64_t ldo;
  int M, N, K;
  int tiles_m, tiles_n;
  int tma_store;  // out can be written with TMA stores (16-byte aligned base and row pitch)
  long long wait_clocks;  // bound of every device-side wait, in SM clocks
};

// ---- cluster-scope helpers ---------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory object in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(pq::smem_u32(p)), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  // default semantics on purpose: a cluster-scope release here waits for the CTA's TMA traffic in
  // flight and costs more than the rest of the stage; the data this arrival publishes is the warp's
  // own shared-memory stores, already ordered by the proxy fence before it
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_local(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(pq::smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait (`limit` SM clocks); also gives up when the CTA's abort flag is raised.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag, long long limit) {
  if (mbar_try_wait_local(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait_local(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) return false;
  }
}

// ---- tcgen05, cta_group::2 forms ---------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc2(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pq::smem_u32(smem_dst)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// One arrival on the barrier at this shared-memory offset in both CTAs of the pair, once every MMA
// issued so far by this thread has completed.
__device__ __forceinline__ void mma2_commit_both(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
          pq::smem_u32(bar)),
      "h"(static_cast<uint16_t>(3))
      : "memory");
}

// ---- TMA store ----------------------------------------------------------------------------------
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, const void* src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(pq::smem_u32(src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---- epilogue -------------------------------------------------------------------------------------
// ZP (Eq. 1 as printed): the stored token codes are u - 8 for unsigned codes u with zero point z; what the
// layer needs is sum_k (u - z) w = sum_k (u - 8) w - (z - 8) sum_k w, so the epilogue subtracts (z - 8) * wsum[n]
// from the exact integer sum before scaling.
// This warp's copy of the dequantization factors of a tile's 256 columns (and of those correction terms).
template <bool ZP>
__device__ __forceinline__ void fill_tile_scales(const GemmParams& p, int n0, int lane, float s_a, int zp8, float* my_scale,
                                                 int32_t* my_zw) {
#pragma unroll
  for (int i = 0; i < BN / 32; ++i) {
    const int col = n0 + i * 32 + lane;
    my_scale[i * 32 + lane] = col < p.N ? s_a * __ldg(p.s_w + col) : 0.0f;
    if (ZP) my_zw[i * 32 + lane] = col < p.N ? zp8 * __ldg(p.wsum + col) : 0;
  }
  __syncwarp();
}

// One warp's 32 rows x 256 columns of an accumulator at tensor-memory address taddr: row m0 + lane of the output.
// SHIFT removes the factors 16 the expanded codes carry (exact). `rs` is the lane's token step (1 in the static
// setting). After the last column block has been read, lane 0 arrives on `acc_empty` (a cluster address in the
// leader CTA), which hands the accumulator back to the MMA warp. n_store counts this warp's TMA stores (rotation of
// the staging buffers).
template <int SHIFT, bool ZP, int EPI_BUFS>
__device__ __forceinline__ void epilogue_tile(const GemmParams& p, const CUtensorMap* tmap_out, uint32_t taddr, int m0, int n0,
                                              int lane, float rs, const float* my_scale, const int32_t* my_zw, uint8_t* my_buf,
                                              uint32_t& n_store, uint32_t acc_empty) {
  const int row = m0 + lane;
#pragma unroll 1
  for (int c = 0; c < BN / 32; ++c) {
    uint32_t r[32];
    pq::tmem_ld_32x32(taddr + c * 32, r);
    pq::tmem_ld_wait();
    if (c == BN / 32 - 1) {  // accumulator fully read
      pq::tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty);
    }
    const int col0 = n0 + c * 32;
    auto sum = [&](int i) { return (static_cast<int32_t>(r[i]) >> SHIFT) - (ZP ? my_zw[c * 32 + i] : 0); };
    if (p.tma_store) {
      uint8_t* buf = my_buf + (n_store % EPI_BUFS) * EPI_BUF;
      if ((c & 1) == 0) {  // the store that last read this buffer is EPI_BUFS stores back
        if (lane == 0) bulk_wait_read<EPI_BUFS - 1>();
        __syncwarp();
      }
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const float4 sa = *reinterpret_cast<const float4*>(my_scale + c * 32 + g * 8);
        const float4 sb = *reinterpret_cast<const float4*>(my_scale + c * 32 + g * 8 + 4);
        const int b = g * 8;
        const __nv_bfloat162 p0 = __floats2bfloat162_rn(static_cast<float>(sum(b + 0)) * sa.x * rs, static_cast<float>(sum(b + 1)) * sa.y * rs);
        const __nv_bfloat162 p1 = __floats2bfloat162_rn(static_cast<float>(sum(b + 2)) * sa.z * rs, static_cast<float>(sum(b + 3)) * sa.w * rs);
        const __nv_bfloat162 p2 = __floats2bfloat162_rn(static_cast<float>(sum(b + 4)) * sb.x * rs, static_cast<float>(sum(b + 5)) * sb.y * rs);
        const __nv_bfloat162 p3 = __floats2bfloat162_rn(static_cast<float>(sum(b + 6)) * sb.z * rs, static_cast<float>(sum(b + 7)) * sb.w * rs);
        const int chunk = (c & 1) * 4 + g;  // 16-byte chunk inside the 128-byte staging row
        *reinterpret_cast<uint4*>(buf + lane * 128 + ((chunk ^ (lane & 7)) << 4)) =
            make_uint4(*reinterpret_cast<const uint32_t*>(&p0), *reinterpret_cast<const uint32_t*>(&p1),
                       *reinterpret_cast<const uint32_t*>(&p2), *reinterpret_cast<const uint32_t*>(&p3));
      }
      if (c & 1) {
        pq::fence_proxy_async_smem();
        __syncwarp();
        const int x = n0 + (c >> 1) * EPI_COLS;
        if (lane == 0 && x < p.N && m0 < p.M) {
          tma_store_2d(tmap_out, buf, x, m0);
          bulk_commit();
        }
        ++n_store;
      }
    } else if (row < p.M) {
      for (int i = 0; i < 32; ++i) {
        const int col = col0 + i;
        if (col < p.N)
          p.out[static_cast<int64_t>(row) * p.ldo + col] = __float2bfloat16_rn(static_cast<float>(sum(i)) * my_scale[c * 32 + i] * rs);
      }
    }
    if (p.acc_dbg && row < p.M) {
      for (int i = 0; i < 32; ++i) {
        const int col = col0 + i;
        if (col < p.N) p.acc_dbg[static_cast<int64_t>(row) * p.N + col] = sum(i);
      }
    }
  }
  __syncwarp();  // every lane is done with my_scale before the next tile overwrites it
}

// ---- host side: tensor maps -----------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map over a dense packed matrix [rows, kbytes] of bytes; box = [box_rows, 64 bytes]. The kernel that reads
// the landing buffer one row per thread asks for the 64-byte swizzle (16-byte chunk index XOR (row >> 1) & 3) so that
// those reads hit distinct banks; the other reads it chunk by chunk and takes it unswizzled.
inline bool make_packed_map(pq_ctx* ctx, CUtensorMap* map, const uint8_t* base, int64_t rows, int64_t kbytes, int box_rows,
                            CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE) {
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(kbytes), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstride[1] = {static_cast<cuuint64_t>(kbytes)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(PK_ROW), static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  return reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
             map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map over a dense s8 matrix [rows, K]; box = [128 rows, 128 bytes] landing in the 128-byte-swizzled
// K-major layout the MMA descriptors read.
inline bool make_s8_map(pq_ctx* ctx, CUtensorMap* map, const uint8_t* base, int64_t rows, int64_t K) {
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstride[1] = {static_cast<cuuint64_t>(K)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(BK), static_cast<cuuint32_t>(BM_CTA)};
  cuuint32_t estr[2] = {1, 1};
  return reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
             map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map over the bf16 output [M, N] with row pitch ldo; box = [32 rows, 64 columns], 128-byte swizzle.
inline bool make_out_map(pq_ctx* ctx, CUtensorMap* map, void* out, int64_t M, int64_t N, int64_t ldo) {
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(M)};
  cuuint64_t gstride[1] = {static_cast<cuuint64_t>(ldo) * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(EPI_COLS), 32};
  cuuint32_t estr[2] = {1, 1};
  return reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
             map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, out, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace pq_pair

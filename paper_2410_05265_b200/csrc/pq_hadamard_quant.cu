// Online Walsh-Hadamard rotation of a linear layer's input (App. B, "Online Rotation") fused with
// the static per-tensor INT4 quantizer (Table 1, O2; Eq. 1) and the nibble pack; the same
// butterfly also serves the calibration helper that produces the static scale, and the 8-bit
// quantizer of the W4A8 precision (Sec. 5.1), which stores one signed byte per element.
//
// A B-wide block (B = 2^LOGB) is transformed by B/64 threads, 64 values per thread, in two
// register passes joined by one trip through shared memory:
//   pass 1: thread u loads 32 bf16 pairs (coalesced 4-byte loads, 128 bytes per warp request) and
//           holds index bits {i0} + the five top bits; six butterfly stages in registers.
//   exchange: values go to shared memory (8-byte stores, 2 floats of padding per 128 so that the
//           transposed reads hit 32 distinct banks).
//   pass 2: thread u' holds index bits i1..i6 of one 128-element segment for one value of i0;
//           the remaining stages run in registers (plus one lane-shuffle stage when B = 8192).
//   quantize: clamp, add 1.5*2^23 (the FP add performs the round-half-even), take the low nibble;
//           lane pairs swap half of their nibbles so that each thread stores 32 contiguous bytes.
#include "pq_common.cuh"

namespace {

constexpr int HQ_THREADS = 128;
constexpr int HQ_CTAS_PER_SM = 5;         // 33 KB of shared memory and about 11K registers each
constexpr int HQ_ELEMS = HQ_THREADS * 64;             // elements handled per CTA iteration
constexpr int HQ_SMEM_FLOATS = HQ_ELEMS + HQ_ELEMS / 64;  // + 2 floats of padding per 128

// PER_TOKEN (the dynamic setting, Table 1, O1): one step per row instead of one per tensor; s_a_in / s_a_out
// are then arrays indexed by row, and the calibration pass is the online first pass of every call.
// ZP (Eq. 1 with its zero point): the quantizer adds z - 8 to the rounded value before the clamp, so
// that the stored signed nibble is the unsigned code minus 8; the calibration pass collects the minimum and
// the maximum of the rotated values (as order-preserving integer keys in s_a_out[0] and s_a_out[1]).
__device__ __forceinline__ uint32_t float_key(float f) {
  const uint32_t b = __float_as_uint(f);
  return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  return __uint_as_float(k ^ ((k >> 31) ? 0x80000000u : 0xFFFFFFFFu));
}

// SWIGLU: the input of the transform is SiLU(x) * x2 (the gate and up halves of the MLP, App. B), computed in fp32
// and rounded to bf16 exactly as the stand-alone kernel stores it, so that fusing it changes no bit; the
// activation tensor of the down projection then never goes to memory.
__device__ __forceinline__ float swiglu_bf16(float g, float u) {
  return __bfloat162float(__float2bfloat16_rn(pq::silu_mul_f32(g, u)));
}

// GRID (with CALIB and ZP; the grid search of Sec. 3 for the static s and z): s_a_in / zp_in hold n_cand candidate
// (s, z) pairs, and the pass adds to s_a_out (n_cand doubles) the squared error of quantizing and dequantizing the
// rotated values with each of them. With PER_TOKEN (the search for the clipping factor that the tokens of the dynamic
// setting share) s_a_in holds every row's unclipped step, x2 (as floats) the n_cand candidate factors, and a row's
// candidate step is factor * step; the codes are the symmetric ones (zero point 8).
// NORM (the RMSNorm in front of a block's first linears, App. B figure): the row is one transform block; its values
// become bf16(x * r * g) with r = 1 / sqrt(mean(x^2) + eps) before the transform, in the arithmetic and with the
// rounding of the stand-alone call, so that fusing changes no bit. x2 is then the gain g [K], clip carries eps.
// NORM == 2 stops there and writes the normalised row (bf16, to xq with row pitch n_cand elements): the stand-alone
// RMSNorm of such widths, which thereby shares every operation that decides r with the fused form.
template <int LOGB, bool ROTATE, bool CALIB, int BITS, bool PER_TOKEN, bool ZP, bool SWIGLU, bool GRID = false, int NORM = 0>
__global__ void __launch_bounds__(HQ_THREADS, HQ_CTAS_PER_SM)
    hadamard_quant_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, int64_t n_rows, int64_t K,
                          const float* __restrict__ s_a_in, uint8_t* __restrict__ xq, float* __restrict__ s_a_out,
                          float clip, const int32_t* __restrict__ zp_in, const __nv_bfloat16* __restrict__ x2, int n_cand) {
  static_assert(BITS == 4 || BITS == 8, "code width");
  constexpr int QMAX = BITS == 4 ? 7 : 127;  // codes lie in [-QMAX - 1, QMAX]
  constexpr int B = 1 << LOGB;
  constexpr int TPB = B / 64;                  // threads per block of the transform
  constexpr int G = HQ_THREADS / TPB;          // blocks per CTA iteration
  constexpr int BLK_FLOATS = B + B / 64;       // padded block footprint in shared memory
  constexpr int RSTRIDE = 1 << (LOGB - 5);     // element distance between consecutive r
  extern __shared__ __align__(16) float sm[];
  __shared__ float norm_red[HQ_THREADS / 32];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // input, scale and output may belong to the previous kernel

  const int tid = threadIdx.x;
  const int blk_local = tid / TPB;
  const int u = tid % TPB;
  const int64_t blocks_per_row = K / B;
  const int64_t total_blocks = n_rows * blocks_per_row;
  const int64_t n_super = (total_blocks + G - 1) / G;
  float* my = sm + blk_local * BLK_FLOATS;
  // The exchange of a B-wide block involves only its own B/64 threads: for B <= 2048 that is a warp or
  // part of one, and a warp-level barrier lets the other blocks of the CTA run ahead (named barriers for
  // the two-warp case of B = 4096 measured slower than the CTA barrier).
  auto block_sync = [&]() {
    if (TPB <= 32) __syncwarp();
    else __syncthreads();
  };

  const float norm = ROTATE ? __fdiv_rn(1.0f, __fsqrt_rn(static_cast<float>(B))) : 1.0f;
  float inv = norm;
  if (!CALIB && !PER_TOKEN) inv = __fdiv_rn(norm, __ldg(s_a_in));
  float cal_max = 0.0f, cal_lo = INFINITY, cal_hi = -INFINITY;
  const int zp = (ZP && !CALIB) ? __ldg(zp_in) - 8 : 0;

  // (row, block inside the row) of this thread's transform block: divided once, then advanced by the grid's stride
  // (a 64-bit division per iteration is a visible share of an instruction-bound kernel)
  const int64_t gb_step = static_cast<int64_t>(gridDim.x) * G;
  const int64_t row_step = gb_step / blocks_per_row, blk_step = gb_step % blocks_per_row;
  int64_t gb = static_cast<int64_t>(blockIdx.x) * G + blk_local;
  int64_t row_it = gb / blocks_per_row, blk_it = gb % blocks_per_row;
  for (int64_t sb = blockIdx.x; sb < n_super; sb += gridDim.x, gb += gb_step) {
    const bool active = gb < total_blocks;
    const int64_t row = active ? row_it : 0;
    const int64_t col0 = active ? blk_it * B : 0;
    row_it += row_step, blk_it += blk_step;
    if (blk_it >= blocks_per_row) blk_it -= blocks_per_row, ++row_it;
    if (!CALIB && PER_TOKEN) {
      const float s_row = __ldg(s_a_in + row);
      inv = __fdiv_rn(norm, s_row == 0.0f ? 1.0f : s_row);  // an all-zero row has no step: any will do
    }

    // ---- pass 1 --------------------------------------------------------------------------
    // V[r] = (x[2u + r*RSTRIDE], x[2u+1 + r*RSTRIDE]) after the stage on index bit 0; the other five
    // stages combine whole pairs, two fp32 additions per instruction.
    float2 V[32];
    {
      const uint32_t* src = reinterpret_cast<const uint32_t*>(x + row * ldx + col0) + u;
      uint32_t w[32];
#pragma unroll
      for (int r = 0; r < 32; ++r) w[r] = active ? __ldg(src + r * (RSTRIDE / 2)) : 0u;
      if (SWIGLU) {
        const uint32_t* src2 = reinterpret_cast<const uint32_t*>(x2 + row * ldx + col0) + u;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          const uint32_t w2 = active ? __ldg(src2 + r * (RSTRIDE / 2)) : 0u;
          const float a = swiglu_bf16(__uint_as_float(w[r] << 16), __uint_as_float(w2 << 16));
          const float b = swiglu_bf16(__uint_as_float(w[r] & 0xFFFF0000u), __uint_as_float(w2 & 0xFFFF0000u));
          V[r] = ROTATE ? make_float2(a + b, a - b) : make_float2(a, b);
        }
      } else if (NORM) {
        // sum of squares of the row: this thread's 64 values in a fixed order, then the block's threads (lanes of a
        // warp by shuffles, warps through shared memory in warp order): the same sequence in both forms
        float ss = 0.0f;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          const float a = __uint_as_float(w[r] << 16), b = __uint_as_float(w[r] & 0xFFFF0000u);
          ss = __fmaf_rn(a, a, __fmaf_rn(b, b, ss));
        }
        constexpr int SPAN = TPB < 32 ? TPB : 32;
#pragma unroll
        for (int o = SPAN / 2; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (TPB > 32) {
          if ((tid & 31) == 0) norm_red[tid >> 5] = ss;
          __syncthreads();
          ss = 0.0f;
#pragma unroll
          for (int i = 0; i < TPB / 32; ++i) ss += norm_red[blk_local * (TPB / 32) + i];
          __syncthreads();
        }
        const float rr = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(ss, static_cast<float>(B)), clip)));
        const uint32_t* gsrc = reinterpret_cast<const uint32_t*>(x2 + col0) + u;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          const uint32_t gw = __ldg(gsrc + r * (RSTRIDE / 2));
          const float a = __bfloat162float(__float2bfloat16_rn(__fmul_rn(__fmul_rn(__uint_as_float(w[r] << 16), rr), __uint_as_float(gw << 16))));
          const float b = __bfloat162float(__float2bfloat16_rn(__fmul_rn(__fmul_rn(__uint_as_float(w[r] & 0xFFFF0000u), rr), __uint_as_float(gw & 0xFFFF0000u))));
          if (NORM == 2) {
            if (active)
              reinterpret_cast<uint32_t*>(reinterpret_cast<__nv_bfloat16*>(xq) + row * n_cand + col0)[u + r * (RSTRIDE / 2)] =
                  (__float_as_uint(a) >> 16) | (__float_as_uint(b) & 0xFFFF0000u);
          }
          V[r] = ROTATE ? make_float2(a + b, a - b) : make_float2(a, b);
        }
        if (NORM == 2) continue;
      } else {
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          const float a = __uint_as_float(w[r] << 16), b = __uint_as_float(w[r] & 0xFFFF0000u);
          V[r] = ROTATE ? make_float2(a + b, a - b) : make_float2(a, b);
        }
      }
    }
    if (ROTATE) {
#pragma unroll
      for (int s = 0; s < 5; ++s) {
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          if ((r & (1 << s)) == 0) {
            const int r2 = r | (1 << s);
            const float2 a = V[r], b = V[r2];
            V[r] = __fadd2_rn(a, b);
            V[r2] = __ffma2_rn(b, make_float2(-1.0f, -1.0f), a);
          }
        }
      }
    }
    // ---- exchange ------------------------------------------------------------------------
#pragma unroll
    for (int r = 0; r < 32; ++r) {
      const int i = r * RSTRIDE + 2 * u;
      *reinterpret_cast<float2*>(my + i + 2 * (i >> 7)) = V[r];
    }
    block_sync();
    const int seg = u >> 1, par = u & 1;
    // ---- pass 2: W[q] = (v[q], v[q + 32]); stages on index bits 1..5 of the segment combine pairs,
    // the stage on bit 6 works inside a pair ---------------------------------------------------
    float2 W[32];
    {
      const float* src = my + seg * 130 + par;
#pragma unroll
      for (int q = 0; q < 32; ++q) W[q] = make_float2(src[2 * q], src[2 * q + 64]);
    }
    block_sync();
    if (ROTATE) {
#pragma unroll
      for (int j = 0; j < 5; ++j) {
        if (j < LOGB - 6) {
#pragma unroll
          for (int q = 0; q < 32; ++q) {
            if ((q & (1 << j)) == 0) {
              const int q2 = q | (1 << j);
              const float2 a = W[q], b = W[q2];
              W[q] = __fadd2_rn(a, b);
              W[q2] = __ffma2_rn(b, make_float2(-1.0f, -1.0f), a);
            }
          }
        }
      }
      if (LOGB - 6 > 5) {
#pragma unroll
        for (int q = 0; q < 32; ++q) W[q] = make_float2(W[q].x + W[q].y, W[q].x - W[q].y);
      }
      if (LOGB == 13) {  // index bit 7 lives in lane bit 1
        const float sgn = (u & 2) ? -1.0f : 1.0f;
#pragma unroll
        for (int q = 0; q < 32; ++q) {
          const float ox = __shfl_xor_sync(0xffffffffu, W[q].x, 2), oy = __shfl_xor_sync(0xffffffffu, W[q].y, 2);
          W[q] = make_float2(fmaf(W[q].x, sgn, ox), fmaf(W[q].y, sgn, oy));
        }
      }
    }
    if (CALIB) {
      float it_max = 0.0f;
      if (active) {
#pragma unroll
        for (int q = 0; q < 32; ++q) it_max = fmaxf(it_max, fmaxf(fabsf(W[q].x * norm), fabsf(W[q].y * norm)));
      }
      if (GRID) {
        double* sse = reinterpret_cast<double*>(s_a_out);
#pragma unroll 1
        for (int c = 0; c < n_cand; ++c) {
          float s, z;
          if (PER_TOKEN) {
            const float s_row = __ldg(s_a_in + row);
            s = s_row == 0.0f ? 1.0f : __fmul_rn(__ldg(reinterpret_cast<const float*>(x2) + c), s_row), z = 8.0f;
          } else {
            s = __ldg(s_a_in + c), z = static_cast<float>(__ldg(zp_in + c));
          }
          const float inv_s = __fdiv_rn(1.0f, s);
          float acc = 0.0f;
          if (active) {
#pragma unroll
            for (int q = 0; q < 32; ++q) {
              const float a = W[q].x * norm, b = W[q].y * norm;
              const float ua = fminf(fmaxf(rintf(a * inv_s) + z, 0.0f), 15.0f), ub = fminf(fmaxf(rintf(b * inv_s) + z, 0.0f), 15.0f);
              const float ea = a - s * (ua - z), eb = b - s * (ub - z);
              acc = fmaf(ea, ea, acc);
              acc = fmaf(eb, eb, acc);
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
          if ((tid & 31) == 0 && acc != 0.0f) atomicAdd(sse + c, static_cast<double>(acc));
        }
      } else if (ZP) {
        if (active) {
#pragma unroll
          for (int q = 0; q < 32; ++q) {
            const float a = W[q].x * norm, b = W[q].y * norm;
            cal_lo = fminf(cal_lo, fminf(a, b)), cal_hi = fmaxf(cal_hi, fmaxf(a, b));
          }
        }
      } else if (PER_TOKEN) {
        // the maximum of this row's block, over the TPB threads that hold it (a warp or a part of one; blocks
        // wider than a warp's 2048 elements, and rows of several blocks, meet in the atomic)
        constexpr int SPAN = TPB < 32 ? TPB : 32;
#pragma unroll
        for (int o = SPAN / 2; o > 0; o >>= 1) it_max = fmaxf(it_max, __shfl_xor_sync(0xffffffffu, it_max, o));
        if ((tid % SPAN) == 0 && active && it_max > 0.0f)
          atomicMax(reinterpret_cast<int*>(s_a_out + row), __float_as_int(__fdiv_rn(it_max * clip, static_cast<float>(QMAX))));
      } else {
        cal_max = fmaxf(cal_max, it_max);
      }
    } else {
      // ---- quantize and pack -----------------------------------------------------------------
      // y * inv + 1.5 * 2^23: the fp32 addition rounds half to even and leaves the integer in the low
      // mantissa bits; clamped as an integer, the low byte is the code as an s8.
      const float2 inv2 = make_float2(inv, inv), magic2 = make_float2(12582912.0f, 12582912.0f);
      // byte stores with a narrower code range (4-bit codes, one per byte): the caller's largest code in n_cand
      const int qmax = (BITS == 8 && n_cand > 0) ? n_cand : QMAX;
      uint32_t pw[16];  // word wd: codes of v[4wd .. 4wd+3], one nibble per byte
#pragma unroll
      for (int wd = 0; wd < 8; ++wd) {
        int lo[4], hi[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const float2 tq = __ffma2_rn(W[4 * wd + b], inv2, magic2);
          lo[b] = max(min(__float_as_int(tq.x) + zp, 0x4B400000 + qmax), 0x4B400000 - qmax - 1);
          hi[b] = max(min(__float_as_int(tq.y) + zp, 0x4B400000 + qmax), 0x4B400000 - qmax - 1);
        }
        pw[wd] = __byte_perm(__byte_perm(lo[0], lo[1], 0x0040), __byte_perm(lo[2], lo[3], 0x0040), 0x5410);
        pw[wd + 8] = __byte_perm(__byte_perm(hi[0], hi[1], 0x0040), __byte_perm(hi[2], hi[3], 0x0040), 0x5410);
      }
      // This thread holds the elements of one parity of its 128-wide segment (pw[0..7]: first half,
      // pw[8..15]: second half); its neighbour holds the other parity. Each sends the half the other
      // is going to store, so that both write contiguous bytes.
      if (BITS == 4) {
        uint32_t fin[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t mine = (par ? pw[8 + j] : pw[j]) & 0x0F0F0F0Fu;
          const uint32_t recv = __shfl_xor_sync(0xffffffffu, (par ? pw[j] : pw[8 + j]) & 0x0F0F0F0Fu, 1);
          fin[j] = par ? (recv | (mine << 4)) : (mine | (recv << 4));
        }
        if (active) {
          uint4* dst = reinterpret_cast<uint4*>(xq + row * (K / 2) + (col0 + seg * 128) / 2 + par * 32);
          dst[0] = make_uint4(fin[0], fin[1], fin[2], fin[3]);
          dst[1] = make_uint4(fin[4], fin[5], fin[6], fin[7]);
        }
      } else {
        uint32_t fin[16];  // 64 consecutive codes: the first half of the segment for parity 0, the second for parity 1
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t mine = par ? pw[8 + j] : pw[j];
          const uint32_t recv = __shfl_xor_sync(0xffffffffu, par ? pw[j] : pw[8 + j], 1);
          const uint32_t even = par ? recv : mine, odd = par ? mine : recv;
          fin[2 * j] = __byte_perm(even, odd, 0x5140);
          fin[2 * j + 1] = __byte_perm(even, odd, 0x7362);
        }
        if (active) {
          uint4* dst = reinterpret_cast<uint4*>(xq + row * K + col0 + seg * 128 + par * 64);
#pragma unroll
          for (int j = 0; j < 4; ++j) dst[j] = make_uint4(fin[4 * j], fin[4 * j + 1], fin[4 * j + 2], fin[4 * j + 3]);
        }
      }
    }
  }
  if (CALIB && GRID) {
    // nothing left to fold: every candidate's error went out with the blocks
  } else if (CALIB && ZP) {
    for (int o = 16; o > 0; o >>= 1) {
      cal_lo = fminf(cal_lo, __shfl_xor_sync(0xffffffffu, cal_lo, o));
      cal_hi = fmaxf(cal_hi, __shfl_xor_sync(0xffffffffu, cal_hi, o));
    }
    if ((tid & 31) == 0 && cal_hi >= cal_lo) {
      atomicMax(reinterpret_cast<uint32_t*>(s_a_out), float_key(cal_hi));
      atomicMin(reinterpret_cast<uint32_t*>(s_a_out) + 1, float_key(cal_lo));
    }
  } else if (CALIB && !PER_TOKEN) {
    for (int o = 16; o > 0; o >>= 1) cal_max = fmaxf(cal_max, __shfl_xor_sync(0xffffffffu, cal_max, o));
    if ((tid & 31) == 0 && cal_max > 0.0f)
      atomicMax(reinterpret_cast<int*>(s_a_out), __float_as_int(__fdiv_rn(cal_max, static_cast<float>(QMAX))));
  }
}

// ---- wide blocks (B = 2048, 4096, 8192) -------------------------------------------------------------
// The first four stages of the transform run on the tensor cores: the inputs are bf16, the factor is +-1, so
// X (16 x 16 bf16) times H_16 is exact apart from the fp32 accumulation. A warp owns 2048 elements of a block
// (B / 2048 warps per block), 64 per thread, and loads them as 32-bit words so that every request of the warp
// covers whole 32-byte sectors of as few 128-byte lines as the roles below allow. The bits of the block-local
// element index play these roles (J = 13 - LOGB):
//   bit 0                 the two halves of a loaded word (k0 of the MMA)
//   lane % 4 (k1, k2)     bits 1, 2 (B = 2048), bits 1, 6 (B = 4096), bits 6, 7 (B = 8192)
//   lane / 4              the next three bits below bit 6 (the MMA's row inside an 8-row half)
//   warp inside the block the bits left below bit 6 (none, bit 5, bits 4 and 5)
//   the thread's own      the five bits above: m3 (rows 0-7 or 8-15 of the A operand), k3 (columns 0-7 or 8-15)
//                         and a 3-bit tile number tau
// One m16n8k16 MMA per eight output columns transforms bits {0, k1, k2, k3}; m3 and tau are then combined in
// registers as packed fp32 pairs (a pair spans bit 0, which is already done), the values cross shared memory
// once (8-byte stores, 16-byte loads, both conflict-free thanks to the padding below) and come back with the
// thread holding 64 consecutive elements, whose not yet transformed bits (lane / 4 and warp above) are combined in
// registers again. Each thread therefore quantizes and stores 64 consecutive elements.
constexpr int HQW_CTAS_PER_SM = 4;
constexpr int HQW_SMEM_FLOATS = 2 * 4736;  // the widest of 4 x 2176, 2 x 4736 and 9088 padded floats per CTA

__device__ __forceinline__ void mma_bf16_m16n8k16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %10, %10, %10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.0f));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&p);
}

template <int LOGB, bool CALIB, int BITS, bool PER_TOKEN, bool ZP, bool SWIGLU, bool GRID = false, int NORM = 0>
__global__ void __launch_bounds__(HQ_THREADS, HQW_CTAS_PER_SM)
    hadamard_quant_wide_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, int64_t n_rows, int64_t K,
                               const float* __restrict__ s_a_in, uint8_t* __restrict__ xq, float* __restrict__ s_a_out,
                               float clip, const int32_t* __restrict__ zp_in, const __nv_bfloat16* __restrict__ x2, int n_cand) {
  static_assert(LOGB >= 11 && LOGB <= 13, "block width");
  static_assert(BITS == 4 || BITS == 8, "code width");
  constexpr int QMAX = BITS == 4 ? 7 : 127;
  constexpr int B = 1 << LOGB;
  constexpr int J = 13 - LOGB;
  constexpr int T0S = J == 0 ? 6 : 1, T1S = J == 2 ? 2 : (J == 1 ? 6 : 7);   // index bits of lane % 4
  constexpr int GS = J + 1;                                                   // lowest index bit of lane / 4
  constexpr int WS = J + 4;                                                   // lowest index bit of the warp
  constexpr int M3S = 8 - J, K3S = 9 - J, TAUS = 10 - J;                      // the thread's own bits
  // padding of the exchange buffer: float i of a block lives at i + pad(i), with
  //   pad = PADK * (i >> M3S) + 16 * bit 6 (B = 4096) or + 8 * bit 6 + 16 * bit 7 (B = 8192)
  constexpr int PADK = J == 2 ? 4 : (J == 1 ? 20 : 28);
  constexpr int BLKF = J == 2 ? 2176 : (J == 1 ? 4736 : 9088);               // floats per block, padding included
  constexpr int WPB = B / 2048;                      // warps per block
  constexpr int G = (HQ_THREADS / 32) / WPB;
  extern __shared__ __align__(16) float sm[];
  __shared__ float norm_red[HQ_THREADS / 32];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int blk_local = warp / WPB, wv = warp % WPB;
  const int64_t blocks_per_row = K / B;
  const int64_t total_blocks = n_rows * blocks_per_row;
  const int64_t n_super = (total_blocks + G - 1) / G;
  float* my = sm + blk_local * BLKF;
  auto block_sync = [&]() {
    if (WPB == 1) __syncwarp();
    else if (WPB == 2) asm volatile("bar.sync %0, 64;" ::"r"(1 + blk_local) : "memory");
    else __syncthreads();
  };

  // B operand of the MMA: H_16[k][n] = (-1)^popcount(k & n) for the columns n = lane / 4 (+ 8)
  uint32_t hb[2][2];
#pragma unroll
  for (int nb = 0; nb < 2; ++nb)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = 2 * t + 8 * h, n = g + 8 * nb;
      hb[nb][h] = ((__popc(k & n) & 1) ? 0xBF80u : 0x3F80u) | ((__popc((k + 1) & n) & 1) ? 0xBF800000u : 0x3F800000u);
    }

  // element offset of this thread's loads inside the block, and its shared-memory offsets (in floats)
  const int e_thr = ((t & 1) << T0S) | ((t >> 1) << T1S) | (g << GS) | (wv << WS);
  const int wthr = e_thr + (J == 1 ? 16 * (t >> 1) : (J == 0 ? 8 * (t & 1) + 16 * (t >> 1) : 0));
  const int hi = lane | (wv << 5);  // pass 2: this thread holds elements 64 hi .. 64 hi + 63 of the block
  const int rthr = (hi << 6) + PADK * (hi >> (M3S - 6)) + (J == 1 ? 16 * (hi & 1) : (J == 0 ? 8 * (hi & 1) + 16 * ((hi >> 1) & 1) : 0));

  const float norm = __fdiv_rn(1.0f, __fsqrt_rn(static_cast<float>(B)));
  float inv = norm;
  if (!CALIB && !PER_TOKEN) inv = __fdiv_rn(norm, __ldg(s_a_in));
  float cal_max = 0.0f, cal_lo = INFINITY, cal_hi = -INFINITY;
  const int zp = (ZP && !CALIB) ? __ldg(zp_in) - 8 : 0;
  [[maybe_unused]] const bool out32 = (reinterpret_cast<uintptr_t>(xq) & 31) == 0;

  // words of a tensor with the element pitch of x, in the order the MMAs take them: wa[tau][m3 | k3 << 1]
  auto load_words = [&](const __nv_bfloat16* base, bool on, uint32_t (&wa)[8][4]) {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(base + e_thr);
#pragma unroll
    for (int tau = 0; tau < 8; ++tau)
#pragma unroll
      for (int v = 0; v < 4; ++v)
        wa[tau][v] = on ? __ldg(src + ((tau << TAUS) | ((v & 1) << M3S) | ((v >> 1) << K3S)) / 2) : 0u;
  };

  const int64_t gb_step = static_cast<int64_t>(gridDim.x) * G;
  const int64_t row_step = gb_step / blocks_per_row, blk_step = gb_step % blocks_per_row;
  int64_t gb = static_cast<int64_t>(blockIdx.x) * G + blk_local;
  int64_t row_it = gb / blocks_per_row, blk_it = gb % blocks_per_row;
  // The words of an iteration are requested during the one before, as soon as its MMAs have taken theirs out of
  // the same registers: the rest of that iteration (some 600 instructions) covers the latency.
  uint32_t w[8][4];
  if (static_cast<int64_t>(blockIdx.x) < n_super) load_words(x + row_it * ldx + blk_it * B, gb < total_blocks, w);
  for (int64_t sb = blockIdx.x; sb < n_super; sb += gridDim.x) {
    const bool active = gb < total_blocks;
    const int64_t row = active ? row_it : 0;
    const int64_t col0 = active ? blk_it * B : 0;
    if (!CALIB && PER_TOKEN && s_a_out == nullptr) {
      const float s_row = __ldg(s_a_in + row);
      inv = __fdiv_rn(norm, s_row == 0.0f ? 1.0f : s_row);
    }
    [[maybe_unused]] uint32_t u[8][4];
    if (SWIGLU) load_words(x2 + row * ldx + col0, active, u);
    gb += gb_step, row_it += row_step, blk_it += blk_step;
    if (blk_it >= blocks_per_row) blk_it -= blocks_per_row, ++row_it;
    const bool more = sb + gridDim.x < n_super;

    if (SWIGLU) {
#pragma unroll
      for (int tau = 0; tau < 8; ++tau)
#pragma unroll
        for (int v = 0; v < 4; ++v)
          w[tau][v] = pack_bf16x2(pq::silu_mul_f32(__uint_as_float(w[tau][v] << 16), __uint_as_float(u[tau][v] << 16)),
                                  pq::silu_mul_f32(__uint_as_float(w[tau][v] & 0xFFFF0000u), __uint_as_float(u[tau][v] & 0xFFFF0000u)));
    } else if (NORM) {
      // sum of squares of the row in a fixed order: the thread's values, the warp's lanes, the block's warps
      float ss = 0.0f;
#pragma unroll
      for (int tau = 0; tau < 8; ++tau)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const float a = __uint_as_float(w[tau][v] << 16), b = __uint_as_float(w[tau][v] & 0xFFFF0000u);
          ss = __fmaf_rn(a, a, __fmaf_rn(b, b, ss));
        }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (WPB > 1) {
        if (lane == 0) norm_red[warp] = ss;
        __syncthreads();
        ss = 0.0f;
#pragma unroll
        for (int i = 0; i < WPB; ++i) ss += norm_red[blk_local * WPB + i];
        __syncthreads();
      }
      const float rr = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(ss, static_cast<float>(B)), clip)));
      uint32_t g_w[8][4];
      load_words(x2 + col0, true, g_w);
#pragma unroll
      for (int tau = 0; tau < 8; ++tau)
#pragma unroll
        for (int v = 0; v < 4; ++v)
          w[tau][v] = pack_bf16x2(__fmul_rn(__fmul_rn(__uint_as_float(w[tau][v] << 16), rr), __uint_as_float(g_w[tau][v] << 16)),
                                  __fmul_rn(__fmul_rn(__uint_as_float(w[tau][v] & 0xFFFF0000u), rr), __uint_as_float(g_w[tau][v] & 0xFFFF0000u)));
      if (NORM == 2) {
        if (active) {
          uint32_t* drow = reinterpret_cast<uint32_t*>(reinterpret_cast<__nv_bfloat16*>(xq) + row * n_cand + col0 + e_thr);
#pragma unroll
          for (int tau = 0; tau < 8; ++tau)
#pragma unroll
            for (int v = 0; v < 4; ++v) drow[((tau << TAUS) | ((v & 1) << M3S) | ((v >> 1) << K3S)) / 2] = w[tau][v];
        }
        if (more) load_words(x + row_it * ldx + blk_it * B, gb < total_blocks, w);
        continue;
      }
    }

    // ---- tensor-core stage on bits {0, 6, 7, k3}; V[m3 | tau << 1][nb] = the pair (n0 = 0, 1) ---------------
    float2 V[16][2];
#pragma unroll
    for (int tau = 0; tau < 8; ++tau)
#pragma unroll
      for (int nb = 0; nb < 2; ++nb) {
        float d[4];
        mma_bf16_m16n8k16(d, w[tau], hb[nb][0], hb[nb][1]);
        V[2 * tau][nb] = make_float2(d[0], d[1]);
        V[2 * tau + 1][nb] = make_float2(d[2], d[3]);
      }
    if (more) load_words(x + row_it * ldx + blk_it * B, gb < total_blocks, w);
#pragma unroll
    for (int s = 0; s < 4; ++s)
#pragma unroll
      for (int c = 0; c < 16; ++c)
        if ((c & (1 << s)) == 0) {
          const int c2 = c | (1 << s);
#pragma unroll
          for (int nb = 0; nb < 2; ++nb) {
            const float2 a = V[c][nb], b = V[c2][nb];
            V[c][nb] = __fadd2_rn(a, b);
            V[c2][nb] = __ffma2_rn(b, make_float2(-1.0f, -1.0f), a);
          }
        }
    // ---- exchange ----------------------------------------------------------------------------------------
#pragma unroll
    for (int nb = 0; nb < 2; ++nb)
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const int m3 = c & 1, tau = c >> 1;
        *reinterpret_cast<float2*>(my + wthr + ((m3 << M3S) | (nb << K3S) | (tau << TAUS)) + PADK * (m3 | (nb << 1) | (tau << 2))) = V[c][nb];
      }
    block_sync();
    // ---- pass 2: W[q] = elements 64 hi + 2q, 2q + 1; stages on bits J+1..5 ----------------------------------
    float2 W[32];
    {
      const float* src = my + rthr;
#pragma unroll
      for (int cc = 0; cc < 16; ++cc) {
        const float4 v = *reinterpret_cast<const float4*>(src + 4 * cc);
        W[2 * cc] = make_float2(v.x, v.y);
        W[2 * cc + 1] = make_float2(v.z, v.w);
      }
    }
    block_sync();
#pragma unroll
    for (int j = J; j < 5; ++j)
#pragma unroll
      for (int q = 0; q < 32; ++q)
        if ((q & (1 << j)) == 0) {
          const int q2 = q | (1 << j);
          const float2 a = W[q], b = W[q2];
          W[q] = __fadd2_rn(a, b);
          W[q2] = __ffma2_rn(b, make_float2(-1.0f, -1.0f), a);
        }
    const int64_t e0 = col0 + (hi << 6);  // first of this thread's 64 consecutive elements in the row
    if (!CALIB && PER_TOKEN && s_a_out != nullptr) {
      // One-pass dynamic form (the row is this one block): the token's step from the block's own maximum, in the
      // operations of the two-pass form (max of |y| * norm, then clip * max / 7: monotone, so the maximum over the
      // warps of the warps' steps is the step of the maximum), written out for the GEMM's epilogue.
      float it_max = 0.0f;
#pragma unroll
      for (int q = 0; q < 32; ++q) it_max = fmaxf(it_max, fmaxf(fabsf(W[q].x * norm), fabsf(W[q].y * norm)));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) it_max = fmaxf(it_max, __shfl_xor_sync(0xffffffffu, it_max, o));
      if (WPB > 1) {
        if (lane == 0) norm_red[warp] = it_max;
        __syncthreads();
        it_max = 0.0f;
#pragma unroll
        for (int i = 0; i < WPB; ++i) it_max = fmaxf(it_max, norm_red[blk_local * WPB + i]);
        __syncthreads();
      }
      const float s_row = it_max > 0.0f ? __fdiv_rn(it_max * clip, static_cast<float>(QMAX)) : 0.0f;
      if (active && hi == 0) s_a_out[row] = s_row;
      inv = __fdiv_rn(norm, s_row == 0.0f ? 1.0f : s_row);
    }
    if (CALIB) {
      float it_max = 0.0f;
      if (active) {
#pragma unroll
        for (int q = 0; q < 32; ++q) it_max = fmaxf(it_max, fmaxf(fabsf(W[q].x * norm), fabsf(W[q].y * norm)));
      }
      if (GRID) {
        double* sse = reinterpret_cast<double*>(s_a_out);
#pragma unroll 1
        for (int c = 0; c < n_cand; ++c) {
          float s, z;
          if (PER_TOKEN) {
            const float s_row = __ldg(s_a_in + row);
            s = s_row == 0.0f ? 1.0f : __fmul_rn(__ldg(reinterpret_cast<const float*>(x2) + c), s_row), z = 8.0f;
          } else {
            s = __ldg(s_a_in + c), z = static_cast<float>(__ldg(zp_in + c));
          }
          const float inv_s = __fdiv_rn(1.0f, s);
          float acc = 0.0f;
          if (active) {
#pragma unroll
            for (int q = 0; q < 32; ++q) {
              const float a = W[q].x * norm, b = W[q].y * norm;
              const float ua = fminf(fmaxf(rintf(a * inv_s) + z, 0.0f), 15.0f), ub = fminf(fmaxf(rintf(b * inv_s) + z, 0.0f), 15.0f);
              const float ea = a - s * (ua - z), eb = b - s * (ub - z);
              acc = fmaf(ea, ea, acc);
              acc = fmaf(eb, eb, acc);
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
          if (lane == 0 && acc != 0.0f) atomicAdd(sse + c, static_cast<double>(acc));
        }
      } else if (ZP) {
        if (active) {
#pragma unroll
          for (int q = 0; q < 32; ++q) {
            const float a = W[q].x * norm, b = W[q].y * norm;
            cal_lo = fminf(cal_lo, fminf(a, b)), cal_hi = fmaxf(cal_hi, fmaxf(a, b));
          }
        }
      } else if (PER_TOKEN) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) it_max = fmaxf(it_max, __shfl_xor_sync(0xffffffffu, it_max, o));
        if (lane == 0 && active && it_max > 0.0f)
          atomicMax(reinterpret_cast<int*>(s_a_out + row), __float_as_int(__fdiv_rn(it_max * clip, static_cast<float>(QMAX))));
      } else {
        cal_max = fmaxf(cal_max, it_max);
      }
    } else {
      // ---- quantize and pack ---------------------------------------------------------------------------
      // The offset code u = clamp(rne(y / s) + 2^(BITS-1), 0, 2^BITS - 1) is taken in two fused multiply-adds:
      // f = sat(y * (inv / U) + 2^(BITS-1) / U) with U = 2^BITS - 1 is (y / s + 2^(BITS-1)) / U clamped to [0, 1] (the
      // clamp of the code range, applied before the rounding, which gives the same code), and f * U + 1.5 * 2^23
      // leaves rne(f * U) in the low mantissa bits. f carries one more rounding (2^-25 of the code range, i.e.
      // 5e-7 of a step for 4 bits, 8e-6 for 8 bits), far inside the distance from a tie within which a code may
      // differ from a double-precision evaluation. u ^ 2^(BITS-1) is the two's-complement code.
      // With a zero point (odd z would move ties) the rounding comes first: y * inv + (1.5 * 2^23 + 8), the integer
      // z - 8 added to the bit pattern, and an integer clamp.
      constexpr int BASE = 0x4B400000;
      // byte stores with a narrower code range (4-bit codes, one per byte): the caller's largest code in n_cand
      const int qmax = (BITS == 8 && n_cand > 0) ? n_cand : QMAX;
      const float U = static_cast<float>(2 * qmax + 1);
      const float invU = __fdiv_rn(inv, U), offU = __fdiv_rn(static_cast<float>(qmax + 1), U);
      auto codes = [&](float2 y) -> uint2 {  // bit patterns whose low BITS bits are the two offset codes
        if (ZP) {
          const float2 tq = __ffma2_rn(y, make_float2(inv, inv), make_float2(12582920.0f, 12582920.0f));
          return make_uint2(static_cast<uint32_t>(max(min(__float_as_int(tq.x) + zp, BASE + 15), BASE)),
                            static_cast<uint32_t>(max(min(__float_as_int(tq.y) + zp, BASE + 15), BASE)));
        }
        float fx, fy;
        asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(fx) : "f"(y.x), "f"(invU), "f"(offU));
        asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(fy) : "f"(y.y), "f"(invU), "f"(offU));
        const float2 tq = __ffma2_rn(make_float2(fx, fy), make_float2(U, U), make_float2(12582912.0f, 12582912.0f));
        return make_uint2(__float_as_uint(tq.x), __float_as_uint(tq.y));
      };
      // a thread's 32 bytes leave as one sector when the output is 32-byte aligned (rows are whole kilobytes)
      auto store32 = [&](uint8_t* dst, const uint32_t* v) {
        if (out32) {
          asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]),
                       "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                       : "memory");
        } else {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(v[0], v[1], v[2], v[3]);
          reinterpret_cast<uint4*>(dst)[1] = make_uint4(v[4], v[5], v[6], v[7]);
        }
      };
      if (BITS == 4) {
        uint32_t fin[8];
#pragma unroll
        for (int wd = 0; wd < 8; ++wd) {
          uint32_t pb[4];  // low byte: the codes of two neighbouring elements
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            const uint2 c = codes(W[4 * wd + b]);
            pb[b] = c.x + (c.y << 4);
          }
          fin[wd] = __byte_perm(__byte_perm(pb[0], pb[1], 0x0040), __byte_perm(pb[2], pb[3], 0x0040), 0x5410) ^ 0x88888888u;
        }
        if (active) store32(xq + row * (K / 2) + e0 / 2, fin);
      } else {
        uint32_t fin[16];
#pragma unroll
        for (int wd = 0; wd < 16; ++wd) {
          const uint2 c0 = codes(W[2 * wd]), c1 = codes(W[2 * wd + 1]);
          // offset codes u = n + qmax + 1 -> signed bytes n (for the full range this is u ^ 0x80)
          fin[wd] = __vsub4(__byte_perm(__byte_perm(c0.x, c0.y, 0x0040), __byte_perm(c1.x, c1.y, 0x0040), 0x5410),
                            static_cast<uint32_t>(qmax + 1) * 0x01010101u);
        }
        if (active) {
          store32(xq + row * K + e0, fin);
          store32(xq + row * K + e0 + 32, fin + 8);
        }
      }
    }
  }
  if (CALIB && GRID) {
  } else if (CALIB && ZP) {
    for (int o = 16; o > 0; o >>= 1) {
      cal_lo = fminf(cal_lo, __shfl_xor_sync(0xffffffffu, cal_lo, o));
      cal_hi = fmaxf(cal_hi, __shfl_xor_sync(0xffffffffu, cal_hi, o));
    }
    if (lane == 0 && cal_hi >= cal_lo) {
      atomicMax(reinterpret_cast<uint32_t*>(s_a_out), float_key(cal_hi));
      atomicMin(reinterpret_cast<uint32_t*>(s_a_out) + 1, float_key(cal_lo));
    }
  } else if (CALIB && !PER_TOKEN) {
    for (int o = 16; o > 0; o >>= 1) cal_max = fmaxf(cal_max, __shfl_xor_sync(0xffffffffu, cal_max, o));
    if (lane == 0 && cal_max > 0.0f)
      atomicMax(reinterpret_cast<int*>(s_a_out), __float_as_int(__fdiv_rn(cal_max, static_cast<float>(QMAX))));
  }
}

template <int LOGB, bool ROTATE, bool CALIB, int BITS, bool PER_TOKEN, bool ZP, bool SWIGLU, bool GRID, int NORM = 0>
pq_status launch(pq_ctx* ctx, const void* x, int64_t ldx, int64_t n_rows, int64_t K, const float* s_a_in, uint8_t* xq,
                 float* s_a_out, float clip, const int32_t* zp_in, const void* x2, cudaStream_t st, int n_cand) {
  constexpr int B = 1 << LOGB;
  constexpr int G = HQ_THREADS / (B / 64);
  int64_t n_super = (n_rows * (K / B) + G - 1) / G;
  // blocks of 2048 and wider take the kernel whose first stages run on the tensor cores
  constexpr bool WIDE = LOGB >= 11 && (ROTATE || NORM == 2);
  void (*kern)(const __nv_bfloat16*, int64_t, int64_t, int64_t, const float*, uint8_t*, float*, float, const int32_t*,
               const __nv_bfloat16*, int);
  size_t smem = HQ_SMEM_FLOATS * sizeof(float);
  int ctas_per_sm = HQ_CTAS_PER_SM;
  if constexpr (WIDE) {
    kern = hadamard_quant_wide_kernel<LOGB, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID, NORM>;
    smem = HQW_SMEM_FLOATS * sizeof(float);
    ctas_per_sm = HQW_CTAS_PER_SM;
  } else {
    kern = hadamard_quant_kernel<LOGB, ROTATE, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID, NORM>;
  }
  // the shared-memory attribute is set once per device and instantiation (the call costs several microseconds of
  // host time, a visible share of a decode-sized launch)
  static bool attr_set[64] = {};
  const int dev = ctx->device;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
      return PQ_ERR_CUDA;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const int64_t resident = static_cast<int64_t>(ctas_per_sm) * ctx->sm_count;
  int64_t grid = n_super < resident ? n_super : resident;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(HQ_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  // may be launched while the previous kernel drains; waits for it on the device before touching memory
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, static_cast<const __nv_bfloat16*>(x), ldx, n_rows, K, s_a_in, xq, s_a_out, clip, zp_in,
                         static_cast<const __nv_bfloat16*>(x2), n_cand) != cudaSuccess)
    return PQ_ERR_CUDA;
  return pq_launch_status();
}

template <bool CALIB, int BITS, bool PER_TOKEN = false, bool ZP = false, bool SWIGLU = false, bool GRID = false>
pq_status dispatch(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block, int64_t row_begin,
                   const float* s_a_in, uint8_t* xq, float* s_a_out, void* stream, float clip = 1.0f,
                   const int32_t* zp_in = nullptr, const void* x2 = nullptr, int n_cand = 0) {
  if ((SWIGLU || (GRID && PER_TOKEN)) && (!x2 || (reinterpret_cast<uintptr_t>(x2) & 3))) return x2 ? PQ_ERR_ALIGN : PQ_ERR_INVALID_ARG;
  if (!ctx || !x || (!CALIB && ((!s_a_in && !s_a_out) || !xq)) || (CALIB && !s_a_out)) return PQ_ERR_INVALID_ARG;
  if (M < 0 || K <= 0 || ldx < K || row_begin < 0 || had_block < 0) return PQ_ERR_INVALID_ARG;
  if (K % 128 != 0) return PQ_ERR_SHAPE;
  if (had_block != 0) {
    if ((had_block & (had_block - 1)) != 0 || had_block < 128 || had_block > 8192 || K % had_block != 0)
      return PQ_ERR_SHAPE;
  }
  if ((ldx & 1) || (reinterpret_cast<uintptr_t>(x) & 3)) return PQ_ERR_ALIGN;
  if (!CALIB && (reinterpret_cast<uintptr_t>(xq) & 15)) return PQ_ERR_ALIGN;
  if (row_begin >= M) return PQ_OK;
  const int64_t n_rows = M - row_begin;
  const void* x0 = static_cast<const __nv_bfloat16*>(x) + row_begin * ldx;
  const void* x20 = SWIGLU ? static_cast<const __nv_bfloat16*>(x2) + row_begin * ldx : ((GRID && PER_TOKEN) ? x2 : nullptr);
  uint8_t* xq0 = CALIB ? nullptr : xq + row_begin * (BITS == 4 ? K / 2 : K);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (PER_TOKEN) {  // the arrays are indexed by row (not the error sums of the grid search)
    if (s_a_in) s_a_in += row_begin;
    if (s_a_out && !GRID) s_a_out += row_begin;
    if (CALIB && !GRID && cudaMemsetAsync(s_a_out, 0, static_cast<size_t>(n_rows) * sizeof(float), st) != cudaSuccess) return PQ_ERR_CUDA;
  }
  switch (had_block) {
    case 0: return launch<7, false, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    case 128: return launch<7, true, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    case 256: return launch<8, true, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    case 512: return launch<9, true, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    case 1024: return launch<10, true, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    case 2048: return launch<11, true, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    case 4096: return launch<12, true, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    case 8192: return launch<13, true, CALIB, BITS, PER_TOKEN, ZP, SWIGLU, GRID>(ctx, x0, ldx, n_rows, K, s_a_in, xq0, s_a_out, clip, zp_in, x20, st, n_cand);
    default: return PQ_ERR_SHAPE;
  }
}

}  // namespace

extern "C" pq_status pq_hadamard_quant_act(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx,
                                           int had_block, int64_t row_begin, const float* s_a, uint8_t* xq,
                                           void* stream) {
  return dispatch<false, 4>(ctx, x, M, K, ldx, had_block, row_begin, s_a, xq, nullptr, stream);
}

extern "C" pq_status pq_calib_act_scale(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                        int64_t row_begin, float* s_a, void* stream) {
  return dispatch<true, 4>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, nullptr, s_a, stream);
}

extern "C" pq_status pq_hadamard_quant_act8(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx,
                                            int had_block, int64_t row_begin, const float* s_a, int8_t* xq8,
                                            void* stream) {
  return dispatch<false, 8>(ctx, x, M, K, ldx, had_block, row_begin, s_a, reinterpret_cast<uint8_t*>(xq8), nullptr, stream);
}

// 4-bit codes stored one per byte (the range of pq_hadamard_quant_act, the layout of pq_hadamard_quant_act8).
extern "C" pq_status pq_hadamard_quant_act_c8(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx,
                                              int had_block, int64_t row_begin, const float* s_a, int8_t* xq8,
                                              void* stream) {
  return dispatch<false, 8>(ctx, x, M, K, ldx, had_block, row_begin, s_a, reinterpret_cast<uint8_t*>(xq8), nullptr, stream, 1.0f,
                            nullptr, nullptr, 7);
}

extern "C" pq_status pq_calib_act_scale8(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                         int64_t row_begin, float* s_a, void* stream) {
  return dispatch<true, 8>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, nullptr, s_a, stream);
}

// ---- per-token dynamic activations (Table 1, O1): the step of a row is computed online from the row ----
extern "C" pq_status pq_dyn_act_scale(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                      int64_t row_begin, float clip, float* s_tok, void* stream) {
  if (!(clip > 0.0f) || !(clip <= 1.0f)) return PQ_ERR_INVALID_ARG;
  return dispatch<true, 4, true>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, nullptr, s_tok, stream, clip);
}

extern "C" pq_status pq_hadamard_quant_act_rows(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx,
                                                int had_block, int64_t row_begin, const float* s_tok, uint8_t* xq,
                                                void* stream) {
  return dispatch<false, 4, true>(ctx, x, M, K, ldx, had_block, row_begin, s_tok, xq, nullptr, stream);
}

// Both in one call. When a row is one transform block of 2048 or more elements the step is formed and used in the
// same pass over the activations (one launch); else the two passes above.
extern "C" pq_status pq_dyn_hadamard_quant_act(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                               int64_t row_begin, float clip, float* s_tok, uint8_t* xq, void* stream) {
  if (!(clip > 0.0f) || !(clip <= 1.0f) || !s_tok) return PQ_ERR_INVALID_ARG;
  if (had_block == K && had_block >= 2048)
    return dispatch<false, 4, true>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, xq, s_tok, stream, clip);
  pq_status rc = dispatch<true, 4, true>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, nullptr, s_tok, stream, clip);
  if (rc != PQ_OK) return rc;
  return dispatch<false, 4, true>(ctx, x, M, K, ldx, had_block, row_begin, s_tok, xq, nullptr, stream);
}

// ---- Eq. 1 with its zero point: asymmetric static per-tensor quantizer -----------------------------------
namespace {
// Max-min initialisation (gamma = beta = 1) from the collected range: s = (mx - mn) / 15, z = -floor(mn / s)
// (Eq. 1 prints the zero point with a floor), every step one IEEE fp32 operation; a constant (or empty) range
// gives s = 1, z = 0.
__global__ void asym_params_kernel(uint32_t* keys, float* s_a, int32_t* z_a) {
  const float mx = key_float(keys[0]), mn = key_float(keys[1]);
  float s = 1.0f;
  int z = 0;
  if (keys[0] >= keys[1] && mx > mn) {
    s = __fdiv_rn(__fsub_rn(mx, mn), 15.0f);
    z = -__float2int_rd(__fdiv_rn(mn, s));
    z = z < 0 ? 0 : (z > 15 ? 15 : z);
  }
  *s_a = s;
  *z_a = z;
}
constexpr int ASYM_KEY0 = 8;  // two words of the context's counter array hold the range keys during a call
}  // namespace

extern "C" pq_status pq_calib_act_asym(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                       int64_t row_begin, float* s_a, int32_t* z_a, void* stream) {
  if (!ctx || !s_a || !z_a) return PQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* keys = ctx->d_tickets + ASYM_KEY0;
  if (cudaMemsetAsync(keys, 0x00, sizeof(uint32_t), st) != cudaSuccess ||
      cudaMemsetAsync(keys + 1, 0xFF, sizeof(uint32_t), st) != cudaSuccess)
    return PQ_ERR_CUDA;
  pq_status rc = dispatch<true, 4, false, true>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, nullptr,
                                                reinterpret_cast<float*>(keys), stream);
  if (rc != PQ_OK) return rc;
  asym_params_kernel<<<1, 1, 0, st>>>(keys, s_a, z_a);
  return pq_launch_status();
}

namespace {
// The n x n candidates of the clipping-factor grid from the collected range, every step one IEEE fp32 operation:
// gamma_i = 1 - i * step, beta_j = 1 - j * step, s = (gamma mx - beta mn) / 15, z = -floor(beta mn / s) in [0, 15].
__global__ void grid_candidates_kernel(const uint32_t* keys, int n, float lo, float* cand_s, int32_t* cand_z) {
  const int c = threadIdx.x;
  if (c >= n * n) return;
  const float mx = key_float(keys[0]), mn = key_float(keys[1]);
  const bool have = keys[0] >= keys[1];
  const float step = n > 1 ? __fdiv_rn(__fsub_rn(1.0f, lo), static_cast<float>(n - 1)) : 0.0f;
  const float gamma = __fsub_rn(1.0f, __fmul_rn(static_cast<float>(c / n), step));
  const float beta = __fsub_rn(1.0f, __fmul_rn(static_cast<float>(c % n), step));
  const float bm = __fmul_rn(beta, mn), d = __fsub_rn(__fmul_rn(gamma, mx), bm);
  float s = 1.0f;
  int z = 0;
  if (have && d > 0.0f) {
    s = __fdiv_rn(d, 15.0f);
    z = -__float2int_rd(__fdiv_rn(bm, s));
    z = z < 0 ? 0 : (z > 15 ? 15 : z);
  }
  cand_s[c] = s, cand_z[c] = z;
}
// The candidate with the smallest error, the first one among equals.
__global__ void grid_argmin_kernel(const double* sse, const float* cand_s, const int32_t* cand_z, int n_cand, float* s_a, int32_t* z_a) {
  int best = 0;
  for (int c = 1; c < n_cand; ++c)
    if (sse[c] < sse[best]) best = c;
  *s_a = cand_s[best], *z_a = cand_z[best];
}
}  // namespace

extern "C" pq_status pq_grid_search_act_asym(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                             int64_t row_begin, int32_t n_grid, float lo, float* s_a, int32_t* z_a, float* cand_s,
                                             int32_t* cand_z, double* sse, void* stream) {
  if (!ctx || !s_a || !z_a || !cand_s || !cand_z || !sse) return PQ_ERR_INVALID_ARG;
  if (n_grid < 1 || n_grid > 16 || !(lo > 0.0f) || !(lo <= 1.0f)) return PQ_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(sse) & 7) return PQ_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_cand = n_grid * n_grid;
  uint32_t* keys = ctx->d_tickets + ASYM_KEY0;
  if (cudaMemsetAsync(keys, 0x00, sizeof(uint32_t), st) != cudaSuccess || cudaMemsetAsync(keys + 1, 0xFF, sizeof(uint32_t), st) != cudaSuccess ||
      cudaMemsetAsync(sse, 0, sizeof(double) * n_cand, st) != cudaSuccess)
    return PQ_ERR_CUDA;
  pq_status rc = dispatch<true, 4, false, true>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, nullptr, reinterpret_cast<float*>(keys), stream);
  if (rc != PQ_OK) return rc;
  grid_candidates_kernel<<<1, 256, 0, st>>>(keys, n_grid, lo, cand_s, cand_z);
  if (pq_launch_status() != PQ_OK) return PQ_ERR_CUDA;
  rc = dispatch<true, 4, false, true, false, true>(ctx, x, M, K, ldx, had_block, row_begin, cand_s, nullptr, reinterpret_cast<float*>(sse), stream,
                                                   1.0f, cand_z, nullptr, n_cand);
  if (rc != PQ_OK) return rc;
  grid_argmin_kernel<<<1, 1, 0, st>>>(sse, cand_s, cand_z, n_cand, s_a, z_a);
  return pq_launch_status();
}

namespace {
__global__ void clip_candidates_kernel(int n, float lo, float* cand) {
  const int i = threadIdx.x;
  if (i >= n) return;
  const float step = n > 1 ? __fdiv_rn(__fsub_rn(1.0f, lo), static_cast<float>(n - 1)) : 0.0f;
  cand[i] = __fsub_rn(1.0f, __fmul_rn(static_cast<float>(i), step));
}
__global__ void clip_argmin_kernel(const double* sse, const float* cand, int n, float* gamma) {
  int best = 0;
  for (int c = 1; c < n; ++c)
    if (sse[c] < sse[best]) best = c;
  *gamma = cand[best];
}
}  // namespace

extern "C" pq_status pq_grid_search_clip_dyn(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, int had_block,
                                             int64_t row_begin, int32_t n_grid, float lo, float* gamma, float* s_tok, float* cand,
                                             double* sse, void* stream) {
  if (!ctx || !gamma || !s_tok || !cand || !sse) return PQ_ERR_INVALID_ARG;
  if (n_grid < 1 || n_grid > 256 || !(lo > 0.0f) || !(lo <= 1.0f)) return PQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(sse) & 7) || (reinterpret_cast<uintptr_t>(cand) & 3)) return PQ_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(sse, 0, sizeof(double) * n_grid, st) != cudaSuccess) return PQ_ERR_CUDA;
  // every row's unclipped step, then one pass that quantizes with each candidate's multiple of it
  pq_status rc = dispatch<true, 4, true>(ctx, x, M, K, ldx, had_block, row_begin, nullptr, nullptr, s_tok, stream, 1.0f);
  if (rc != PQ_OK) return rc;
  clip_candidates_kernel<<<1, 256, 0, st>>>(n_grid, lo, cand);
  if (pq_launch_status() != PQ_OK) return PQ_ERR_CUDA;
  rc = dispatch<true, 4, true, false, false, true>(ctx, x, M, K, ldx, had_block, row_begin, s_tok, nullptr, reinterpret_cast<float*>(sse), stream,
                                                   1.0f, nullptr, cand, n_grid);
  if (rc != PQ_OK) return rc;
  clip_argmin_kernel<<<1, 1, 0, st>>>(sse, cand, n_grid, gamma);
  return pq_launch_status();
}

extern "C" pq_status pq_hadamard_quant_act_asym(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx,
                                                int had_block, int64_t row_begin, const float* s_a, const int32_t* z_a,
                                                uint8_t* xq, void* stream) {
  if (!z_a) return PQ_ERR_INVALID_ARG;
  return dispatch<false, 4, false, true>(ctx, x, M, K, ldx, had_block, row_begin, s_a, xq, nullptr, stream, 1.0f, z_a);
}

// ---- RMSNorm in front of the rotation (the block's first linears): the row is one transform block ----------
namespace {
template <int NORM>
pq_status dispatch_norm(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, const void* g, float eps, int64_t row_begin,
                        const float* s_a, void* dst, int64_t ld_dst, void* stream) {
  if (!ctx || !x || !g || !dst || (NORM == 1 && !s_a)) return PQ_ERR_INVALID_ARG;
  if (M < 0 || K <= 0 || ldx < K || row_begin < 0 || (NORM == 2 && ld_dst < K)) return PQ_ERR_INVALID_ARG;
  if ((K & (K - 1)) != 0 || K < 128 || K > 8192) return PQ_ERR_SHAPE;
  if ((ldx & 1) || (reinterpret_cast<uintptr_t>(x) & 3) || (reinterpret_cast<uintptr_t>(g) & 3)) return PQ_ERR_ALIGN;
  if (NORM == 1 && (reinterpret_cast<uintptr_t>(dst) & 15)) return PQ_ERR_ALIGN;
  if (NORM == 2 && ((ld_dst & 1) || (reinterpret_cast<uintptr_t>(dst) & 3))) return PQ_ERR_ALIGN;
  if (row_begin >= M) return PQ_OK;
  const int64_t n_rows = M - row_begin;
  const void* x0 = static_cast<const __nv_bfloat16*>(x) + row_begin * ldx;
  uint8_t* d0 = NORM == 1 ? static_cast<uint8_t*>(dst) + row_begin * (K / 2)
                          : reinterpret_cast<uint8_t*>(static_cast<__nv_bfloat16*>(dst) + row_begin * ld_dst);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int ld = static_cast<int>(ld_dst);
  constexpr bool R = NORM == 1;
  switch (K) {
    case 128: return launch<7, R, false, 4, false, false, false, false, NORM>(ctx, x0, ldx, n_rows, K, s_a, d0, nullptr, eps, nullptr, g, st, ld);
    case 256: return launch<8, R, false, 4, false, false, false, false, NORM>(ctx, x0, ldx, n_rows, K, s_a, d0, nullptr, eps, nullptr, g, st, ld);
    case 512: return launch<9, R, false, 4, false, false, false, false, NORM>(ctx, x0, ldx, n_rows, K, s_a, d0, nullptr, eps, nullptr, g, st, ld);
    case 1024: return launch<10, R, false, 4, false, false, false, false, NORM>(ctx, x0, ldx, n_rows, K, s_a, d0, nullptr, eps, nullptr, g, st, ld);
    case 2048: return launch<11, R, false, 4, false, false, false, false, NORM>(ctx, x0, ldx, n_rows, K, s_a, d0, nullptr, eps, nullptr, g, st, ld);
    case 4096: return launch<12, R, false, 4, false, false, false, false, NORM>(ctx, x0, ldx, n_rows, K, s_a, d0, nullptr, eps, nullptr, g, st, ld);
    case 8192: return launch<13, R, false, 4, false, false, false, false, NORM>(ctx, x0, ldx, n_rows, K, s_a, d0, nullptr, eps, nullptr, g, st, ld);
    default: return PQ_ERR_SHAPE;
  }
}
}  // namespace

extern "C" pq_status pq_rmsnorm_hadamard_quant_act(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, const void* g, float eps,
                                                   int64_t row_begin, const float* s_a, uint8_t* xq, void* stream) {
  return dispatch_norm<1>(ctx, x, M, K, ldx, g, eps, row_begin, s_a, xq, 0, stream);
}

// The stand-alone RMSNorm of a row that is one transform block (K a power of two up to 8192): the same first pass.
pq_status pq_rmsnorm_pow2_launch(pq_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, const void* g, float eps, void* y,
                                 int64_t ldy, void* stream) {
  return dispatch_norm<2>(ctx, x, M, K, ldx, g, eps, 0, nullptr, y, ldy, stream);
}

// ---- SwiGLU fused into the rotation of the down projection's input (App. B: R4 sits between the two) ------
extern "C" pq_status pq_swiglu_hadamard_quant_act(pq_ctx* ctx, const void* gate, const void* up, int64_t M, int64_t K,
                                                  int64_t ld_in, int had_block, int64_t row_begin, const float* s_a,
                                                  uint8_t* xq, void* stream) {
  return dispatch<false, 4, false, false, true>(ctx, gate, M, K, ld_in, had_block, row_begin, s_a, xq, nullptr, stream, 1.0f,
                                                nullptr, up);
}

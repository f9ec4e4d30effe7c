// CPU oracle for the PrefixQuant W4A4KV4 inference path (static setting, "O2" of Table 1).
//
// THIS IS TEST INFRASTRUCTURE. It is a plain, slow, scalar restatement of what the path
// computes, written from the paper; it shares no code with the CUDA library and nothing in
// the product path may call it. Only the tests, the smoke check and the bench's CPU-baseline
// legs load it.
//
// Conventions
//   * bf16 / fp16 tensors are passed as raw uint16 bit patterns, decoded exactly to double.
//   * All floating-point work is double, except weight and KV quantization, where the decision
//     that produces an integer code is taken in IEEE fp32 (division, round-half-even) because
//     that is the precision the GPU kernels use for the same decision (bf16 inputs, fp32 steps:
//     exact ties of x / (max/7) do occur, and only an equal-precision decision is reproducible).
//   * Packed INT4: element 2j in the low nibble, element 2j+1 in the high nibble, two's
//     complement, packed along the contraction (or head) dimension.
//   * Threading is over independent rows only; arithmetic per row is strictly sequential.
//
// Pins (see tests/test_oracle_pins.py): H H^T = n I, rotation of unit vectors / all-ones,
// involution, Parseval, comparison with a library-built Sylvester matrix product; quantizer
// range / ties / idempotence / hand-worked Eq. (1) values (4-bit and 8-bit); brute-force integer GEMMs;
// attention against closed forms and a library softmax-attention; RoPE against the complex
// rotation form; RMSNorm and SwiGLU closed forms.
// Readings fixed by the benchmark spec rather than the paper (symmetric max/7 scale,
// round-half-even, low-nibble-first, 2048-wide blocks) are "parity unpinned by the paper".

#include <algorithm>
#include <atomic>
#include <cfenv>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <thread>
#include <vector>

namespace {

int g_threads = 0;

int n_threads() {
  if (g_threads > 0) return g_threads;
  unsigned h = std::thread::hardware_concurrency();
  return h == 0 ? 1 : static_cast<int>(h);
}

// Run fn(i) for i in [0, n) on the host cores; rows are independent, so no ordering matters.
void parallel_rows(int64_t n, const std::function<void(int64_t)>& fn) {
  int nt = static_cast<int>(std::min<int64_t>(n_threads(), n));
  if (nt <= 1) {
    for (int64_t i = 0; i < n; ++i) fn(i);
    return;
  }
  std::atomic<int64_t> next{0};
  std::vector<std::thread> pool;
  for (int t = 0; t < nt; ++t)
    pool.emplace_back([&] {
      for (;;) {
        int64_t i = next.fetch_add(1);
        if (i >= n) break;
        fn(i);
      }
    });
  for (auto& th : pool) th.join();
}

double bf16_to_double(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return static_cast<double>(f);
}

double fp16_to_double(uint16_t h) {
  int sign = (h >> 15) & 1;
  int exp = (h >> 10) & 0x1f;
  int man = h & 0x3ff;
  double v;
  if (exp == 0)
    v = std::ldexp(static_cast<double>(man), -24);
  else if (exp == 31)
    v = man ? NAN : INFINITY;
  else
    v = std::ldexp(static_cast<double>(man + 1024), exp - 25);
  return sign ? -v : v;
}

// One rounding, double -> bf16, round-half-to-even (8 significant bits, fp32 exponent range).
uint16_t double_to_bf16(double x) {
  if (std::isnan(x)) return 0x7fc0;
  uint16_t sign = std::signbit(x) ? 0x8000 : 0;
  double a = std::fabs(x);
  if (a == 0.0) return sign;
  if (std::isinf(a)) return sign | 0x7f80;
  int e = std::ilogb(a);
  if (e < -126) e = -126;  // subnormal quantum
  double q = std::ldexp(a, 7 - e);
  double r = std::nearbyint(q);  // FE_TONEAREST: ties to even
  double v = std::ldexp(r, e - 7);
  float f = static_cast<float>(v);  // exact: v has <= 8 significant bits
  if (std::isinf(f)) return sign | 0x7f80;
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return sign | static_cast<uint16_t>(u >> 16);
}

inline int clampi(long v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : static_cast<int>(v)); }

inline int nib_get(const uint8_t* row, int64_t j) {
  uint8_t b = row[j >> 1];
  int n = (j & 1) ? (b >> 4) : (b & 0xf);
  return n >= 8 ? n - 16 : n;
}

inline void nib_set(uint8_t* row, int64_t j, int code) {
  uint8_t n = static_cast<uint8_t>(code & 0xf);
  uint8_t& b = row[j >> 1];
  if (j & 1)
    b = static_cast<uint8_t>((b & 0x0f) | (n << 4));
  else
    b = static_cast<uint8_t>((b & 0xf0) | n);
}

// Rotation of one row (App. B "Details of Rotation"): y = x H_B / sqrt(B) on each contiguous
// B-wide block, with the Sylvester-ordered matrix H[i][j] = (-1)^popcount(i & j), written as
// the matrix product itself. B == 0 means "no rotation".
void rotate_row(const double* x, double* y, int64_t K, int B) {
  if (B == 0) {
    for (int64_t j = 0; j < K; ++j) y[j] = x[j];
    return;
  }
  const double norm = 1.0 / std::sqrt(static_cast<double>(B));
  for (int64_t base = 0; base < K; base += B) {
    for (int j = 0; j < B; ++j) {
      double s = 0.0;
      for (int i = 0; i < B; ++i) {
        double v = x[base + i];
        s += (__builtin_popcount(static_cast<unsigned>(i & j)) & 1) ? -v : v;
      }
      y[base + j] = s * norm;
    }
  }
}

}  // namespace

extern "C" {

void orc_set_threads(int n) { g_threads = n; }
int orc_get_threads() { return n_threads(); }

// ---- format helpers exposed for the tests --------------------------------------------------
void orc_bf16_to_f64(const uint16_t* in, double* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_double(in[i]);
}
void orc_f64_to_bf16(const double* in, uint16_t* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = double_to_bf16(in[i]);
}
void orc_fp16_to_f64(const uint16_t* in, double* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = fp16_to_double(in[i]);
}
void orc_unpack_int4(const uint8_t* in, int8_t* out, int64_t rows, int64_t K) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t j = 0; j < K; ++j) out[r * K + j] = static_cast<int8_t>(nib_get(in + r * (K / 2), j));
}
void orc_pack_int4(const int8_t* in, uint8_t* out, int64_t rows, int64_t K) {
  std::memset(out, 0, static_cast<size_t>(rows * (K / 2)));
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t j = 0; j < K; ++j) nib_set(out + r * (K / 2), j, in[r * K + j]);
}

// ---- rotation (App. B) -----------------------------------------------------------------------
// x double [M,K] -> y double [M,K]; B = block width (power of two dividing K) or 0.
void orc_rotate_f64(const double* x, double* y, int64_t M, int64_t K, int B) {
  parallel_rows(M, [&](int64_t m) { rotate_row(x + m * K, y + m * K, K, B); });
}

// x bf16 [M,K] with row stride ldx (elements) -> y double [M,K].
void orc_rotate_bf16(const uint16_t* x, int64_t ldx, double* y, int64_t M, int64_t K, int B) {
  parallel_rows(M, [&](int64_t m) {
    std::vector<double> xr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), y + m * K, K, B);
  });
}

// ---- static per-tensor activation scale (Table 1, O2; Sec. 3 "Dynamic and Static") -----------
// s_a = fp32( max |fp32(y)| / 7 ) over rows >= row_begin of the rotated calibration batch:
// rows below row_begin are the prefixed outlier tokens and never take part.
float orc_calib_act_scale(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin) {
  std::vector<double> rowmax(M, 0.0);
  parallel_rows(M, [&](int64_t m) {
    if (m < row_begin) return;
    std::vector<double> xr(K), yr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    double mx = 0.0;
    for (int64_t j = 0; j < K; ++j) mx = std::max(mx, std::fabs(static_cast<double>(static_cast<float>(yr[j]))));
    rowmax[m] = mx;
  });
  double mx = 0.0;
  for (int64_t m = row_begin; m < M; ++m) mx = std::max(mx, rowmax[m]);
  if (mx == 0.0) return 1.0f;
  return static_cast<float>(mx / 7.0);
}

// ---- activation quantization (Eq. 1, symmetric signed form) ---------------------------------
// code = clamp(round_half_even(y / s_a), -8, 7), y the rotated row. Rows < row_begin are left
// untouched. tie_dist (nullable, [M,K] float) receives |y/s_a - nearest half-integer|, the
// distance of the pre-rounding value from the closest rounding tie.
void orc_quant_act(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, float s_a,
                   uint8_t* xq, float* tie_dist) {
  const double s = static_cast<double>(s_a);
  parallel_rows(M, [&](int64_t m) {
    if (m < row_begin) return;
    std::vector<double> xr(K), yr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    uint8_t* out = xq + m * (K / 2);
    for (int64_t j = 0; j < K; ++j) {
      double r = yr[j] / s;
      long c = std::lrint(std::nearbyint(r));
      nib_set(out, j, clampi(c, -8, 7));
      if (tie_dist) {
        double f = r - std::floor(r);  // in [0,1)
        tie_dist[m * K + j] = static_cast<float>(std::fabs(f - 0.5));
      }
    }
  });
}

// Plain quantizer on double inputs, for pins: code = clamp(rne(v / s), -8, 7).
void orc_quant_f64(const double* v, int64_t n, double s, int8_t* codes) {
  for (int64_t i = 0; i < n; ++i) codes[i] = static_cast<int8_t>(clampi(std::lrint(std::nearbyint(v[i] / s)), -8, 7));
}

// ---- weight quantization: RTN, one scale per output channel (Table 1; Table 6 "RTN") --------
// s_w[n] = fp32(max_k |W[n,k]|) / 7 in fp32 (1 if the row is all zero);
// code = clamp(rint_fp32(W[n,k] / s_w[n]), -8, 7) with an fp32 IEEE division.
// tie_dist (nullable, [N,K] float) receives | W / s_w - nearest half-integer | with the quotient taken in
// double: the distance of the exact pre-rounding value from the closest rounding tie, which bounds where
// the fp32 decision can differ from a double one.
void orc_quant_weights(const uint16_t* W, int64_t ldw, int64_t N, int64_t K, uint8_t* wq, float* s_w, float* tie_dist) {
  parallel_rows(N, [&](int64_t n) {
    float mx = 0.0f;
    for (int64_t k = 0; k < K; ++k) mx = std::max(mx, std::fabs(static_cast<float>(bf16_to_double(W[n * ldw + k]))));
    volatile float sv = (mx == 0.0f) ? 1.0f : mx / 7.0f;
    float s = sv;
    s_w[n] = s;
    uint8_t* out = wq + n * (K / 2);
    for (int64_t k = 0; k < K; ++k) {
      float w = static_cast<float>(bf16_to_double(W[n * ldw + k]));
      volatile float q = w / s;  // fp32 division, no double intermediate
      float r = std::nearbyintf(q);
      nib_set(out, k, clampi(static_cast<long>(r), -8, 7));
      if (tie_dist) {
        const double rd = static_cast<double>(w) / static_cast<double>(s);
        tie_dist[n * K + k] = static_cast<float>(std::fabs(rd - std::floor(rd) - 0.5));
      }
    }
  });
}

// ---- integer GEMM (Sec. 3: low-bit matrix multiplication) --------------------------------------
// acc[t,n] = sum_k xq[t,k] * wq[n,k], accumulated in int64, returned as int32.
// Returns 0, or 1 if any accumulator does not fit int32.
int orc_gemm_i4(const uint8_t* xq, const uint8_t* wq, int64_t M, int64_t N, int64_t K, int32_t* acc) {
  std::atomic<int> overflow{0};
  std::vector<int8_t> w(static_cast<size_t>(N * K));
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) w[n * K + k] = static_cast<int8_t>(nib_get(wq + n * (K / 2), k));
  parallel_rows(M, [&](int64_t t) {
    std::vector<int8_t> xr(K);
    for (int64_t k = 0; k < K; ++k) xr[k] = static_cast<int8_t>(nib_get(xq + t * (K / 2), k));
    for (int64_t n = 0; n < N; ++n) {
      const int8_t* wr = w.data() + n * K;
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += static_cast<int64_t>(xr[k]) * static_cast<int64_t>(wr[k]);
      if (s > INT32_MAX || s < INT32_MIN) overflow = 1;
      acc[t * N + n] = static_cast<int32_t>(s);
    }
  });
  return overflow.load();
}

// Dequantization epilogue: out[t,n] = bf16( acc * s_a * s_w[n] ), product in double, one rounding.
void orc_dequant_bf16(const int32_t* acc, int64_t M, int64_t N, float s_a, const float* s_w, uint16_t* out) {
  parallel_rows(M, [&](int64_t t) {
    for (int64_t n = 0; n < N; ++n)
      out[t * N + n] =
          double_to_bf16(static_cast<double>(acc[t * N + n]) * static_cast<double>(s_a) * static_cast<double>(s_w[n]));
  });
}

// ---- 8-bit activations (the W4A8KV4 precision of Sec. 5.1; Eq. 1 with N = 8, static per-tensor) -----
// s_a = fp32( max |fp32(y)| / 127 ) over rows >= row_begin of the rotated calibration batch.
float orc_calib_act_scale8(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin) {
  double mx = 0.0;
  std::vector<double> xr(K), yr(K);
  for (int64_t m = row_begin; m < M; ++m) {
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    for (int64_t j = 0; j < K; ++j) mx = std::max(mx, std::fabs(static_cast<double>(static_cast<float>(yr[j]))));
  }
  if (mx == 0.0) return 1.0f;
  return static_cast<float>(mx / 127.0);
}

// code = clamp(round_half_even(y / s_a), -128, 127), one signed byte per element, y the rotated row.
// Rows < row_begin are left untouched; tie_dist as in orc_quant_act.
void orc_quant_act8(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, float s_a,
                    int8_t* xq, float* tie_dist) {
  const double s = static_cast<double>(s_a);
  parallel_rows(M, [&](int64_t m) {
    if (m < row_begin) return;
    std::vector<double> xr(K), yr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    for (int64_t j = 0; j < K; ++j) {
      double r = yr[j] / s;
      xq[m * K + j] = static_cast<int8_t>(clampi(std::lrint(std::nearbyint(r)), -128, 127));
      if (tie_dist) tie_dist[m * K + j] = static_cast<float>(std::fabs(r - std::floor(r) - 0.5));
    }
  });
}

// acc[t,n] = sum_k xq[t,k] * wq[n,k] with 8-bit activation codes and packed 4-bit weight codes,
// accumulated in int64, returned as int32. Returns 0, or 1 if any accumulator does not fit int32.
int orc_gemm_i8i4(const int8_t* xq, const uint8_t* wq, int64_t M, int64_t N, int64_t K, int32_t* acc) {
  std::atomic<int> overflow{0};
  parallel_rows(M, [&](int64_t t) {
    for (int64_t n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k)
        s += static_cast<int64_t>(xq[t * K + k]) * static_cast<int64_t>(nib_get(wq + n * (K / 2), k));
      if (s > INT32_MAX || s < INT32_MIN) overflow = 1;
      acc[t * N + n] = static_cast<int32_t>(s);
    }
  });
  return overflow.load();
}

// ---- per-token dynamic activation quantization (Table 1, O1; Sec. 3 "Dynamic and Static") ---------
// One step per token, computed online from the rotated row itself: s[t] = fp32(clip * max |fp32(y_t)| / 7),
// clip being the layer's clipping factor shared by all tokens (gamma of Eq. 1, symmetric form); 1 for an
// all-zero row. Rows below row_begin keep whatever s holds.
void orc_dyn_act_scale(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, float clip,
                       float* s) {
  parallel_rows(M, [&](int64_t m) {
    if (m < row_begin) return;
    std::vector<double> xr(K), yr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    double mx = 0.0;
    for (int64_t j = 0; j < K; ++j) mx = std::max(mx, std::fabs(static_cast<double>(static_cast<float>(yr[j]))));
    s[m] = mx == 0.0 ? 1.0f : static_cast<float>(static_cast<double>(clip) * mx / 7.0);
  });
}

// code[t,k] = clamp(round_half_even(y[t,k] / s[t]), -8, 7) with one step per row; otherwise as orc_quant_act.
void orc_quant_act_rows(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, const float* s_tok,
                        uint8_t* xq, float* tie_dist) {
  parallel_rows(M, [&](int64_t m) {
    if (m < row_begin) return;
    const double s = static_cast<double>(s_tok[m]);
    std::vector<double> xr(K), yr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    uint8_t* out = xq + m * (K / 2);
    for (int64_t j = 0; j < K; ++j) {
      double r = yr[j] / s;
      nib_set(out, j, clampi(std::lrint(std::nearbyint(r)), -8, 7));
      if (tie_dist) tie_dist[m * K + j] = static_cast<float>(std::fabs(r - std::floor(r) - 0.5));
    }
  });
}

// out[t,n] = bf16( acc[t,n] * s_tok[t] * s_w[n] ), product in double, one rounding.
void orc_dequant_bf16_rows(const int32_t* acc, int64_t M, int64_t N, const float* s_tok, const float* s_w, uint16_t* out) {
  parallel_rows(M, [&](int64_t t) {
    for (int64_t n = 0; n < N; ++n)
      out[t * N + n] = double_to_bf16(static_cast<double>(acc[t * N + n]) * static_cast<double>(s_tok[t]) *
                                      static_cast<double>(s_w[n]));
  });
}

// ---- outlier tokens (Sec. 4.1, "Definition of Outlier Token", Eq. 2) ------------------------------------
// M[i] = max_c |X[i,c]|; R[i] = M[i] / median(M); token i is an upper outlier when R[i] > eta1 and a lower
// outlier when 1 / R[i] > eta2 (flags 1 and 2, else 0). The median of an even number of tokens is the mean
// of the two middle values. M is exact (bf16 inputs); the median and the two ratios M / median and
// median / M are rounded to fp32, the precision in which the thresholds are compared.
void orc_outlier_tokens(const uint16_t* x, int64_t ldx, int64_t T, int64_t C, float eta1, float eta2, float* M, float* R,
                        int32_t* flags, float* median_out) {
  std::vector<float> m(T);
  for (int64_t i = 0; i < T; ++i) {
    double mx = 0.0;
    for (int64_t c = 0; c < C; ++c) mx = std::max(mx, std::fabs(bf16_to_double(x[i * ldx + c])));
    m[i] = static_cast<float>(mx);
    M[i] = m[i];
  }
  std::vector<float> sorted(m);
  std::sort(sorted.begin(), sorted.end());
  const float med = T == 0 ? 0.0f
                           : static_cast<float>(0.5 * (static_cast<double>(sorted[(T - 1) / 2]) + static_cast<double>(sorted[T / 2])));
  *median_out = med;
  for (int64_t i = 0; i < T; ++i) {
    const float r = static_cast<float>(static_cast<double>(m[i]) / static_cast<double>(med));
    const float inv = static_cast<float>(static_cast<double>(med) / static_cast<double>(m[i]));
    R[i] = r;
    flags[i] = r > eta1 ? 1 : (inv > eta2 ? 2 : 0);
  }
}

// ---- Eq. 1 with its zero point: asymmetric static per-tensor activations (N = 4) -------------------------
// Range of the rotated calibration rows >= row_begin: mn = min fp32(y), mx = max fp32(y).
void orc_calib_act_minmax(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, float* mn_out,
                          float* mx_out) {
  double mn = INFINITY, mx = -INFINITY;
  std::vector<double> xr(K), yr(K);
  for (int64_t m = row_begin; m < M; ++m) {
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    for (int64_t j = 0; j < K; ++j) {
      const double v = static_cast<double>(static_cast<float>(yr[j]));
      mn = std::min(mn, v), mx = std::max(mx, v);
    }
  }
  *mn_out = static_cast<float>(mn), *mx_out = static_cast<float>(mx);
}

// Max-min initialisation (gamma = beta = 1): s = (mx - mn) / (2^N - 1), z = -floor(mn / s): Eq. 1 prints the
// zero point with floor brackets (only X / s carries the rounding brackets), and the floor is taken here as
// printed. Every step is an IEEE fp32 operation (the precision the GPU takes them in); a constant tensor
// gets s = 1, z = 0. z is kept inside the code range.
void orc_asym_params(float mn, float mx, int bits, float* s_out, int32_t* z_out) {
  const int qmax = (1 << bits) - 1;
  if (!(mx > mn)) {
    *s_out = 1.0f, *z_out = 0;
    return;
  }
  const float d = static_cast<float>(static_cast<double>(mx) - static_cast<double>(mn));
  const float s = static_cast<float>(static_cast<double>(d) / static_cast<double>(qmax));
  const float q = static_cast<float>(static_cast<double>(mn) / static_cast<double>(s));
  *s_out = s;
  *z_out = clampi(-std::lrint(std::floor(static_cast<double>(q))), 0, qmax);
}

// X_INT = clamp(round_half_even(y / s) + z, 0, 15), one byte per element, y the rotated row; rows < row_begin
// are left untouched; tie_dist as in orc_quant_act.
void orc_quant_act_asym(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, float s_a, int32_t z,
                        uint8_t* u, float* tie_dist) {
  const double s = static_cast<double>(s_a);
  parallel_rows(M, [&](int64_t m) {
    if (m < row_begin) return;
    std::vector<double> xr(K), yr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    for (int64_t j = 0; j < K; ++j) {
      double r = yr[j] / s;
      u[m * K + j] = static_cast<uint8_t>(clampi(std::lrint(std::nearbyint(r)) + z, 0, 15));
      if (tie_dist) tie_dist[m * K + j] = static_cast<float>(std::fabs(r - std::floor(r) - 0.5));
    }
  });
}

// ---- grid search for the static s and z (Sec. 3, "Initialization of Quantization Parameters") --------------
// Candidates of Eq. 1 over a grid of clipping factors: gamma_i = 1 - i * step, beta_j = 1 - j * step with
// step = (1 - lo) / (n - 1) (i, j = 0 .. n-1; n = 1: the max-min pair alone), candidate i * n + j being
//   s = (gamma_i * mx - beta_j * mn) / (2^N - 1),   z = -floor(beta_j * mn / s)   clamped to the code range,
// every step one IEEE fp32 operation (the precision the GPU forms them in); a range that is not positive gives
// s = 1, z = 0.
void orc_grid_candidates(float mn, float mx, int bits, int n, float lo, float* s_out, int32_t* z_out) {
  const int qmax = (1 << bits) - 1;
  volatile float step = n > 1 ? (1.0f - lo) / static_cast<float>(n - 1) : 0.0f;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j) {
      volatile float fi = static_cast<float>(i) * step, fj = static_cast<float>(j) * step;
      volatile float gamma = 1.0f - fi, beta = 1.0f - fj;
      volatile float gm = gamma * mx, bm = beta * mn;
      volatile float d = gm - bm;
      float s = 1.0f;
      int32_t z = 0;
      if (d > 0.0f) {
        volatile float sv = d / static_cast<float>(qmax);
        s = sv;
        volatile float q = bm / sv;
        z = clampi(-std::lrint(std::floor(static_cast<double>(q))), 0, qmax);
      }
      s_out[i * n + j] = s, z_out[i * n + j] = z;
    }
}

// Sum over the rotated rows >= row_begin of (y - s (u - z))^2 with u = clamp(round_half_even(y / s) + z, 0, 2^N - 1):
// the squared error of quantizing and dequantizing the tensor with one candidate, in double.
double orc_quant_sse_asym(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, int bits, float s_a,
                          int32_t z) {
  const int qmax = (1 << bits) - 1;
  const double s = static_cast<double>(s_a);
  std::vector<double> row_sse(M, 0.0);
  parallel_rows(M, [&](int64_t m) {
    if (m < row_begin) return;
    std::vector<double> xr(K), yr(K);
    for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
    rotate_row(xr.data(), yr.data(), K, B);
    double acc = 0.0;
    for (int64_t j = 0; j < K; ++j) {
      const long u = clampi(std::lrint(std::nearbyint(yr[j] / s)) + z, 0, qmax);
      const double e = yr[j] - s * static_cast<double>(u - z);
      acc += e * e;
    }
    row_sse[m] = acc;
  });
  double total = 0.0;
  for (int64_t m = row_begin; m < M; ++m) total += row_sse[m];
  return total;
}

// The search itself: range of the rotated calibration rows, the n x n candidates, the squared error of each, and
// the candidate with the smallest error (the first one in index order among equals). sse_out (nullable) [n*n].
void orc_grid_search_act(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, int bits, int n, float lo,
                         float* s_out, int32_t* z_out, double* sse_out) {
  float mn, mx;
  orc_calib_act_minmax(x, ldx, M, K, B, row_begin, &mn, &mx);
  std::vector<float> cs(n * n);
  std::vector<int32_t> cz(n * n);
  orc_grid_candidates(mn, mx, bits, n, lo, cs.data(), cz.data());
  int best = 0;
  double best_sse = INFINITY;
  for (int c = 0; c < n * n; ++c) {
    const double sse = orc_quant_sse_asym(x, ldx, M, K, B, row_begin, bits, cs[c], cz[c]);
    if (sse_out) sse_out[c] = sse;
    if (sse < best_sse) best_sse = sse, best = c;
  }
  *s_out = cs[best], *z_out = cz[best];
}

// Grid search for the clipping factor of per-token dynamic quantization (Sec. 3, "Initialization of Quantization
// Parameters": gamma is shared by all tokens of a layer and chosen by mean squared error). Symmetric form, as in
// orc_dyn_act_scale: candidate i has gamma_i = 1 - i * (1 - lo) / (n - 1) (fp32 steps as in orc_grid_candidates), every
// row takes its own step fp32(gamma_i * max |y_t| / 7), and sse[i] = sum over rows >= row_begin and columns of
// (y - s_t q)^2 with q = clamp(round_half_even(y / s_t), -8, 7), in double. The smallest error wins, the first one in
// index order among equals. gamma_out [1], cand_out (nullable) [n], sse_out (nullable) [n].
void orc_grid_search_clip_dyn(const uint16_t* x, int64_t ldx, int64_t M, int64_t K, int B, int64_t row_begin, int n, float lo,
                              float* gamma_out, float* cand_out, double* sse_out) {
  volatile float step = n > 1 ? (1.0f - lo) / static_cast<float>(n - 1) : 0.0f;
  int best = 0;
  double best_sse = INFINITY;
  float best_gamma = 1.0f;
  for (int i = 0; i < n; ++i) {
    volatile float fi = static_cast<float>(i) * step;
    volatile float gamma = 1.0f - fi;
    std::vector<float> s_tok(M, 1.0f);
    orc_dyn_act_scale(x, ldx, M, K, B, row_begin, gamma, s_tok.data());
    std::vector<double> row_sse(M, 0.0);
    parallel_rows(M, [&](int64_t m) {
      if (m < row_begin) return;
      const double s = static_cast<double>(s_tok[m]);
      std::vector<double> xr(K), yr(K);
      for (int64_t j = 0; j < K; ++j) xr[j] = bf16_to_double(x[m * ldx + j]);
      rotate_row(xr.data(), yr.data(), K, B);
      double acc = 0.0;
      for (int64_t j = 0; j < K; ++j) {
        const long q = clampi(std::lrint(std::nearbyint(yr[j] / s)), -8, 7);
        const double e = yr[j] - s * static_cast<double>(q);
        acc += e * e;
      }
      row_sse[m] = acc;
    });
    double total = 0.0;
    for (int64_t m = row_begin; m < M; ++m) total += row_sse[m];
    if (cand_out) cand_out[i] = gamma;
    if (sse_out) sse_out[i] = total;
    if (total < best_sse) best_sse = total, best = i, best_gamma = gamma;
  }
  (void)best;
  *gamma_out = best_gamma;
}

// acc[t,n] = sum_k (u[t,k] - z) * wq[n,k]: the dequantized activation (up to its step) times the weight codes,
// written out as such (no correction-term algebra). Returns 1 if an accumulator does not fit int32.
int orc_gemm_asym(const uint8_t* u, int32_t z, const uint8_t* wq, int64_t M, int64_t N, int64_t K, int32_t* acc) {
  std::atomic<int> overflow{0};
  parallel_rows(M, [&](int64_t t) {
    for (int64_t n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k)
        s += (static_cast<int64_t>(u[t * K + k]) - z) * static_cast<int64_t>(nib_get(wq + n * (K / 2), k));
      if (s > INT32_MAX || s < INT32_MIN) overflow = 1;
      acc[t * N + n] = static_cast<int32_t>(s);
    }
  });
  return overflow.load();
}

// ---- per-head static KV scale and KV4 append (Table 1, O2: per-head static KV cache) ----------
// kv bf16 [B,T,H,D]; s[h] = fp32(max |kv[:,:,h,:]|) / 7 in double then fp32 (1 if all zero).
void orc_calib_kv_scale(const uint16_t* kv, int64_t B, int64_t T, int64_t H, int64_t D, float* s) {
  for (int64_t h = 0; h < H; ++h) {
    double mx = 0.0;
    for (int64_t b = 0; b < B; ++b)
      for (int64_t t = 0; t < T; ++t)
        for (int64_t d = 0; d < D; ++d) mx = std::max(mx, std::fabs(bf16_to_double(kv[((b * T + t) * H + h) * D + d])));
    s[h] = mx == 0.0 ? 1.0f : static_cast<float>(mx / 7.0);
  }
}

// k, v bf16 [B,T_new,H,D] -> codes written at rows len[b] .. len[b]+T_new-1 of
// kq, vq u8 [B,H,Tmax,D/2]; len[b] += T_new. Returns 1 (nothing written) if any sequence would
// exceed Tmax. tie_k, tie_v (nullable, [B,T_new,H,D] float): distance of the exact quotient x / s (taken in
// double) from the closest rounding tie, as in orc_quant_act.
int orc_kv4_append(const uint16_t* k, const uint16_t* v, int64_t B, int64_t T_new, int64_t H, int64_t D,
                   const float* s_k, const float* s_v, uint8_t* kq, uint8_t* vq, int32_t* len, int64_t Tmax,
                   float* tie_k, float* tie_v) {
  for (int64_t b = 0; b < B; ++b)
    if (len[b] + T_new > Tmax) return 1;
  for (int64_t b = 0; b < B; ++b) {
    for (int64_t t = 0; t < T_new; ++t)
      for (int64_t h = 0; h < H; ++h) {
        int64_t pos = len[b] + t;
        uint8_t* kr = kq + ((b * H + h) * Tmax + pos) * (D / 2);
        uint8_t* vr = vq + ((b * H + h) * Tmax + pos) * (D / 2);
        for (int64_t d = 0; d < D; ++d) {
          // the code is decided in IEEE fp32 (bf16 input, fp32 step), the precision of the GPU kernel
          float kf = static_cast<float>(bf16_to_double(k[((b * T_new + t) * H + h) * D + d]));
          float vf = static_cast<float>(bf16_to_double(v[((b * T_new + t) * H + h) * D + d]));
          volatile float qk = kf / s_k[h];
          volatile float qv = vf / s_v[h];
          nib_set(kr, d, clampi(static_cast<long>(std::nearbyintf(qk)), -8, 7));
          nib_set(vr, d, clampi(static_cast<long>(std::nearbyintf(qv)), -8, 7));
          const int64_t idx = ((b * T_new + t) * H + h) * D + d;
          if (tie_k) {
            const double r = static_cast<double>(kf) / static_cast<double>(s_k[h]);
            tie_k[idx] = static_cast<float>(std::fabs(r - std::floor(r) - 0.5));
          }
          if (tie_v) {
            const double r = static_cast<double>(vf) / static_cast<double>(s_v[h]);
            tie_v[idx] = static_cast<float>(std::fabs(r - std::floor(r) - 0.5));
          }
        }
      }
    len[b] += static_cast<int32_t>(T_new);
  }
  return 0;
}

// ---- attention over [full-precision prefix || INT4 cache] (Eq. 3) -------------------------------
// One (query row, head) of softmax attention in double over the union of
//   n_prefix prefix keys/values (fp16, [Hkv, n_prefix, D], one copy shared by every sequence) and
//   n_ctx quantized keys/values (codes * per-head scale).
// sk_tok, sv_tok (nullable): one step per cached key (group-wise dynamic KV, Table 1 O1); they replace sk, sv.
static void attend_one(const double* q, int64_t D, double sm_scale, const uint16_t* pk, const uint16_t* pv,
                       int64_t n_prefix, const uint8_t* kq, const uint8_t* vq, int64_t n_ctx, double sk, double sv,
                       double* out, const float* sk_tok = nullptr, const float* sv_tok = nullptr) {
  int64_t n = n_prefix + n_ctx;
  std::vector<double> sc(n);
  for (int64_t j = 0; j < n; ++j) {
    double s = 0.0;
    if (j < n_prefix)
      for (int64_t d = 0; d < D; ++d) s += q[d] * fp16_to_double(pk[j * D + d]);
    else
      for (int64_t d = 0; d < D; ++d)
        s += q[d] * (nib_get(kq + (j - n_prefix) * (D / 2), d) * (sk_tok ? static_cast<double>(sk_tok[j - n_prefix]) : sk));
    sc[j] = s * sm_scale;
  }
  double mx = -INFINITY;
  for (int64_t j = 0; j < n; ++j) mx = std::max(mx, sc[j]);
  double den = 0.0;
  for (int64_t j = 0; j < n; ++j) {
    sc[j] = std::exp(sc[j] - mx);
    den += sc[j];
  }
  for (int64_t d = 0; d < D; ++d) out[d] = 0.0;
  for (int64_t j = 0; j < n; ++j) {
    double p = sc[j] / den;
    if (j < n_prefix)
      for (int64_t d = 0; d < D; ++d) out[d] += p * fp16_to_double(pv[j * D + d]);
    else
      for (int64_t d = 0; d < D; ++d)
        out[d] += p * (nib_get(vq + (j - n_prefix) * (D / 2), d) * (sv_tok ? static_cast<double>(sv_tok[j - n_prefix]) : sv));
  }
}

// Decode: one query token per sequence, every cached key visible.
// q bf16 [B,Hq,D]; prefix_k/v fp16 [Hkv,n_prefix,D]; kq/vq u8 [B,Hkv,Tmax,D/2]; len int32 [B];
// out bf16 [B,Hq,D]; out_f64 (nullable) receives the unrounded result.
void orc_decode_attn(const uint16_t* q, const uint16_t* prefix_k, const uint16_t* prefix_v, const uint8_t* kq,
                     const uint8_t* vq, const float* s_k, const float* s_v, const int32_t* len, int64_t B, int64_t Hq,
                     int64_t Hkv, int64_t D, int64_t n_prefix, int64_t Tmax, double sm_scale, uint16_t* out,
                     double* out_f64) {
  int64_t group = Hq / Hkv;
  parallel_rows(B * Hq, [&](int64_t i) {
    int64_t b = i / Hq, g = i % Hq, h = g / group;
    std::vector<double> qd(D), od(D);
    for (int64_t d = 0; d < D; ++d) qd[d] = bf16_to_double(q[(b * Hq + g) * D + d]);
    attend_one(qd.data(), D, sm_scale, prefix_k + h * n_prefix * D, prefix_v + h * n_prefix * D, n_prefix,
               kq + (b * Hkv + h) * Tmax * (D / 2), vq + (b * Hkv + h) * Tmax * (D / 2), len[b], s_k[h], s_v[h],
               od.data());
    for (int64_t d = 0; d < D; ++d) {
      out[(b * Hq + g) * D + d] = double_to_bf16(od[d]);
      if (out_f64) out_f64[(b * Hq + g) * D + d] = od[d];
    }
  });
}

// Prefill: T query tokens of one sequence; query t sees the whole prefix and cached keys 0..t
// (the prefix sits at the beginning of the sequence, Sec. 4.2).
// q bf16 [T,Hq,D]; kq/vq u8 [Hkv,Tmax,D/2] of this sequence; out bf16 [T,Hq,D]; out_f64 (nullable)
// receives the unrounded result.
void orc_prefill_attn(const uint16_t* q, const uint16_t* prefix_k, const uint16_t* prefix_v, const uint8_t* kq,
                      const uint8_t* vq, const float* s_k, const float* s_v, int64_t T, int64_t Hq, int64_t Hkv,
                      int64_t D, int64_t n_prefix, int64_t Tmax, double sm_scale, uint16_t* out, double* out_f64) {
  int64_t group = Hq / Hkv;
  parallel_rows(T * Hq, [&](int64_t i) {
    int64_t t = i / Hq, g = i % Hq, h = g / group;
    std::vector<double> qd(D), od(D);
    for (int64_t d = 0; d < D; ++d) qd[d] = bf16_to_double(q[(t * Hq + g) * D + d]);
    attend_one(qd.data(), D, sm_scale, prefix_k + h * n_prefix * D, prefix_v + h * n_prefix * D, n_prefix,
               kq + h * Tmax * (D / 2), vq + h * Tmax * (D / 2), t + 1, s_k[h], s_v[h], od.data());
    for (int64_t d = 0; d < D; ++d) {
      out[(t * Hq + g) * D + d] = double_to_bf16(od[d]);
      if (out_f64) out_f64[(t * Hq + g) * D + d] = od[d];
    }
  });
}

// ---- group-wise dynamic KV4 (Table 1, O1: "group-wise dynamic" KV cache, group size 128 = the head dimension) --
// Every (token, head) vector of 128 values is one group with its own step, computed online when the token is
// written: s = fp32(max |x|) / 7 in fp32 (1 for an all-zero vector), code = clamp(rint_fp32(x / s), -8, 7) with the
// fp32 decision of the static path. Steps go to sk_tok, sv_tok f32 [B,H,Tmax] at the token's position.
int orc_kv4_append_dyn(const uint16_t* k, const uint16_t* v, int64_t B, int64_t T_new, int64_t H, int64_t D, uint8_t* kq,
                       uint8_t* vq, float* sk_tok, float* sv_tok, int32_t* len, int64_t Tmax) {
  for (int64_t b = 0; b < B; ++b)
    if (len[b] + T_new > Tmax) return 1;
  for (int64_t b = 0; b < B; ++b) {
    for (int64_t t = 0; t < T_new; ++t)
      for (int64_t h = 0; h < H; ++h) {
        const int64_t pos = len[b] + t;
        for (int which = 0; which < 2; ++which) {
          const uint16_t* src = (which ? v : k) + ((b * T_new + t) * H + h) * D;
          uint8_t* row = (which ? vq : kq) + ((b * H + h) * Tmax + pos) * (D / 2);
          float mx = 0.0f;
          for (int64_t d = 0; d < D; ++d) mx = std::max(mx, std::fabs(static_cast<float>(bf16_to_double(src[d]))));
          volatile float sv_ = mx == 0.0f ? 1.0f : mx / 7.0f;
          const float s = sv_;
          (which ? sv_tok : sk_tok)[(b * H + h) * Tmax + pos] = s;
          for (int64_t d = 0; d < D; ++d) {
            volatile float q = static_cast<float>(bf16_to_double(src[d])) / s;
            nib_set(row, d, clampi(static_cast<long>(std::nearbyintf(q)), -8, 7));
          }
        }
      }
    len[b] += static_cast<int32_t>(T_new);
  }
  return 0;
}

// Decode attention (Eq. 3) over [prefix || INT4 cache] with one step per cached key and value vector.
void orc_decode_attn_dyn(const uint16_t* q, const uint16_t* prefix_k, const uint16_t* prefix_v, const uint8_t* kq,
                         const uint8_t* vq, const float* sk_tok, const float* sv_tok, const int32_t* len, int64_t B, int64_t Hq,
                         int64_t Hkv, int64_t D, int64_t n_prefix, int64_t Tmax, double sm_scale, uint16_t* out, double* out_f64) {
  int64_t group = Hq / Hkv;
  parallel_rows(B * Hq, [&](int64_t i) {
    int64_t b = i / Hq, g = i % Hq, h = g / group;
    std::vector<double> qd(D), od(D);
    for (int64_t d = 0; d < D; ++d) qd[d] = bf16_to_double(q[(b * Hq + g) * D + d]);
    attend_one(qd.data(), D, sm_scale, prefix_k + h * n_prefix * D, prefix_v + h * n_prefix * D, n_prefix,
               kq + (b * Hkv + h) * Tmax * (D / 2), vq + (b * Hkv + h) * Tmax * (D / 2), len[b], 0.0, 0.0, od.data(),
               sk_tok + (b * Hkv + h) * Tmax, sv_tok + (b * Hkv + h) * Tmax);
    for (int64_t d = 0; d < D; ++d) {
      out[(b * Hq + g) * D + d] = double_to_bf16(od[d]);
      if (out_f64) out_f64[(b * Hq + g) * D + d] = od[d];
    }
  });
}

// Causal prefill attention of one sequence with per-key steps (sk_tok, sv_tok [Hkv,Tmax] of this sequence).
void orc_prefill_attn_dyn(const uint16_t* q, const uint16_t* prefix_k, const uint16_t* prefix_v, const uint8_t* kq,
                          const uint8_t* vq, const float* sk_tok, const float* sv_tok, int64_t T, int64_t Hq, int64_t Hkv,
                          int64_t D, int64_t n_prefix, int64_t Tmax, double sm_scale, uint16_t* out, double* out_f64) {
  int64_t group = Hq / Hkv;
  parallel_rows(T * Hq, [&](int64_t i) {
    int64_t t = i / Hq, g = i % Hq, h = g / group;
    std::vector<double> qd(D), od(D);
    for (int64_t d = 0; d < D; ++d) qd[d] = bf16_to_double(q[(t * Hq + g) * D + d]);
    attend_one(qd.data(), D, sm_scale, prefix_k + h * n_prefix * D, prefix_v + h * n_prefix * D, n_prefix,
               kq + h * Tmax * (D / 2), vq + h * Tmax * (D / 2), t + 1, 0.0, 0.0, od.data(), sk_tok + h * Tmax, sv_tok + h * Tmax);
    for (int64_t d = 0; d < D; ++d) {
      out[(t * Hq + g) * D + d] = double_to_bf16(od[d]);
      if (out_f64) out_f64[(t * Hq + g) * D + d] = od[d];
    }
  });
}

// ---- transformer-block glue of a Llama block (App. B figure; used by the full-block config) ----
// RMSNorm: y = x / sqrt(mean(x^2) + eps) * g, rounded once to bf16.
void orc_rmsnorm(const uint16_t* x, const uint16_t* g, int64_t M, int64_t K, double eps, uint16_t* y) {
  parallel_rows(M, [&](int64_t m) {
    double ss = 0.0;
    for (int64_t j = 0; j < K; ++j) {
      double v = bf16_to_double(x[m * K + j]);
      ss += v * v;
    }
    double r = 1.0 / std::sqrt(ss / static_cast<double>(K) + eps);
    for (int64_t j = 0; j < K; ++j)
      y[m * K + j] = double_to_bf16(bf16_to_double(x[m * K + j]) * r * bf16_to_double(g[j]));
  });
}

// Rotary embedding, rotate-half pairing: for i < D/2, angle = pos * theta^(-2i/D),
//   y[i] = x[i] cos - x[i+D/2] sin,  y[i+D/2] = x[i+D/2] cos + x[i] sin.
// x bf16 [T,H,D], token t at position pos0 + t; result rounded once to bf16.
void orc_rope(const uint16_t* x, int64_t T, int64_t H, int64_t D, int64_t pos0, double theta, uint16_t* y) {
  parallel_rows(T, [&](int64_t t) {
    double pos = static_cast<double>(pos0 + t);
    for (int64_t h = 0; h < H; ++h)
      for (int64_t i = 0; i < D / 2; ++i) {
        double ang = pos * std::pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(D));
        double c = std::cos(ang), s = std::sin(ang);
        double a = bf16_to_double(x[(t * H + h) * D + i]);
        double b = bf16_to_double(x[(t * H + h) * D + i + D / 2]);
        y[(t * H + h) * D + i] = double_to_bf16(a * c - b * s);
        y[(t * H + h) * D + i + D / 2] = double_to_bf16(b * c + a * s);
      }
  });
}

// Rotary embedding followed by the online head-wise rotation R3 (App. B, "Online Rotation": the outputs
// of q_proj and k_proj after RoPE are multiplied by the Hadamard matrix of the head dimension):
// y = RoPE(x) H_D / sqrt(D) per head, everything in double, one rounding to bf16.
void orc_rope_rotate(const uint16_t* x, int64_t T, int64_t H, int64_t D, int64_t pos0, double theta, uint16_t* y) {
  parallel_rows(T, [&](int64_t t) {
    double pos = static_cast<double>(pos0 + t);
    std::vector<double> r(D), z(D);
    for (int64_t h = 0; h < H; ++h) {
      for (int64_t i = 0; i < D / 2; ++i) {
        double ang = pos * std::pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(D));
        double c = std::cos(ang), s = std::sin(ang);
        double a = bf16_to_double(x[(t * H + h) * D + i]);
        double b = bf16_to_double(x[(t * H + h) * D + i + D / 2]);
        r[i] = a * c - b * s;
        r[i + D / 2] = b * c + a * s;
      }
      rotate_row(r.data(), z.data(), D, static_cast<int>(D));
      for (int64_t i = 0; i < D; ++i) y[(t * H + h) * D + i] = double_to_bf16(z[i]);
    }
  });
}

// SwiGLU gate: y = silu(gate) * up = gate / (1 + exp(-gate)) * up, rounded once to bf16.
void orc_silu_mul(const uint16_t* gate, const uint16_t* up, int64_t n, uint16_t* y) {
  for (int64_t i = 0; i < n; ++i) {
    double g = bf16_to_double(gate[i]), u = bf16_to_double(up[i]);
    y[i] = double_to_bf16(g / (1.0 + std::exp(-g)) * u);
  }
}

// Residual: y = a + b, rounded once to bf16.
void orc_add(const uint16_t* a, const uint16_t* b, int64_t n, uint16_t* y) {
  for (int64_t i = 0; i < n; ++i) y[i] = double_to_bf16(bf16_to_double(a[i]) + bf16_to_double(b[i]));
}

}  // extern "C"

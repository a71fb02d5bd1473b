// CPU oracle for Multi-Scale Dequant (MSD).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, scalar statement of
// what the method computes, written from the paper.  It shares no code, header,
// table or constant generator with the CUDA library; nothing in the product
// path may link, import or call it.  Only tests, the smoke check and the
// benchmark's CPU-baseline leg use it.
//
// Conventions
//  * BF16 values travel as uint16_t bit patterns (upper half of an IEEE FP32).
//  * All "scale" arithmetic that decides an integer code (alpha, x/alpha, the
//    residual, beta, r/beta) is IEEE FP32 with true division, round-half-to-even
//    and denormals kept; the residual is one fused multiply-add, which makes it
//    exact.  Built with -ffp-contract=off so the compiler fuses nothing else.
//  * Every "reference" quantity (combined outputs, softmax, error metrics) is
//    FP64 and rounded once to the output type.
//  * OpenMP only spreads independent rows / heads over threads; it changes no
//    arithmetic.
//
// Pins (see tests/test_oracle_*.py): Theorem 1 (INT8 bound M/64516), Theorem 2
// (E1M2 bound alpha/64, tight), Tab. mxfp4-evolution / mxfp4-decomp / mxfp4-bound
// statistics, brute-force integer dot products, identity / one-hot / zero inputs,
// softmax special cases.  Parity unpinned: the per-token-scale attention layout
// has no printed number in the paper (Tab. flash-error-dist uses per-channel
// scales and head_dim 64); only structural pins and the ordering "MSD error <
// dequant error" hold it.

#include <algorithm>
#include <cfenv>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline float bf16_to_f32(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

// FP64 -> BF16 with a single round-half-to-even (no intermediate FP32 rounding).
inline uint16_t f64_to_bf16(double d) {
  if (std::isnan(d)) return 0x7FC0;
  uint16_t sign = std::signbit(d) ? 0x8000 : 0;
  double a = std::fabs(d);
  if (a == 0.0) return sign;
  if (std::isinf(a)) return sign | 0x7F80;
  int e = std::ilogb(a);
  if (e < -126) e = -126;                    // subnormal range shares the ulp of 2^-126
  double ulp = std::ldexp(1.0, e - 7);       // BF16 keeps 8 significand bits
  double n = std::nearbyint(a / ulp);        // exact scaling, RNE
  double v = n * ulp;                        // representable in FP32 exactly
  if (v >= std::ldexp(1.0, 128)) return sign | 0x7F80;
  float f = static_cast<float>(v);
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return sign | static_cast<uint16_t>(u >> 16);
}

inline int8_t clamp_i8(float v) {
  // v is already an integer-valued float (or +-inf / nan from degenerate scales)
  if (!(v == v)) return 0;
  if (v > 127.0f) return 127;
  if (v < -128.0f) return -128;
  return static_cast<int8_t>(v);
}

// Two-pass INT8 decomposition of one vector of FP32 values (Eq. alpha, x1,
// residual, beta, x2; Algorithm 1 lines 1-5).  `alpha_fixed` < 0 means "derive
// alpha from the row maximum"; otherwise the given alpha is used (the constant
// scale of the softmax probabilities, Sec. 4.2 step 3).
// (c1, c2) are the scaling constants: (127, 254) in Eq. alpha / Eq. beta, or the
// "fractional scaling" pair (127.49, 254.98) of Sec. 3.3, which keeps the extreme
// element's residual below alpha/2 and tightens the bound to M/65015.
void two_pass_int8(const float* x, int64_t n, int64_t stride, float alpha_fixed,
                   int8_t* q1, int8_t* q2, float* alpha_out, float* beta_out,
                   float c1 = 127.0f, float c2 = 254.0f) {
  float alpha;
  if (alpha_fixed >= 0.0f) {
    alpha = alpha_fixed;
  } else {
    float m = 0.0f;
    for (int64_t k = 0; k < n; ++k) m = std::max(m, std::fabs(x[k * stride]));
    alpha = m / c1;                                      // Eq. alpha
  }
  float beta = alpha / c2;                               // Eq. beta
  for (int64_t k = 0; k < n; ++k) {
    float v = x[k * stride];
    int8_t a = 0, b = 0;
    if (alpha > 0.0f) {
      a = clamp_i8(std::nearbyintf(v / alpha));          // Eq. x1
      float r = std::fmaf(-alpha, static_cast<float>(a), v);   // Eq. residual (exact)
      if (beta > 0.0f) b = clamp_i8(std::nearbyintf(r / beta)); // Eq. x2
    }
    q1[k] = a;
    q2[k] = b;
  }
  *alpha_out = alpha;
  *beta_out = beta;
}

// ---- 4-bit floating-point grids --------------------------------------------
// grid 0: E2M1 (0, .5, 1, 1.5, 2, 3, 4, 6) - what block-scaled FP4 tensor cores multiply.
// grid 1: E1M2 (0, .25, ..., 1.75)         - the grid the paper states (Sec. 2.2, 3.2.1).
const double kGrid[2][8] = {{0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0},
                            {0.0, 0.25, 0.5, 0.75, 1.0, 1.25, 1.5, 1.75}};

// Round-to-nearest on the grid, ties to the even code, saturating (Alg. 2 lines 4, 7).
inline uint8_t round_fp4(double s, int grid) {
  const double* g = kGrid[grid];
  uint8_t sign = std::signbit(s) ? 8 : 0;
  double a = std::fabs(s);
  if (!(a == a)) return 0;
  int best = 7;
  if (a < g[7]) {
    int hi = 1;
    while (g[hi] < a) ++hi;                 // g[hi-1] < a <= g[hi] (or a == 0 -> hi = 1)
    int lo = hi - 1;
    double dlo = a - g[lo], dhi = g[hi] - a;
    if (dlo < dhi) best = lo;
    else if (dhi < dlo) best = hi;
    else best = (lo % 2 == 0) ? lo : hi;    // tie -> even code
  }
  return sign | static_cast<uint8_t>(best);
}

inline double fp4_value(uint8_t code, int grid) {
  double v = kGrid[grid][code & 7];
  return (code & 8) ? -v : v;
}

// Smallest integer a with m <= c * 2^a  (Eq. alpha-mxfp4: alpha = 2^ceil(log2(M_b / c))),
// found by exact comparisons instead of a rounded logarithm.
inline int alpha_exponent(double m, double c) {
  int a = std::ilogb(m / c);
  while (std::ldexp(c, a) < m) ++a;
  while (std::ldexp(c, a - 1) >= m) --a;
  return a;
}

const int kE8M0Bias = 127;

// Two-pass MXFP4 decomposition of one 32-element block (Algorithm 2).
// c_bound / beta_shift are the (alpha bound, log2(alpha/beta)) pair of
// Tab. mxfp4-evolution; the exponent of alpha is kept >= beta_shift - 127 so
// that beta is still an E8M0 code.  A zero block takes that minimum exponent.
void two_pass_mxfp4_block(const double* x, int grid, double c_bound, int beta_shift,
                          uint8_t* c1, uint8_t* c2, int* ea, int* eb) {
  double mb = 0.0;
  for (int k = 0; k < 32; ++k) mb = std::max(mb, std::fabs(x[k]));   // line 1
  int amin = beta_shift - kE8M0Bias;
  int a = amin;
  if (mb > 0.0) a = std::max(amin, alpha_exponent(mb, c_bound));     // line 2
  a = std::min(a, 127);
  int b = a - beta_shift;                                            // line 6
  double alpha = std::ldexp(1.0, a), beta = std::ldexp(1.0, b);
  for (int k = 0; k < 32; ++k) {
    uint8_t q1 = round_fp4(x[k] / alpha, grid);                      // lines 3-4
    double r = x[k] - alpha * fp4_value(q1, grid);                   // line 5 (exact)
    uint8_t q2 = round_fp4(r / beta, grid);                          // line 7
    c1[k] = q1;
    c2[k] = q2;
  }
  *ea = a;
  *eb = b;
}

inline void pack_nibbles(const uint8_t* codes, int n, uint8_t* out) {
  for (int i = 0; i < n / 2; ++i) out[i] = static_cast<uint8_t>((codes[2 * i] & 15) | ((codes[2 * i + 1] & 15) << 4));
}
inline uint8_t nibble(const uint8_t* packed, int64_t i) {
  uint8_t b = packed[i >> 1];
  return (i & 1) ? (b >> 4) : (b & 15);
}

// E4M3 (max 448, 3 mantissa bits, subnormal step 2^-9) round-half-to-even, saturating.
inline double round_e4m3(double s) {
  double a = std::fabs(s);
  if (a == 0.0 || !(a == a)) return 0.0;
  int e = std::ilogb(a);
  e = std::max(e, -6);
  double step = std::ldexp(1.0, e - 3);
  double q = std::nearbyint(a / step) * step;
  q = std::min(q, 448.0);
  return std::signbit(s) ? -q : q;
}

}  // namespace

extern "C" {

int msdo_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void msdo_set_threads(int n) {
#ifdef _OPENMP
  omp_set_num_threads(n > 0 ? n : 1);
#else
  (void)n;
#endif
}

void msdo_round_bf16(const double* in, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = f64_to_bf16(in[i]);
}

// ---------------------------------------------------------------------------
// Offline quantizers (inputs of the method, Sec. 3.1 / 2.2 / 4.1)
// ---------------------------------------------------------------------------

// Symmetric INT8 per output channel: scale = rowmax/127, RNE, clamp to +-127.
void msdo_quantize_weight_int8(const float* w, int64_t N, int64_t K, int8_t* wq, float* w_scale) {
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    const float* row = w + n * K;
    float m = 0.0f;
    for (int64_t k = 0; k < K; ++k) m = std::max(m, std::fabs(row[k]));
    float s = m / 127.0f;
    w_scale[n] = s;
    for (int64_t k = 0; k < K; ++k) {
      float q = (s > 0.0f) ? std::nearbyintf(row[k] / s) : 0.0f;
      q = std::min(127.0f, std::max(-127.0f, q));
      wq[n * K + k] = static_cast<int8_t>(q);
    }
  }
}

// MXFP4 weights: one E8M0 scale per 32 contiguous K, scale = 2^(floor(log2 blockmax) - 2),
// E2M1 values, RNE with saturation; element 2i in the low nibble.
void msdo_quantize_weight_mxfp4(const float* w, int64_t N, int64_t K, uint8_t* w_fp4, uint8_t* w_e8m0) {
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    for (int64_t kb = 0; kb < K / 32; ++kb) {
      const float* blk = w + n * K + kb * 32;
      double mb = 0.0;
      for (int k = 0; k < 32; ++k) mb = std::max(mb, std::fabs(static_cast<double>(blk[k])));
      int e = (mb > 0.0) ? std::ilogb(mb) - 2 : -kE8M0Bias;
      e = std::min(127, std::max(-kE8M0Bias, e));
      double s = std::ldexp(1.0, e);
      uint8_t codes[32];
      for (int k = 0; k < 32; ++k) codes[k] = round_fp4(blk[k] / s, 0);
      pack_nibbles(codes, 32, w_fp4 + n * (K / 2) + kb * 16);
      w_e8m0[n * (K / 32) + kb] = static_cast<uint8_t>(e + kE8M0Bias);
    }
  }
}

// INT8 KV cache: one symmetric scale per row (= per token per KV head), scale = max/127.
void msdo_quantize_rows_int8(const uint16_t* x_bf16, int64_t rows, int64_t D, int8_t* q, float* scale) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    float m = 0.0f;
    for (int64_t k = 0; k < D; ++k) m = std::max(m, std::fabs(bf16_to_f32(x_bf16[r * D + k])));
    float s = m / 127.0f;
    scale[r] = s;
    for (int64_t k = 0; k < D; ++k) {
      float v = (s > 0.0f) ? std::nearbyintf(bf16_to_f32(x_bf16[r * D + k]) / s) : 0.0f;
      v = std::min(127.0f, std::max(-127.0f, v));
      q[r * D + k] = static_cast<int8_t>(v);
    }
  }
}

// ---------------------------------------------------------------------------
// Decompositions
// ---------------------------------------------------------------------------

// Two-pass INT8 decomposition per row (Sec. 3.2, Eqs. alpha..x2; Alg. 1 lines 1-5) with the
// scaling constants given (Sec. 3.3, "fractional scaling": 127.49 and 254.98 instead of 127 and 254).
void msdo_decompose_int8_c(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx, float c1, float c2,
                           int8_t* q1, int8_t* q2, float* alpha, float* beta) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    std::vector<float> row(K);
    for (int64_t k = 0; k < K; ++k) row[k] = bf16_to_f32(x_bf16[i * ldx + k]);
    two_pass_int8(row.data(), K, 1, -1.0f, q1 + i * K, q2 + i * K, alpha + i, beta + i, c1, c2);
  }
}

// Two-pass INT8 decomposition per row (Sec. 3.2, Eqs. alpha..x2; Alg. 1 lines 1-5).
void msdo_decompose_int8(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx,
                         int8_t* q1, int8_t* q2, float* alpha, float* beta) {
  msdo_decompose_int8_c(x_bf16, M, K, ldx, 127.0f, 254.0f, q1, q2, alpha, beta);
}

// Same rule on FP32 data with a caller-fixed alpha (< 0: derive from the row max).  Used by the
// pins that feed non-BF16 values and by the P decomposition of the attention oracle.
void msdo_decompose_int8_f32(const float* x, int64_t M, int64_t K, float alpha_fixed,
                             int8_t* q1, int8_t* q2, float* alpha, float* beta) {
  for (int64_t i = 0; i < M; ++i)
    two_pass_int8(x + i * K, K, 1, alpha_fixed, q1 + i * K, q2 + i * K, alpha + i, beta + i);
}

// Two-pass MXFP4 decomposition per 32-element block (Sec. 3.2.1, Alg. 2).
// grid: 0 = E2M1, 1 = E1M2.  Paper-literal: grid 1, c_bound 1.859375, beta_shift 4.
// Outputs: packed nibbles [M, K/2] (element 2i low), E8M0 bytes [M, K/32].
void msdo_decompose_mxfp4(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx, int grid,
                          double c_bound, int beta_shift, uint8_t* q1, uint8_t* q2,
                          uint8_t* e1, uint8_t* e2) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t kb = 0; kb < K / 32; ++kb) {
      double blk[32];
      uint8_t c1[32], c2[32];
      int ea, eb;
      for (int k = 0; k < 32; ++k) blk[k] = bf16_to_f32(x_bf16[i * ldx + kb * 32 + k]);
      two_pass_mxfp4_block(blk, grid, c_bound, beta_shift, c1, c2, &ea, &eb);
      pack_nibbles(c1, 32, q1 + i * (K / 2) + kb * 16);
      pack_nibbles(c2, 32, q2 + i * (K / 2) + kb * 16);
      e1[i * (K / 32) + kb] = static_cast<uint8_t>(ea + kE8M0Bias);
      e2[i * (K / 32) + kb] = static_cast<uint8_t>(eb + kE8M0Bias);
    }
  }
}

// alpha*q1 (+ beta*q2 when q2 != NULL) in FP64, for the error pins.
void msdo_mxfp4_reconstruct(const uint8_t* q1, const uint8_t* q2, const uint8_t* e1, const uint8_t* e2,
                            int64_t M, int64_t K, int grid, double* out) {
  for (int64_t i = 0; i < M; ++i)
    for (int64_t k = 0; k < K; ++k) {
      int64_t sb = i * (K / 32) + k / 32;
      double v = std::ldexp(fp4_value(nibble(q1 + i * (K / 2), k), grid), e1[sb] - kE8M0Bias);
      if (q2) v += std::ldexp(fp4_value(nibble(q2 + i * (K / 2), k), grid), e2[sb] - kE8M0Bias);
      out[i * K + k] = v;
    }
}

// Single-pass MXFP8 activation baseline (Sec. 6.5: E4M3 values, one E8M0 scale per 32 elements,
// scale = 2^ceil(log2(M_b/448))); returns the dequantized values.
void msdo_mxfp8_quantize(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx, double* xq) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t kb = 0; kb < K / 32; ++kb) {
      double mb = 0.0;
      for (int k = 0; k < 32; ++k) mb = std::max(mb, std::fabs(static_cast<double>(bf16_to_f32(x_bf16[i * ldx + kb * 32 + k]))));
      int a = (mb > 0.0) ? std::max(-kE8M0Bias, alpha_exponent(mb, 448.0)) : -kE8M0Bias;
      double s = std::ldexp(1.0, a);
      for (int k = 0; k < 32; ++k) {
        double v = bf16_to_f32(x_bf16[i * ldx + kb * 32 + k]);
        xq[i * K + kb * 32 + k] = s * round_e4m3(v / s);
      }
    }
}

// ---------------------------------------------------------------------------
// GEMMs
// ---------------------------------------------------------------------------

// Exact integer GEMM acc[i,n] = sum_k a[i,k] * w[n,k]  (Alg. 1 lines 6-7), INT64 accumulate;
// returns the number of outputs outside INT32 (must be 0).
int64_t msdo_int8_gemm_acc(const int8_t* a, const int8_t* w, int64_t M, int64_t N, int64_t K, int32_t* acc) {
  int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t i = 0; i < M; ++i) {
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += static_cast<int64_t>(a[i * K + k]) * static_cast<int64_t>(w[n * K + k]);
      if (s > INT32_MAX || s < INT32_MIN) ++overflow;
      acc[i * N + n] = static_cast<int32_t>(s);
    }
  return overflow;
}

// W8A16 MSD linear layer (Alg. 1): decompose, two exact integer GEMMs, y = s_W * (alpha*Y1 + beta*Y2)
// combined in FP64 and rounded once.  ytype 0: BF16 (uint16_t), 1: FP32, 2: FP64 (unrounded).
// acc_dbg (nullable): [2, M, N] INT32 accumulators.
int64_t msdo_gemm_w8a16_c(const uint16_t* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                          int64_t K, float c1, float c2, void* y, int ytype, int32_t* acc_dbg) {
  std::vector<int8_t> q1(M * K), q2(M * K);
  std::vector<float> alpha(M), beta(M);
  msdo_decompose_int8_c(x_bf16, M, K, K, c1, c2, q1.data(), q2.data(), alpha.data(), beta.data());
  std::vector<int32_t> acc(2 * M * N);
  int64_t ov = msdo_int8_gemm_acc(q1.data(), w, M, N, K, acc.data());
  ov += msdo_int8_gemm_acc(q2.data(), w, M, N, K, acc.data() + M * N);
  if (acc_dbg) std::memcpy(acc_dbg, acc.data(), sizeof(int32_t) * 2 * M * N);
  for (int64_t i = 0; i < M; ++i)
    for (int64_t n = 0; n < N; ++n) {
      double v = static_cast<double>(w_scale[n]) *
                 (static_cast<double>(alpha[i]) * acc[i * N + n] + static_cast<double>(beta[i]) * acc[M * N + i * N + n]);
      if (ytype == 0) static_cast<uint16_t*>(y)[i * N + n] = f64_to_bf16(v);
      else if (ytype == 1) static_cast<float*>(y)[i * N + n] = static_cast<float>(v);
      else static_cast<double*>(y)[i * N + n] = v;
    }
  return ov;
}

int64_t msdo_gemm_w8a16(const uint16_t* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                        int64_t K, void* y, int ytype, int32_t* acc_dbg) {
  return msdo_gemm_w8a16_c(x_bf16, w, w_scale, M, N, K, 127.0f, 254.0f, y, ytype, acc_dbg);
}

// FP64 reference on the dequantized weights: y = sum_k x[i,k] * (s_W[n] * w[n,k])  (Eq. in Sec. 3.1).
void msdo_gemm_ref_w8(const uint16_t* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K, double* y) {
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t i = 0; i < M; ++i) {
      double s = 0.0;
      for (int64_t k = 0; k < K; ++k) s += static_cast<double>(bf16_to_f32(x_bf16[i * K + k])) * w[n * K + k];
      y[i * N + n] = s * static_cast<double>(w_scale[n]);
    }
}

// Dequantize-then-BF16 comparison path (Sec. 3.1, Sec. 6.1 "Dequant"): weights become bf16(s_W*w),
// products of BF16 inputs accumulated without further rounding.
void msdo_gemm_dequant_bf16_w8(const uint16_t* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K, double* y) {
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    std::vector<double> wd(K);
    for (int64_t k = 0; k < K; ++k) wd[k] = bf16_to_f32(f64_to_bf16(static_cast<double>(w_scale[n] * static_cast<float>(w[n * K + k]))));
    for (int64_t i = 0; i < M; ++i) {
      double s = 0.0;
      for (int64_t k = 0; k < K; ++k) s += static_cast<double>(bf16_to_f32(x_bf16[i * K + k])) * wd[k];
      y[i * N + n] = s;
    }
  }
}

// W4A16 MSD linear layer (Alg. 2 + Tab. mxfp4-compute): two block-scaled FP4 GEMMs,
// y = sum_blocks 2^(ea+ew) <q1,w> + 2^(eb+ew) <q2,w>, in FP64, rounded once.
// mode 0: MSD two-pass;  mode 1: single-pass MXFP8 activations;  mode 2: unquantized activations.
void msdo_gemm_w4a16(const uint16_t* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, int64_t M, int64_t N,
                     int64_t K, int grid, double c_bound, int beta_shift, int mode, void* y, int ytype) {
  std::vector<double> xa(M * K);
  if (mode == 0) {
    std::vector<uint8_t> q1(M * K / 2), q2(M * K / 2), e1(M * K / 32), e2(M * K / 32);
    msdo_decompose_mxfp4(x_bf16, M, K, K, grid, c_bound, beta_shift, q1.data(), q2.data(), e1.data(), e2.data());
    msdo_mxfp4_reconstruct(q1.data(), q2.data(), e1.data(), e2.data(), M, K, grid, xa.data());
  } else if (mode == 1) {
    msdo_mxfp8_quantize(x_bf16, M, K, K, xa.data());
  } else {
    for (int64_t i = 0; i < M * K; ++i) xa[i] = bf16_to_f32(x_bf16[i]);
  }
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    std::vector<double> wd(K);
    for (int64_t k = 0; k < K; ++k)
      wd[k] = std::ldexp(fp4_value(nibble(w_fp4 + n * (K / 2), k), 0), w_e8m0[n * (K / 32) + k / 32] - kE8M0Bias);
    for (int64_t i = 0; i < M; ++i) {
      double s = 0.0;
      for (int64_t k = 0; k < K; ++k) s += xa[i * K + k] * wd[k];
      if (ytype == 0) static_cast<uint16_t*>(y)[i * N + n] = f64_to_bf16(s);
      else if (ytype == 1) static_cast<float*>(y)[i * N + n] = static_cast<float>(s);
      else static_cast<double*>(y)[i * N + n] = s;
    }
  }
}

// ---------------------------------------------------------------------------
// Decode attention over an INT8 KV cache (Sec. 4, Alg. 3) with one scale per token per KV head.
//
//   q_bf16 [B,Hq,D]; k [T,Hkv,D] INT8; v [T,Hkv,Dv] INT8 or NULL (V = first Dv entries of the K row);
//   k_scale [T,Hkv]; v_scale [T,Hkv] or NULL (= k_scale); cu_seqlens [B+1] token offsets.
//   mode 0  definition: one softmax over the whole context (Alg. 3 lines 6-12 with a global row max).
//   mode 1  tiled (Sec. 4.3): context cut at split_starts (per sequence, relative token offsets,
//           [B, n_splits+1], or with starts_per_head != 0 per sequence and query head, [B, Hq, n_splits+1];
//           unused trailing entries repeat the length), each split walked in tiles of
//           `tile` tokens with a running max; each tile quantises P against the running max in force
//           and with alpha_P = max(tile's v_scale)/127; splits merged with the usual log-sum-exp rule.
//   mode 4  tiled with held references (reading of Sec. 4.3 for kernels that keep integer PV sums across tiles):
//           as mode 1, but per split the reference maximum of a head moves only when a tile's maximum exceeds it,
//           to that maximum + m_margin, and alpha_P = a_ref/127 with a_ref a running bound of the value scales
//           that is set to sv_growth * (tile's largest value scale) when exceeded.  P <= 1 and P~ <= a_ref always
//           hold, so nothing clips; m_margin = 0, sv_growth = 1 is the plain online softmax with a running alpha_P.
//   mode 2  FP64 reference on the dequantized cache (no MSD).
//   mode 3  dequantize-to-BF16 comparison path (Sec. 6.4 "Dequant"): K,V -> bf16(q*s); P -> BF16 before PV.
// Per-token reading: s_K[j] multiplies score column j; s_V[j] is folded into P before decomposition.
// out [B,Hq,Dv] FP64 (unrounded); lse [B,Hq] nullable; s_dbg nullable: [2, Hq, T] INT32 QK^T accumulators.
// ---------------------------------------------------------------------------
void msdo_attn_decode_int8kv(const uint16_t* q_bf16, const int8_t* k, const int8_t* v, const float* k_scale,
                             const float* v_scale, const int32_t* cu_seqlens, int32_t B, int32_t Hq, int32_t Hkv,
                             int32_t D, int32_t Dv, float softmax_scale, int mode, int32_t tile,
                             const int32_t* split_starts, int32_t n_splits, double* out, double* lse,
                             int32_t* s_dbg, double m_margin, float sv_growth, int32_t starts_per_head) {
  const int64_t T = cu_seqlens[B];
  const int G = Hq / Hkv;
  const int8_t* vv = v ? v : k;
  const int64_t vstride = v ? Dv : D;
  const float* vs = v_scale ? v_scale : k_scale;
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
  for (int32_t b = 0; b < B; ++b)
    for (int32_t h = 0; h < Hq; ++h) {
      const int32_t hk = h / G;
      const int64_t t0 = cu_seqlens[b];
      const int64_t L = cu_seqlens[b + 1] - t0;
      double* o = out + (static_cast<int64_t>(b) * Hq + h) * Dv;
      for (int d = 0; d < Dv; ++d) o[d] = 0.0;
      if (lse) lse[static_cast<int64_t>(b) * Hq + h] = -std::numeric_limits<double>::infinity();
      if (L <= 0) continue;
      const uint16_t* qrow = q_bf16 + (static_cast<int64_t>(b) * Hq + h) * D;
      std::vector<double> S(L);
      if (mode <= 1 || mode == 4) {
        // lines 1-5: decompose Q, two exact integer products, merge
        std::vector<float> qf(D);
        for (int d = 0; d < D; ++d) qf[d] = bf16_to_f32(qrow[d]);
        std::vector<int8_t> q1(D), q2(D);
        float aq, bq;
        two_pass_int8(qf.data(), D, 1, -1.0f, q1.data(), q2.data(), &aq, &bq);
        for (int64_t j = 0; j < L; ++j) {
          const int8_t* kr = k + ((t0 + j) * Hkv + hk) * D;
          int64_t s1 = 0, s2 = 0;
          for (int d = 0; d < D; ++d) { s1 += q1[d] * kr[d]; s2 += q2[d] * kr[d]; }
          if (s_dbg) { s_dbg[static_cast<int64_t>(h) * T + t0 + j] = static_cast<int32_t>(s1);
                       s_dbg[(static_cast<int64_t>(Hq) + h) * T + t0 + j] = static_cast<int32_t>(s2); }
          S[j] = (static_cast<double>(aq) * s1 + static_cast<double>(bq) * s2) *
                 static_cast<double>(k_scale[(t0 + j) * Hkv + hk]) * static_cast<double>(softmax_scale);
        }
      } else {
        for (int64_t j = 0; j < L; ++j) {
          const int8_t* kr = k + ((t0 + j) * Hkv + hk) * D;
          double ks = k_scale[(t0 + j) * Hkv + hk];
          double s = 0.0;
          for (int d = 0; d < D; ++d) {
            double kd = (mode == 3) ? bf16_to_f32(f64_to_bf16(static_cast<double>(static_cast<float>(ks) * static_cast<float>(kr[d])))) : ks * kr[d];
            s += static_cast<double>(bf16_to_f32(qrow[d])) * kd;
          }
          S[j] = s * static_cast<double>(softmax_scale);
        }
      }
      if (mode == 2 || mode == 3) {
        double m = -std::numeric_limits<double>::infinity();
        for (int64_t j = 0; j < L; ++j) m = std::max(m, S[j]);
        double l = 0.0;
        for (int64_t j = 0; j < L; ++j) {
          double p = std::exp(S[j] - m);
          l += p;
          const int8_t* vr = vv + ((t0 + j) * Hkv + hk) * vstride;
          double sv = vs[(t0 + j) * Hkv + hk];
          if (mode == 3) p = bf16_to_f32(f64_to_bf16(p));
          for (int d = 0; d < Dv; ++d) {
            double vd = (mode == 3) ? bf16_to_f32(f64_to_bf16(static_cast<double>(static_cast<float>(sv) * static_cast<float>(vr[d])))) : sv * vr[d];
            o[d] += p * vd;
          }
        }
        for (int d = 0; d < Dv; ++d) o[d] /= l;
        if (lse) lse[static_cast<int64_t>(b) * Hq + h] = m + std::log(l);
        continue;
      }
      // MSD softmax + P decomposition + PV (lines 6-13)
      std::vector<int32_t> bounds;
      int64_t tl = L;
      if (mode == 0) { bounds = {0, static_cast<int32_t>(L)}; }
      else {
        const int64_t row = starts_per_head ? static_cast<int64_t>(b) * Hq + h : b;
        for (int s = 0; s <= n_splits; ++s) bounds.push_back(std::min<int64_t>(L, split_starts[row * (n_splits + 1) + s]));
        tl = tile;
      }
      double m_tot = -std::numeric_limits<double>::infinity(), l_tot = 0.0;
      std::vector<double> o_tot(Dv, 0.0);
      for (size_t s = 0; s + 1 < bounds.size(); ++s) {
        if (bounds[s + 1] <= bounds[s]) continue;
        double m_run = -std::numeric_limits<double>::infinity(), l_run = 0.0;
        float a_ref = 0.0f;                                  // mode 4: running bound of the value scales
        std::vector<double> o_run(Dv, 0.0);
        for (int64_t j0 = bounds[s]; j0 < bounds[s + 1]; j0 += tl) {
          int64_t j1 = std::min<int64_t>(bounds[s + 1], j0 + tl);
          double m_new = m_run;
          float sv_max = 0.0f;
          for (int64_t j = j0; j < j1; ++j) sv_max = std::max(sv_max, vs[(t0 + j) * Hkv + hk]);
          float alpha_p;
          if (mode <= 1) {
            for (int64_t j = j0; j < j1; ++j) m_new = std::max(m_new, S[j]);
            alpha_p = sv_max / 127.0f;                         // line 8 under per-token V scales
          } else {
            // mode 4, held references: the reference maximum moves only when a tile's maximum exceeds it and is then
            // set m_margin above that maximum (so P <= 1 still holds and later tiles rarely move it again); the
            // probability scale follows a running bound of the value scales that grows by the factor sv_growth when
            // exceeded.  Between such events both stay as they are, so integer PV sums of consecutive tiles share
            // one scale and one reference (Alg. 3 line 12 applied once per run of tiles instead of once per tile).
            double t_max = -std::numeric_limits<double>::infinity();
            for (int64_t j = j0; j < j1; ++j) t_max = std::max(t_max, S[j]);
            if (t_max > m_run) m_new = t_max + m_margin;
            if (sv_max > a_ref) a_ref = sv_max * sv_growth;
            alpha_p = a_ref / 127.0f;
          }
          double resc = std::exp(m_run - m_new);              // 0 on the first tile
          int64_t n = j1 - j0;
          std::vector<float> pt(n);
          double lsum = 0.0;
          for (int64_t j = j0; j < j1; ++j) {
            double p = std::exp(S[j] - m_new);                 // line 7
            lsum += p;
            pt[j - j0] = static_cast<float>(p) * vs[(t0 + j) * Hkv + hk];
          }
          std::vector<int8_t> p1(n), p2(n);
          float ap, bp;
          two_pass_int8(pt.data(), n, 1, alpha_p, p1.data(), p2.data(), &ap, &bp);   // line 9
          std::vector<int64_t> o1(Dv, 0), o2(Dv, 0);
          for (int64_t j = j0; j < j1; ++j) {
            const int8_t* vr = vv + ((t0 + j) * Hkv + hk) * vstride;
            for (int d = 0; d < Dv; ++d) { o1[d] += p1[j - j0] * vr[d]; o2[d] += p2[j - j0] * vr[d]; }   // lines 10-11
          }
          for (int d = 0; d < Dv; ++d)
            o_run[d] = o_run[d] * resc + static_cast<double>(ap) * o1[d] + static_cast<double>(bp) * o2[d];   // line 12 + rescale
          l_run = l_run * resc + lsum;
          m_run = m_new;
        }
        double m_new = std::max(m_tot, m_run);
        double w_old = std::exp(m_tot - m_new), w_new = std::exp(m_run - m_new);
        for (int d = 0; d < Dv; ++d) o_tot[d] = o_tot[d] * w_old + o_run[d] * w_new;
        l_tot = l_tot * w_old + l_run * w_new;
        m_tot = m_new;
      }
      for (int d = 0; d < Dv; ++d) o[d] = o_tot[d] / l_tot;       // line 13
      if (lse) lse[static_cast<int64_t>(b) * Hq + h] = m_tot + std::log(l_tot);
    }
}

}  // extern "C"

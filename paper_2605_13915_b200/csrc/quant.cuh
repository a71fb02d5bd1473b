// Element-wise INT8 quantisation shared by the decomposition kernel, the GEMM's in-kernel row decomposition and the
// attention kernel's query set-up.
#pragma once
#include <cuda_runtime.h>

namespace msd {

// clamp(rne(fl(v / scale)), -128, 127), bit for bit, without paying for an IEEE division per element:
// c = rne(v * (1/scale)) can differ from the rounded true quotient only when the quotient sits within a few ulps of a
// half-integer: |v*inv - v/scale| <= 127 * 2^-23 < 2^-16, so whenever the exact remainder v - scale*c is further than
// 2^-14 * scale from +-scale/2, c is the nearest integer of the true quotient with a margin that the quotient's own
// FP32 rounding (< 2^-17) cannot cross.  The rare elements inside that band take the true division.
__device__ __forceinline__ int quant_i8(float v, float scale, float inv_scale) {
  const float c = rintf(v * inv_scale);
  const float rem = __fmaf_rn(-scale, c, v);                  // exact for |c| <= 2^7 and BF16-derived inputs
  const float dist = fabsf(fabsf(rem) - 0.5f * scale);
  int q;
  if (dist > scale * 6.103515625e-05f && fabsf(c) <= 127.0f) q = __float2int_rn(c);
  else q = __float2int_rn(__fdiv_rn(v, scale));               // true division, round-half-to-even
  return max(-128, min(127, q));
}

// ---- 16 BF16 values (two 128-bit words) at a time: the unit of the row decomposition (Alg. 1 lines 1-5) ----
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ float chunk_absmax(const uint4& a, const uint4& b) {
  // |x| of a BF16 pair: clear both sign bits, then compare as floats
  float m = 0.0f;
  const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    m = fmaxf(m, fabsf(bf16lo(w[i])));
    m = fmaxf(m, fabsf(bf16hi(w[i])));
  }
  return m;
}

// Two-pass quantisation of 16 values; returns the packed codes of both passes.
__device__ __forceinline__ void chunk_quantize(const uint4& a, const uint4& b, float alpha, float beta, float inv_alpha,
                                               float inv_beta, uint4& o1, uint4& o2) {
  const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
  uint32_t p1[4] = {0, 0, 0, 0}, p2[4] = {0, 0, 0, 0};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float v = h ? bf16hi(w[i]) : bf16lo(w[i]);
      int c1 = 0, c2 = 0;
      if (alpha > 0.0f) {
        c1 = quant_i8(v, alpha, inv_alpha);                               // Eq. x1
        const float r = __fmaf_rn(-alpha, static_cast<float>(c1), v);     // Eq. residual, exact
        if (beta > 0.0f) c2 = quant_i8(r, beta, inv_beta);                // Eq. x2
      }
      const int e = 2 * i + h;
      p1[e >> 2] |= static_cast<uint32_t>(c1 & 0xFF) << (8 * (e & 3));
      p2[e >> 2] |= static_cast<uint32_t>(c2 & 0xFF) << (8 * (e & 3));
    }
  }
  o1 = make_uint4(p1[0], p1[1], p1[2], p1[3]);
  o2 = make_uint4(p2[0], p2[1], p2[2], p2[3]);
}

}  // namespace msd

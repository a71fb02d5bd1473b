// Element-wise INT8 quantisation shared by the decomposition kernel and the attention kernel's query set-up.
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

}  // namespace msd

// The per-column quantiser's code without a division per element (Section 4.6, per-column variant).
#pragma once

#include "twa_common.cuh"

// The quantiser's code of p without a division per element.  With r = RN(1 / s) the product q0 = p r
// lies within 2^-16 of the IEEE quotient p / s wherever the clamp to +-qmax (<= 127) does not decide
// the code anyway, so both round to the same integer unless q0 is that close to a half-integer; then,
// and only then, *hard is set and the caller takes the IEEE division.  The distance of q0 to the
// integer it rounds to is exact in float32.  Valid while r is finite (the caller checks s).
__device__ __forceinline__ int encode_by_reciprocal(float p, float r, float qmax, bool* hard) {
  const float q0 = fminf(fmaxf(p * r, -qmax), qmax);
  const float y = q0 + 12582912.0f;                    // 1.5 * 2^23: rounds to an integer, half to even
  const float t = q0 - (y - 12582912.0f);
  *hard = fabsf(t) >= 0.5f - 0x1p-15f;
  return __float_as_int(y) - 0x4B400000;
}

// RN(1 / s) when the reciprocal path is valid for the scale s, else 0 (every element then takes the
// division): s zero, or so small that its reciprocal is not finite or the error bound of
// encode_by_reciprocal, which assumes a normal s, does not hold.
__device__ __forceinline__ float encode_reciprocal(float s) { return s >= 0x1p-100f ? __frcp_rn(s) : 0.0f; }

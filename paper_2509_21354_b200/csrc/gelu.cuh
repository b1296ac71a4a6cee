// GELU in its exact (erf) form x * Phi(x) for the aggregator MLP kernels (Eq. 2).
#pragma once
#include <cuda_runtime.h>

namespace kve {

// erf by the rational-times-exponential formula 7.1.26 of Abramowitz & Stegun (absolute error below
// 1.5e-7, i.e. at the level of fp32 rounding of the activations), odd extension for x < 0
__device__ __forceinline__ float erf_as(float x) {
  const float ax = fabsf(x);
  const float t = __fdividef(1.f, fmaf(0.3275911f, ax, 1.f));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  const float y = 1.f - poly * t * __expf(-ax * ax);
  return copysignf(y, x);
}
__device__ __forceinline__ float gelu_tc(float x) { return 0.5f * x * (1.f + erf_as(x * 0.70710678118654752440f)); }

}  // namespace kve

// Elementwise math shared by the elementwise kernels and by the persistent dual-list kernel, so
// that both produce the same bits.
#pragma once

namespace erase {

// Phi(u) and phi(u) of the standard normal for the exact-erf GELU on bf16 data: erf from the
// Abramowitz-Stegun 7.1.26 rational form (|error| <= 1.5e-7, far below bf16 resolution) -- one
// reciprocal, one exponential and a 5-term polynomial shared by the value and the derivative,
// about half the instructions of erff + expf, which is what bounded the GELU passes (3.3 TB/s).
__device__ __forceinline__ void normal_cdf_pdf_fast(float u, float& cdf, float& pdf) {
  const float x = fabsf(u) * 0.70710678118654752f;
  const float t = __fdividef(1.f, fmaf(0.3275911f, x, 1.f));
  const float e = __expf(-0.5f * u * u);
  float q = fmaf(1.061405429f, t, -1.453152027f);
  q = fmaf(q, t, 1.421413741f);
  q = fmaf(q, t, -0.284496736f);
  q = fmaf(q, t, 0.254829592f);
  q = 0.5f * q * t * e;                 // (1 - erf(x)) / 2
  cdf = u >= 0.f ? 1.f - q : q;
  pdf = 0.39894228040143268f * e;
}
// GELU and its derivative on bf16 data (the value is rounded to bf16 by the caller)
__device__ __forceinline__ float gelu_bf16_value(float u) {
  float c, p;
  normal_cdf_pdf_fast(u, c, p);
  return u * c;
}
__device__ __forceinline__ float gelu_bf16_deriv(float u) {
  float c, p;
  normal_cdf_pdf_fast(u, c, p);
  return fmaf(u, p, c);
}

}  // namespace erase

// Device helpers shared by the GEMM epilogues: activations of Section 2 and
// typed conversions.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "ffsplit.h"

namespace ffsp {

__device__ __forceinline__ float gelu_erf_f(float z) { return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_tanh_f(float z) {
  const float u = 0.79788456080286536f * (z + 0.044715f * z * z * z);
  return 0.5f * z * (1.0f + tanhf(u));
}
__device__ __forceinline__ float silu_f(float z) { return z / (1.0f + __expf(-z)); }
__device__ __forceinline__ float silu_precise_f(float z) { return z / (1.0f + expf(-z)); }

// Fast GELU for bf16 outputs: x * Phi(x) ~ 0.5 x (1 + tanh(x (c0 + c1 x^2 + c2 x^4))) with one
// MUFU tanh.  For the erf definition (c0, c1, c2) are a minimax fit of atanh(erf(x / sqrt 2)) / x
// (max abs error of the fit 2.6e-5 with an exact tanh); for the tanh definition they are the
// definition's own constants.  x^2 is clamped at 36: beyond |x| = 6, Phi is 0 or 1 to 1e-9 and
// the clamp keeps the fitted polynomial positive.  tanh.approx.f32 adds up to 2^-11 relative.
struct GeluCoef { float c0, c1, c2; };
__device__ __forceinline__ GeluCoef gelu_coef(int act) {
  GeluCoef c;
  if (act == FFSPLIT_GELU_TANH) { c.c0 = 0.79788456080286536f; c.c1 = 0.035677408136300125f; c.c2 = 0.0f; }
  else { c.c0 = 7.97507884e-01f; c.c1 = 3.70056460e-02f; c.c2 = -3.51516789e-04f; }
  return c;
}
__device__ __forceinline__ float tanh_approx(float u) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return t;
}
__device__ __forceinline__ float gelu_fast(float x, const GeluCoef& c) {
  const float x2 = fminf(x * x, 36.0f);
  const float u = x * fmaf(fmaf(c.c2, x2, c.c1), x2, c.c0);
  const float hx = 0.5f * x;
  return fmaf(hx, tanh_approx(u), hx);
}
// The same for two values at once with the packed fp32 instructions of sm_100 (fma / mul on register pairs):
// every component goes through exactly the operations of gelu_fast, so the results are bit-identical, at
// 10 instead of 16 instructions per pair.
__device__ __forceinline__ float2 gelu_fast2(float2 x, const GeluCoef& c) {
  float2 x2 = __fmul2_rn(x, x);
  x2.x = fminf(x2.x, 36.0f);
  x2.y = fminf(x2.y, 36.0f);
  float2 t = __ffma2_rn(make_float2(c.c2, c.c2), x2, make_float2(c.c1, c.c1));
  t = __ffma2_rn(t, x2, make_float2(c.c0, c.c0));
  const float2 u = __fmul2_rn(x, t);
  const float2 hx = __fmul2_rn(make_float2(0.5f, 0.5f), x);
  const float2 th = make_float2(tanh_approx(u.x), tanh_approx(u.y));
  return __ffma2_rn(hx, th, hx);
}
// 16 values in place.
__device__ __forceinline__ void gelu_fast16(float* v, const GeluCoef& c) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float2 r = gelu_fast2(make_float2(v[2 * i], v[2 * i + 1]), c);
    v[2 * i] = r.x;
    v[2 * i + 1] = r.y;
  }
}
// SiLU with one MUFU: x * sigmoid(x) = 0.5 x (1 + tanh(x / 2)).
__device__ __forceinline__ float silu_fast(float x) {
  const float hx = 0.5f * x;
  return fmaf(hx, tanh_approx(hx), hx);
}

// GELU variants by runtime switch (uniform across the grid).
// GELU for the scoring pass of bf16 layers.  erf from the rational approximation 7.1.26 of Abramowitz and
// Stegun, erf(x) = 1 - (a1 t + ... + a5 t^5) exp(-x^2), t = 1 / (1 + p x), |error| <= 1.5e-7, with a fast
// reciprocal and exponential on top: about 1e-6 absolute in all, three orders below the bf16 rounding of the
// operands, at a third of erff's instructions.
__device__ __forceinline__ float gelu_erf_score_f(float z) {
  const float x = fabsf(z) * 0.70710678118654752f;
  const float t = __fdividef(1.0f, fmaf(0.3275911f, x, 1.0f));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  const float erf_abs = fmaf(-poly * t, __expf(-x * x), 1.0f);
  return 0.5f * z * (1.0f + copysignf(erf_abs, z));
}
// The square of the same GELU for two values at once, on the packed fp32 instructions: with
// q = (a1 t + ... + a5 t^5) exp(-x^2) / 2 (the coefficients carry the 1/2), Phi(z) = 1 - q for z >= 0 and q for z < 0,
// so GELU(z) = z Phi(z) without forming erf.  Ten instructions per value instead of nineteen; the same rational
// approximation, reciprocal and exponential, hence the same accuracy (about 1e-6 absolute).
__device__ __forceinline__ float2 gelu_erf_score_sq2(float2 z) {
  const float2 x = __fmul2_rn(make_float2(fabsf(z.x), fabsf(z.y)), make_float2(0.70710678118654752f, 0.70710678118654752f));
  const float2 den = __ffma2_rn(make_float2(0.3275911f, 0.3275911f), x, make_float2(1.0f, 1.0f));
  float2 t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t.x) : "f"(den.x));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t.y) : "f"(den.y));
  float2 poly = __ffma2_rn(make_float2(0.5f * 1.061405429f, 0.5f * 1.061405429f), t, make_float2(0.5f * -1.453152027f, 0.5f * -1.453152027f));
  poly = __ffma2_rn(poly, t, make_float2(0.5f * 1.421413741f, 0.5f * 1.421413741f));
  poly = __ffma2_rn(poly, t, make_float2(0.5f * -0.284496736f, 0.5f * -0.284496736f));
  poly = __ffma2_rn(poly, t, make_float2(0.5f * 0.254829592f, 0.5f * 0.254829592f));
  const float2 pt = __fmul2_rn(poly, t);
  const float2 ex = __fmul2_rn(__fmul2_rn(x, x), make_float2(-1.4426950408889634f, -1.4426950408889634f));
  float2 e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(ex.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(ex.y));
  const float2 q = __fmul2_rn(pt, e);
  const float2 om = __ffma2_rn(q, make_float2(-1.0f, -1.0f), make_float2(1.0f, 1.0f));
  const float2 phi = make_float2(z.x >= 0.f ? om.x : q.x, z.y >= 0.f ? om.y : q.y);
  const float2 g = __fmul2_rn(z, phi);
  return __fmul2_rn(g, g);
}
__device__ __forceinline__ float act_gelu_score(float z, int act) {
  return act == FFSPLIT_GELU_TANH ? gelu_tanh_f(z) : gelu_erf_score_f(z);
}

__device__ __forceinline__ float act_gelu(float z, int act) {
  return act == FFSPLIT_GELU_TANH ? gelu_tanh_f(z) : gelu_erf_f(z);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

}  // namespace ffsp

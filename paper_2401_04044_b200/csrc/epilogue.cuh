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

// GELU variants by runtime switch (uniform across the grid).
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

// Device helpers shared by the scan kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "m2rnn.h"

namespace m2rnn {

// Forget gate f and its derivative w.r.t. the gate tensor entry (forget-gate equation).
// VALUE: f = x.  LOGIT: f = sigmoid(x).  PSI: f = (1+e^{x+beta})^{-alpha}, evaluated as
// exp(-alpha*softplus(x+beta)) so neither tail overflows; df/dx = -alpha*sigmoid(x+beta)*f.
__device__ __forceinline__ float gate_value(int kind, float x, float alpha, float beta, float *dfdx) {
  float f, d;
  if (kind == M2RNN_GATE_VALUE) {
    f = x;
    d = 1.0f;
  } else if (kind == M2RNN_GATE_LOGIT) {
    if (x >= 0.f) {
      f = 1.0f / (1.0f + expf(-x));
    } else {
      float e = expf(x);
      f = e / (1.0f + e);
    }
    d = f * (1.0f - f);
  } else {
    float u = x + beta;
    float sp = (u > 0.f) ? u + log1pf(expf(-u)) : log1pf(expf(u));
    float sg = (u >= 0.f) ? 1.0f / (1.0f + expf(-u)) : expf(u) / (1.0f + expf(u));
    f = expf(-alpha * sp);
    d = -alpha * sg * f;
  }
  if (dfdx) *dfdx = d;
  return f;
}

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

}  // namespace m2rnn

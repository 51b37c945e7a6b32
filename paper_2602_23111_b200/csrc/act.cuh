// Derivatives of the element-wise activations whose backward pass can run on a rebuilt input
// (Section 5.1, non-linear layers): SiLU f(x) = x sigmoid(x) and GeLU f(x) = x Phi(x).
#pragma once
#include <cuda_runtime.h>

namespace prac {

enum : int { ACT_SILU = 0, ACT_GELU = 1 };

__device__ __forceinline__ float act_derivative(float x, int act) {
  if (act == ACT_SILU) {
    const float sg = 1.f / (1.f + expf(-x));
    return sg * fmaf(x, 1.f - sg, 1.f);
  }
  const float Phi = 0.5f * (1.f + erff(x * 0.70710678118654752f));
  const float phi = 0.39894228040143268f * expf(-0.5f * x * x);
  return fmaf(x, phi, Phi);
}

// The same with the hardware exponential and the approximate reciprocal (relative error ~1e-6;
// one instruction each), the activation fixed at compile time: for results that are rounded to
// bf16 anyway.
__device__ __forceinline__ float rcp_approx(float y) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y));
  return r;
}
template <int ACT>
__device__ __forceinline__ float act_derivative_fast(float x) {
  if (ACT == ACT_SILU) {
    const float sg = rcp_approx(1.f + __expf(-x));
    return sg * fmaf(x, 1.f - sg, 1.f);
  }
  const float Phi = 0.5f * (1.f + erff(x * 0.70710678118654752f));
  const float phi = 0.39894228040143268f * __expf(-0.5f * x * x);
  return fmaf(x, phi, Phi);
}

}  // namespace prac

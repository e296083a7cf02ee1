// Elementwise arithmetic of the virtual instructions (Table 1) in fp32, shared by the vector
// interpreter and the epilogue interpreter of the matmul meta-kernel.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "dvm_format.h"

namespace dvm {

__device__ __forceinline__ float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// exp(x) = 2^(x * log2 e) with the product carried in two fp32 pieces (t exact to 2^-24 |t|, plus the
// rounding residual of the multiply and the low part of log2 e), the power of two from the SFU
// (ex2.approx, relative error <= 2^-22) and a first-order correction: about 3e-7 relative error over the
// whole finite range, in 7 instructions instead of expf's ~12.
__device__ __forceinline__ float fast_exp(float x) {
  const float L2E_HI = 1.44269502162933349609375f, L2E_LO = 1.925963033500011e-8f;
  const float t = x * L2E_HI;
  float r = __fmaf_rn(x, L2E_HI, -t);
  r = __fmaf_rn(x, L2E_LO, r);
  float p;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p) : "f"(t));
  // outside the finite range (t = +-inf from a masked score, overflow, NaN) the SFU value stands alone:
  // exp(-inf) must be exactly +0
  return fabsf(t) < 126.0f ? __fmaf_rn(p * r, 0.693147182464599609375f, p) : p;
}
// reciprocal and quotient from the SFU (rcp.approx, 1 ulp): 2 ulp quotients
__device__ __forceinline__ float fast_rcp(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float fast_div(float a, float b) { return __fdividef(a, b); }

__device__ __forceinline__ float scalar_arith(int op, float a, float b) {
  switch (op) {
    case DVM_A_ADD: return a + b;
    case DVM_A_SUB: return a - b;
    case DVM_A_RSUB: return b - a;
    case DVM_A_MUL: return a * b;
    case DVM_A_DIV: return fast_div(a, b);
    case DVM_A_RDIV: return fast_div(b, a);
    case DVM_A_MIN: return a < b ? a : b;
    default: return a > b ? a : b;
  }
}

__device__ __forceinline__ float scalar_unary(int op, float x) {
  switch (op) {
    case DVM_U_EXP: return fast_exp(x);
    case DVM_U_SQRT: return sqrtf(x);
    case DVM_U_RSQRT: return rsqrtf(x);
    case DVM_U_ABS: return fabsf(x);
    case DVM_U_LOG: return logf(x);
    case DVM_U_ERF: return erff(x);
    case DVM_U_SIGMOID: return fast_rcp(1.0f + fast_exp(-x));
    case DVM_U_NEG: return -x;
    case DVM_U_RECIP: return fast_rcp(x);
    case DVM_U_FLOOR: return floorf(x);
    case DVM_U_ROUND: return rintf(x);
    case DVM_U_TANH: return tanhf(x);
    case DVM_U_ISFINITE: return fabsf(x) < __int_as_float(0x7f800000) ? 1.0f : 0.0f;  // false for NaN, too
    default: return round_bf16(x);
  }
}

}  // namespace dvm

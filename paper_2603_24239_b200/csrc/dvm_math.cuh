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

// erf(x) on pairs, branch-free: x * P(x^2) for |x| < 1, sign(x) * (1 - 2^Q(min(|x|, 4))) beyond (erfc(4) is below
// half an ulp of 1).  P (degree 6 in x^2) and Q (degree 9) are Chebyshev-node least-squares fits of
// erf(sqrt(s)) / sqrt(s) on [0, 1] and of log2(erfc(x)) on [1, 4]; evaluated in fp32 the absolute error stays
// below 1.5e-7 and the relative error below 2e-7 (checked against a float64 erf on 4e6 points).
__device__ __forceinline__ float2 packed_erf(float2 x) {
#define DVM_C2(v) make_float2(v, v)
  const float2 s = __fmul2_rn(x, x);
  float2 p = DVM_C2(7.882497448008507e-05f);
  p = __ffma2_rn(p, s, DVM_C2(-0.0008018855005502701f));
  p = __ffma2_rn(p, s, DVM_C2(0.005189312156289816f));
  p = __ffma2_rn(p, s, DVM_C2(-0.02685432881116867f));
  p = __ffma2_rn(p, s, DVM_C2(0.11283597350120544f));
  p = __ffma2_rn(p, s, DVM_C2(-0.3761262595653534f));
  p = __ffma2_rn(p, s, DVM_C2(1.1283791065216064f));
  const float2 small = __fmul2_rn(p, x);
  const float2 ax = make_float2(fabsf(x.x), fabsf(x.y));
  const float2 xc = make_float2(fminf(ax.x, 4.0f), fminf(ax.y, 4.0f));
  float2 q = DVM_C2(-9.497055231122431e-08f);   // the coefficients of -log2(erfc), negated: q = log2(erfc)
  q = __ffma2_rn(q, xc, DVM_C2(4.465436177270021e-06f));
  q = __ffma2_rn(q, xc, DVM_C2(-8.666094799991697e-05f));
  q = __ffma2_rn(q, xc, DVM_C2(0.0009714207262732089f));
  q = __ffma2_rn(q, xc, DVM_C2(-0.007243836298584938f));
  q = __ffma2_rn(q, xc, DVM_C2(0.038952041417360306f));
  q = __ffma2_rn(q, xc, DVM_C2(-0.160005584359169f));
  q = __ffma2_rn(q, xc, DVM_C2(-0.9104687571525574f));
  q = __ffma2_rn(q, xc, DVM_C2(-1.6311174631118774f));
  q = __ffma2_rn(q, xc, DVM_C2(0.0005778000340797007f));
  float2 e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(q.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(q.y));
  const float2 big = __ffma2_rn(e, DVM_C2(-1.0f), DVM_C2(1.0f));
#undef DVM_C2
  return make_float2(ax.x >= 1.0f ? copysignf(big.x, x.x) : small.x, ax.y >= 1.0f ? copysignf(big.y, x.y) : small.y);  // (a NaN takes the product's way)
}

// Table 1, Cast to an integer type, as an fp32 value: the fraction dropped toward zero (+ 0: one zero), then kept
// inside the type's range (2^31 stands for the largest i32: the store's conversion saturates); NaN gives 0.
// the stored forms: an i32 word, a byte (conversions toward zero that saturate; NaN gives 0)
__device__ __forceinline__ uint32_t store_i32(float x) { return (uint32_t)__float2int_rz(x); }
__device__ __forceinline__ uint32_t store_u8(float x) { return min(__float2uint_rz(x), 255u); }
__device__ __forceinline__ uint32_t pack_u8x4(float a, float b, float c, float d) {
  return store_u8(a) | (store_u8(b) << 8) | (store_u8(c) << 16) | (store_u8(d) << 24);
}
__device__ __forceinline__ float trunc_i32(float x) { return x != x ? 0.0f : fminf(fmaxf(truncf(x) + 0.0f, -2147483648.0f), 2147483648.0f); }
__device__ __forceinline__ float trunc_u8(float x) { return x != x ? 0.0f : fminf(fmaxf(truncf(x) + 0.0f, 0.0f), 255.0f); }

// The fused activations (DVM_OP_ACT), on pairs.  Every step rounds as the separate instructions would.
__device__ __forceinline__ float2 packed_gelu(float2 t) {
  const float2 e = packed_erf(__fmul2_rn(t, make_float2(0.707106769084930419921875f, 0.707106769084930419921875f)));
  const float2 u = __fadd2_rn(e, make_float2(1.0f, 1.0f));
  return __fmul2_rn(__fmul2_rn(t, u), make_float2(0.5f, 0.5f));
}
__device__ __forceinline__ float2 packed_silu(float2 t) {
  return make_float2(t.x * fast_rcp(1.0f + fast_exp(-t.x)), t.y * fast_rcp(1.0f + fast_exp(-t.y)));
}

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
    case DVM_U_ERF: return packed_erf(make_float2(x, x)).x;
    case DVM_U_SIGMOID: return fast_rcp(1.0f + fast_exp(-x));
    case DVM_U_NEG: return -x;
    case DVM_U_RECIP: return fast_rcp(x);
    case DVM_U_FLOOR: return floorf(x);
    case DVM_U_ROUND: return rintf(x);
    case DVM_U_TANH: return tanhf(x);
    case DVM_U_ISFINITE: return fabsf(x) < __int_as_float(0x7f800000) ? 1.0f : 0.0f;  // false for NaN, too
    case DVM_U_TRUNC_I32: return trunc_i32(x);
    case DVM_U_TRUNC_U8: return trunc_u8(x);
    default: return round_bf16(x);
  }
}

}  // namespace dvm

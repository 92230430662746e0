// Element-level epilogues shared by the GEMM kernels, and small vector-store helpers.
#pragma once

#include "wf_internal.h"
#include "wf_ptx.cuh"

namespace wf {

// Exact (erf-form) GELU: 0.5 u (1 + erf(u / sqrt 2)).
__device__ __forceinline__ float gelu_erf(float u) {
  return 0.5f * u * (1.0f + erff(u * 0.70710678118654752f));
}

// GELU for bf16 outputs: x * sigmoid(p(x)) with the odd polynomial
// p(x) = x (1.5950158 + 0.0740113 x^2 - 0.00070304 x^4) fitted to logit(Phi(x)) (max absolute
// deviation of x * sigmoid(p(x)) from the erf form: 2.6e-5 over the real line), evaluated as
// 0.5 x (1 + tanh(p(x) / 2)) with the hardware tanh: one special-function instruction per element
// instead of an exponential and a reciprocal.  tanh.approx is good to 2^-11 relative, which adds
// at most 2.5e-4 |x| to the result: an eighth of the bf16 rounding step of large outputs, and
// below 8e-4 in absolute terms on the negative tail where the result itself is under 0.17.
__device__ __forceinline__ float gelu_sigmoid_poly(float x) {
  constexpr float c0 = 0.5f * 1.5950157568597356f, c1 = 0.5f * 0.07401130190182707f,
                  c2 = -0.5f * 0.0007030350661891551f;
  const float xc = fminf(fmaxf(x, -8.0f), 8.0f);  // keeps the quartic from turning p over for |x| > 8.6
  const float x2 = xc * xc;
  float t = fmaf(x2, c2, c1);
  t = fmaf(x2, t, c0);
  float th;
  asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(xc * t));
  const float hx = 0.5f * x;
  return fmaf(hx, th, hx);
}

// The same for two values at once with two-wide float32 instructions (half the arithmetic
// instructions; the epilogue warps share their schedulers with the MMA and TMA threads).
__device__ __forceinline__ void gelu_sigmoid_poly2(float& x0, float& x1) {
  constexpr float c0 = 0.5f * 1.5950157568597356f, c1 = 0.5f * 0.07401130190182707f,
                  c2 = -0.5f * 0.0007030350661891551f;
  const uint64_t x = ptx::pack_f32x2(x0, x1);
  float q0, q1;
  ptx::unpack_f32x2(ptx::mul_f32x2(x, x), q0, q1);
  // x^2 capped at 64 keeps the quartic positive; the argument then keeps growing with |x| and the
  // tanh saturates on the right side
  const uint64_t x2 = ptx::pack_f32x2(fminf(q0, 64.0f), fminf(q1, 64.0f));
  uint64_t t = ptx::fma_f32x2(x2, ptx::pack_f32x2(c2, c2), ptx::pack_f32x2(c1, c1));
  t = ptx::fma_f32x2(x2, t, ptx::pack_f32x2(c0, c0));
  float a0, a1, th0, th1;
  ptx::unpack_f32x2(ptx::mul_f32x2(x, t), a0, a1);
  asm("tanh.approx.f32 %0, %1;" : "=f"(th0) : "f"(a0));
  asm("tanh.approx.f32 %0, %1;" : "=f"(th1) : "f"(a1));
  const uint64_t hx = ptx::mul_f32x2(x, ptx::pack_f32x2(0.5f, 0.5f));
  ptx::unpack_f32x2(ptx::fma_f32x2(hx, ptx::pack_f32x2(th0, th1), hx), x0, x1);
}

__device__ __forceinline__ void store_elem(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_elem(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// One output element of C = epilogue(acc).  `row`/`col` are GEMM coordinates.
template <int EPI, typename OutT>
__device__ __forceinline__ void epilogue_store(const EpiParams& ep, long row, int col, float acc) {
  float v = acc + __ldg(ep.bias + col);
  if (EPI == kEpiBias) {
    store_elem(reinterpret_cast<OutT*>(ep.out) + row * ep.ldc + col, v);
  } else if (EPI == kEpiBiasGelu) {
    store_elem(reinterpret_cast<OutT*>(ep.out) + row * ep.ldc + col, gelu_erf(v));
  } else if (EPI == kEpiBiasResid) {
    float* p = ep.resid + row * ep.ldc + col;
    *p = *p + v;
  } else if (EPI == kEpiConv1) {
    store_elem(reinterpret_cast<OutT*>(ep.out) + row * ep.ldc + col,
               ep.row_valid[row] ? gelu_erf(v) : 0.0f);
  } else {  // kEpiConv2
    int2 d = ep.row_dst[row];
    if (d.x >= 0) ep.resid[(long)d.x * ep.ldc + col] = gelu_erf(v) + __ldg(ep.pe + (long)d.y * ep.ldc + col);
  }
}

}  // namespace wf

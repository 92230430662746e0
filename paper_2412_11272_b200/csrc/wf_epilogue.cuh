// Element-level epilogues shared by the GEMM kernels, and small vector-store helpers.
#pragma once

#include "wf_internal.h"

namespace wf {

// Exact (erf-form) GELU: 0.5 u (1 + erf(u / sqrt 2)).
__device__ __forceinline__ float gelu_erf(float u) {
  return 0.5f * u * (1.0f + erff(u * 0.70710678118654752f));
}

// GELU for bf16 outputs: x * sigmoid(p(x)) with the odd polynomial
// p(x) = x (1.5950158 + 0.0740113 x^2 - 0.00070304 x^4) fitted to logit(Phi(x)); the argument of p
// is clamped to [-8, 8] (beyond, sigmoid is 0 or 1 to 1e-12).  Max absolute deviation from the
// erf form: 2.6e-5 over the real line, two orders of magnitude under bf16 rounding of the result.
__device__ __forceinline__ float gelu_sigmoid_poly(float x) {
  constexpr float kL2e = 1.4426950408889634f;
  constexpr float c0 = -1.5950157568597356f * kL2e, c1 = -0.07401130190182707f * kL2e,
                  c2 = 0.0007030350661891551f * kL2e;
  float xc = fminf(fmaxf(x, -8.0f), 8.0f);
  float x2 = xc * xc;
  float t = fmaf(x2, c2, c1);
  t = fmaf(x2, t, c0);
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(xc * t));
  return __fdividef(x, 1.0f + e);
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

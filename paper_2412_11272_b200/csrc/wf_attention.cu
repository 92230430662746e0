// Non-causal variable-length attention for bf16 activations, head dimension 64.
//
// One CTA = 64 query rows of one (sequence, head); 4 warps x 16 rows.  Keys and values of
// that sequence only are streamed in tiles of 64 through a double-buffered, XOR-swizzled
// shared-memory ring (cp.async); scores and outputs are accumulated with warp-level bf16
// MMAs in float32, softmax is the online (running max / running sum) form in base 2.
// Rows are addressed through the token prefix sums, so no padded token is ever touched.
#include "wf_internal.h"
#include "wf_ptx.cuh"

namespace wf {

using namespace ptx;

constexpr int kAttnQ = 64;
constexpr int kAttnK = 64;

__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Copies rows r0 .. r0+63 (64 bf16 each) of one head's q, k or v into a swizzled tile.
// Rows at or beyond n are zero-filled.
__device__ __forceinline__ void load_tile(uint32_t smem_tile, const __nv_bfloat16* base, long ld, int r0,
                                          int n, int tid) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int idx = tid + 128 * i;
    int row = idx >> 3, chunk = idx & 7;
    int grow = r0 + row;
    bool valid = grow < n;
    const __nv_bfloat16* src = base + (long)(valid ? grow : n - 1) * ld + chunk * 8;
    cp_async_16(smem_tile + swz(row, chunk), src, valid);
  }
}

__global__ void __launch_bounds__(128) attention_bf16_kernel(const __nv_bfloat16* __restrict__ qkv,
                                                             __nv_bfloat16* __restrict__ out,
                                                             const int* __restrict__ meta, MetaLayout ml,
                                                             int d_model) {
  __shared__ __align__(1024) uint8_t smem[5 * 8192];  // Q | K0 | K1 | V0 | V1
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK = sQ + 8192, sV = sQ + 3 * 8192;

  const int seq = meta[ml.attn_work + 2 * blockIdx.x];
  const int q0 = meta[ml.attn_work + 2 * blockIdx.x + 1];
  const int head = blockIdx.y;
  const int tok0 = meta[ml.tok_off + seq];
  const int n = meta[ml.tok_off + seq + 1] - tok0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q4 = lane & 3;
  const long ld = 3L * d_model;
  const __nv_bfloat16* qb = qkv + (long)tok0 * ld + head * kHeadDim;
  const __nv_bfloat16* kb = qb + d_model;
  const __nv_bfloat16* vb = qb + 2 * d_model;
  const int n_kt = (n + kAttnK - 1) / kAttnK;

  load_tile(sQ, qb, ld, q0, n, tid);
  load_tile(sK, kb, ld, 0, n, tid);
  load_tile(sV, vb, ld, 0, n, tid);
  cp_async_commit();

  uint32_t qf[4][4];
  float o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[j][e] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  const float scale = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) and log2(e)

  for (int kt = 0; kt < n_kt; ++kt) {
    const int buf = kt & 1;
    if (kt + 1 < n_kt) {
      load_tile(sK + (buf ^ 1) * 8192, kb, ld, (kt + 1) * kAttnK, n, tid);
      load_tile(sV + (buf ^ 1) * 8192, vb, ld, (kt + 1) * kAttnK, n, tid);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (kt == 0) {
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        int chunk = 2 * ks + (lane >> 4);
        ldmatrix_x4(sQ + swz(row, chunk), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    const uint32_t tK = sK + buf * 8192, tV = sV + buf * 8192;

    float s[8][4];
#pragma unroll
    for (int t = 0; t < 8; ++t)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[t][e] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        int row = 16 * jp + (lane & 7) + ((lane >> 4) & 1) * 8;
        int chunk = 2 * ks + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(tK + swz(row, chunk), b0, b1, b2, b3);
        mma_bf16_16816(s[2 * jp], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b0, b1);
        mma_bf16_16816(s[2 * jp + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b2, b3);
      }
    }
    const int kbase = kt * kAttnK;
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int key = kbase + 8 * t + 2 * q4 + (e & 1);
        float v = key < n ? s[t][e] * scale : -INFINITY;
        s[t][e] = v;
        if (e < 2) mx_lo = fmaxf(mx_lo, v); else mx_hi = fmaxf(mx_hi, v);
      }
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);  // finite: key kbase < n
    const float c_lo = exp2f(m_lo - mn_lo), c_hi = exp2f(m_hi - mn_hi);
    m_lo = mn_lo;
    m_hi = mn_hi;
    float rs_lo = 0.f, rs_hi = 0.f;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      s[t][0] = exp2f(s[t][0] - mn_lo);
      s[t][1] = exp2f(s[t][1] - mn_lo);
      s[t][2] = exp2f(s[t][2] - mn_hi);
      s[t][3] = exp2f(s[t][3] - mn_hi);
      rs_lo += s[t][0] + s[t][1];
      rs_hi += s[t][2] + s[t][3];
    }
    l_lo = l_lo * c_lo + rs_lo;
    l_hi = l_hi * c_hi + rs_hi;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      o[j][0] *= c_lo; o[j][1] *= c_lo;
      o[j][2] *= c_hi; o[j][3] *= c_hi;
    }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t a0 = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
      uint32_t a1 = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
      uint32_t a2 = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      uint32_t a3 = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        int row = 16 * kk + (lane & 7) + ((lane >> 3) & 1) * 8;
        int chunk = 2 * jp + (lane >> 4);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(tV + swz(row, chunk), b0, b1, b2, b3);
        mma_bf16_16816(o[2 * jp], a0, a1, a2, a3, b0, b1);
        mma_bf16_16816(o[2 * jp + 1], a0, a1, a2, a3, b2, b3);
      }
    }
    __syncthreads();  // this buffer is refilled by the loads issued in the next iteration
  }

  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const float i_lo = 1.0f / l_lo, i_hi = 1.0f / l_hi;
  const int r_lo = q0 + warp * 16 + g, r_hi = r_lo + 8;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    int col = head * kHeadDim + 8 * j + 2 * q4;
    if (r_lo < n)
      *reinterpret_cast<uint32_t*>(out + (long)(tok0 + r_lo) * d_model + col) = pack_bf16(o[j][0] * i_lo, o[j][1] * i_lo);
    if (r_hi < n)
      *reinterpret_cast<uint32_t*>(out + (long)(tok0 + r_hi) * d_model + col) = pack_bf16(o[j][2] * i_hi, o[j][3] * i_hi);
  }
}

cudaError_t attention_bf16_configure() { return cudaSuccess; }

void launch_attention_bf16(const __nv_bfloat16* qkv, __nv_bfloat16* out, const int* meta, MetaLayout ml,
                           int n_work, int d_model, cudaStream_t s) {
  if (n_work <= 0) return;
  dim3 grid(n_work, d_model / kHeadDim);
  attention_bf16_kernel<<<grid, 128, 0, s>>>(qkv, out, meta, ml, d_model);
}

}  // namespace wf

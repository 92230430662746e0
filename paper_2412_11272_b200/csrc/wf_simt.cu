// float32 SIMT kernels (the float32 encoder path), LayerNorm, and weight-layout conversion.
#include "wf_internal.h"
#include "wf_epilogue.cuh"
#include "wf_ptx.cuh"

namespace wf {

// ---------------------------------------------------------------------------------------------
// C = epilogue(A W^T): A [M, K] with row pitch lda (pitch < K gives the overlapping-row view
// the conv stem uses), W [N, K] with pitch ldw.  64 x 64 x 16 tiles, 4 x 4 outputs per thread.
// K, lda, ldw multiples of 4 and 16-byte aligned bases (checked by the caller).
template <int EPI>
__global__ void __launch_bounds__(256) gemm_f32_kernel(const float* __restrict__ A, long lda,
                                                       const float* __restrict__ W, long ldw, long M,
                                                       int N, int K, EpiParams ep) {
  __shared__ __align__(16) float As[16][68];
  __shared__ __align__(16) float Bs[16][68];
  const int tid = threadIdx.x;
  const long m0 = (long)blockIdx.y * 64;
  const int n0 = blockIdx.x * 64;
  const int lrow = tid >> 2, lk = (tid & 3) * 4;
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += 16) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (m0 + lrow < M && k0 + lk < K) a = *reinterpret_cast<const float4*>(A + (m0 + lrow) * lda + k0 + lk);
    if (n0 + lrow < N && k0 + lk < K) b = *reinterpret_cast<const float4*>(W + (long)(n0 + lrow) * ldw + k0 + lk);
    As[lk + 0][lrow] = a.x; As[lk + 1][lrow] = a.y; As[lk + 2][lrow] = a.z; As[lk + 3][lrow] = a.w;
    Bs[lk + 0][lrow] = b.x; Bs[lk + 1][lrow] = b.y; Bs[lk + 2][lrow] = b.z; Bs[lk + 3][lrow] = b.w;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      float ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    long row = m0 + ty * 4 + i;
    if (row >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int col = n0 + tx * 4 + j;
      if (col < N) epilogue_store<EPI, float>(ep, row, col, acc[i][j]);
    }
  }
}

void launch_gemm_f32(const float* A, long lda, const float* W, long ldw, long M, int N, int K, int epi,
                     const EpiParams& ep, cudaStream_t s) {
  if (M <= 0 || N <= 0) return;
  dim3 grid((N + 63) / 64, (unsigned)((M + 63) / 64));
  switch (epi) {
    case kEpiBias: gemm_f32_kernel<kEpiBias><<<grid, 256, 0, s>>>(A, lda, W, ldw, M, N, K, ep); break;
    case kEpiBiasGelu: gemm_f32_kernel<kEpiBiasGelu><<<grid, 256, 0, s>>>(A, lda, W, ldw, M, N, K, ep); break;
    case kEpiBiasResid: gemm_f32_kernel<kEpiBiasResid><<<grid, 256, 0, s>>>(A, lda, W, ldw, M, N, K, ep); break;
    case kEpiConv1: gemm_f32_kernel<kEpiConv1><<<grid, 256, 0, s>>>(A, lda, W, ldw, M, N, K, ep); break;
    default: gemm_f32_kernel<kEpiConv2><<<grid, 256, 0, s>>>(A, lda, W, ldw, M, N, K, ep); break;
  }
}

// ---------------------------------------------------------------------------------------------
// LayerNorm over d = 128 NV channels, one warp per row, the row held in registers
// (mean, then centred sum of squares: no cancellation), biased variance, eps 1e-5.
// SPLIT: the row is read from the two bf16 planes of the bf16 path's residual stream (x = hi + lo).
template <int NV, bool SPLIT, typename OutT>
__global__ void __launch_bounds__(256) layernorm_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ x_hi,
                                                        const __nv_bfloat16* __restrict__ x_lo,
                                                        const float* __restrict__ g,
                                                        const float* __restrict__ b,
                                                        OutT* __restrict__ out, long M) {
  ptx::griddep_wait();
  ptx::griddep_launch_dependents();
  const long row = (long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  constexpr int d = NV * 128;
  float4 v[NV];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    if (SPLIT) {
      const uint2 h = *reinterpret_cast<const uint2*>(x_hi + row * d + (lane + 32 * i) * 4);
      const uint2 l = *reinterpret_cast<const uint2*>(x_lo + row * d + (lane + 32 * i) * 4);
      v[i].x = __uint_as_float(h.x << 16) + __uint_as_float(l.x << 16);
      v[i].y = __uint_as_float(h.x & 0xffff0000u) + __uint_as_float(l.x & 0xffff0000u);
      v[i].z = __uint_as_float(h.y << 16) + __uint_as_float(l.y << 16);
      v[i].w = __uint_as_float(h.y & 0xffff0000u) + __uint_as_float(l.y & 0xffff0000u);
    } else {
      v[i] = reinterpret_cast<const float4*>(x + row * d)[lane + 32 * i];
    }
    sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float mean = sum * (1.0f / d);
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    v[i].x -= mean; v[i].y -= mean; v[i].z -= mean; v[i].w -= mean;
    sq += (v[i].x * v[i].x + v[i].y * v[i].y) + (v[i].z * v[i].z + v[i].w * v[i].w);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float rstd = rsqrtf(sq * (1.0f / d) + 1e-5f);
  const float4* g4 = reinterpret_cast<const float4*>(g);
  const float4* b4 = reinterpret_cast<const float4*>(b);
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    float4 gg = __ldg(g4 + lane + 32 * i), bb = __ldg(b4 + lane + 32 * i);
    float4 y;
    y.x = v[i].x * rstd * gg.x + bb.x;
    y.y = v[i].y * rstd * gg.y + bb.y;
    y.z = v[i].z * rstd * gg.z + bb.z;
    y.w = v[i].w * rstd * gg.w + bb.w;
    store4(out + row * d + (lane + 32 * i) * 4, y);
  }
}

template <bool SPLIT, typename OutT>
static void layernorm_dispatch(const float* x, const __nv_bfloat16* x_hi, const __nv_bfloat16* x_lo, const float* g,
                               const float* b, OutT* out, long M, int d, bool pdl, cudaStream_t s) {
  unsigned grid = (unsigned)((M + 7) / 8);
#define WF_LN_CASE(NV) \
  case NV: launch_dependent(layernorm_kernel<NV, SPLIT, OutT>, dim3(grid), dim3(256), 0, s, 1, pdl, x, x_hi, x_lo, g, b, out, M); break;
  switch (d / 128) {
    WF_LN_CASE(1) WF_LN_CASE(2) WF_LN_CASE(3) WF_LN_CASE(4) WF_LN_CASE(5)
    WF_LN_CASE(6) WF_LN_CASE(7) WF_LN_CASE(8) WF_LN_CASE(9) WF_LN_CASE(10)
    default: break;  // create() rejects d_model > 1280
  }
#undef WF_LN_CASE
}

void launch_layernorm(const float* x, const float* g, const float* b, float* out, long M, int d, cudaStream_t s) {
  if (M <= 0) return;
  layernorm_dispatch<false, float>(x, nullptr, nullptr, g, b, out, M, d, false, s);
}

void launch_layernorm_split(const __nv_bfloat16* x_hi, const __nv_bfloat16* x_lo, const float* g, const float* b,
                            __nv_bfloat16* out, long M, int d, bool pdl, cudaStream_t s) {
  if (M <= 0) return;
  layernorm_dispatch<true, __nv_bfloat16>(nullptr, x_hi, x_lo, g, b, out, M, d, pdl, s);
}

// ---------------------------------------------------------------------------------------------
// Create-time fold of a LayerNorm's affine part into the weight that follows it; one CTA per
// output row n: wg[n,k] = bf16(W[n,k] g[k]), colsum[n] = sum_k float(wg[n,k]) (of the rounded
// values: the GEMM epilogue's mean * colsum then cancels the common mode of x exactly as the
// tensor core saw it), cbias[n] = bias[n] + sum_k W[n,k] b[k].
__global__ void __launch_bounds__(256) ln_fold_kernel(const float* __restrict__ W, const float* __restrict__ g,
                                                      const float* __restrict__ b, const float* __restrict__ bias,
                                                      __nv_bfloat16* __restrict__ wg, float* __restrict__ colsum,
                                                      float* __restrict__ cbias, int K) {
  __shared__ float red[2][8];
  const int n = blockIdx.x, tid = threadIdx.x;
  float s = 0.f, c = 0.f;
  for (int k = tid; k < K; k += 256) {
    const float w = W[(long)n * K + k];
    const __nv_bfloat16 q = __float2bfloat16_rn(w * g[k]);
    wg[(long)n * K + k] = q;
    s += __bfloat162float(q);
    c = fmaf(w, b[k], c);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    c += __shfl_xor_sync(0xffffffffu, c, o);
  }
  if ((tid & 31) == 0) { red[0][tid >> 5] = s; red[1][tid >> 5] = c; }
  __syncthreads();
  if (tid == 0) {
    float ts = 0.f, tc = 0.f;
    for (int i = 0; i < 8; ++i) { ts += red[0][i]; tc += red[1][i]; }
    colsum[n] = ts;
    cbias[n] = tc + (bias ? bias[n] : 0.f);
  }
}
void launch_ln_fold(const float* W, const float* g, const float* b, const float* bias, __nv_bfloat16* wg,
                    float* colsum, float* cbias, int N, int K, cudaStream_t s) {
  if (N <= 0) return;
  ln_fold_kernel<<<N, 256, 0, s>>>(W, g, b, bias, wg, colsum, cbias, K);
}

// ---------------------------------------------------------------------------------------------
// float32 attention: one CTA = 16 queries of one (sequence, head); 8 warps x 2 queries.  Keys
// and values are staged 64 at a time; scores are lane-per-key, outputs lane-per-channel.
__global__ void __launch_bounds__(256) attention_f32_kernel(const float* __restrict__ qkv,
                                                            float* __restrict__ out,
                                                            const int* __restrict__ meta,
                                                            MetaLayout ml, int d_model) {
  __shared__ float Ks[64][65];
  __shared__ float Vs[64][64];
  __shared__ float Qs[16][64];
  __shared__ float Ps[8][2][64];
  const int seq = meta[ml.attn_work + 2 * blockIdx.x];
  const int q0 = meta[ml.attn_work + 2 * blockIdx.x + 1];
  const int head = blockIdx.y;
  const int tok0 = meta[ml.tok_off + seq];
  const int n = meta[ml.tok_off + seq + 1] - tok0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long ld = 3L * d_model;
  const float* qb = qkv + (long)tok0 * ld + head * kHeadDim;
  const float* kb = qb + d_model;
  const float* vb = qb + 2 * d_model;

  for (int i = tid; i < 16 * 64; i += 256) {
    int r = i >> 6, c = i & 63;
    Qs[r][c] = (q0 + r < n) ? qb[(long)(q0 + r) * ld + c] * 0.125f : 0.f;
  }
  float m_run[2], l_run[2], o0[2], o1[2];
#pragma unroll
  for (int qi = 0; qi < 2; ++qi) { m_run[qi] = -INFINITY; l_run[qi] = 0.f; o0[qi] = 0.f; o1[qi] = 0.f; }

  for (int k0 = 0; k0 < n; k0 += 64) {
    __syncthreads();
    for (int i = tid; i < 64 * 64; i += 256) {
      int r = i >> 6, c = i & 63;
      bool ok = k0 + r < n;
      Ks[r][c] = ok ? kb[(long)(k0 + r) * ld + c] : 0.f;
      Vs[r][c] = ok ? vb[(long)(k0 + r) * ld + c] : 0.f;
    }
    __syncthreads();
    float sc[2][2];
#pragma unroll
    for (int qi = 0; qi < 2; ++qi) { sc[qi][0] = 0.f; sc[qi][1] = 0.f; }
    for (int c = 0; c < 64; ++c) {
      float ka = Ks[lane][c], kb2 = Ks[lane + 32][c];
#pragma unroll
      for (int qi = 0; qi < 2; ++qi) {
        float qv = Qs[warp * 2 + qi][c];
        sc[qi][0] = fmaf(qv, ka, sc[qi][0]);
        sc[qi][1] = fmaf(qv, kb2, sc[qi][1]);
      }
    }
#pragma unroll
    for (int qi = 0; qi < 2; ++qi) {
      if (k0 + lane >= n) sc[qi][0] = -INFINITY;
      if (k0 + lane + 32 >= n) sc[qi][1] = -INFINITY;
      float mx = fmaxf(sc[qi][0], sc[qi][1]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float m_new = fmaxf(m_run[qi], mx);  // finite: key k0 is always inside the sequence
      float p0 = expf(sc[qi][0] - m_new), p1 = expf(sc[qi][1] - m_new);
      float ps = p0 + p1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      float corr = expf(m_run[qi] - m_new);
      l_run[qi] = l_run[qi] * corr + ps;
      o0[qi] *= corr; o1[qi] *= corr;
      m_run[qi] = m_new;
      Ps[warp][qi][lane] = p0;
      Ps[warp][qi][lane + 32] = p1;
    }
    __syncwarp();
    for (int key = 0; key < 64; ++key) {
      float v0 = Vs[key][lane], v1 = Vs[key][lane + 32];
#pragma unroll
      for (int qi = 0; qi < 2; ++qi) {
        float p = Ps[warp][qi][key];
        o0[qi] = fmaf(p, v0, o0[qi]);
        o1[qi] = fmaf(p, v1, o1[qi]);
      }
    }
    __syncwarp();
  }
#pragma unroll
  for (int qi = 0; qi < 2; ++qi) {
    int q = q0 + warp * 2 + qi;
    if (q < n) {
      float inv = 1.0f / l_run[qi];
      float* orow = out + (long)(tok0 + q) * d_model + head * kHeadDim;
      orow[lane] = o0[qi] * inv;
      orow[lane + 32] = o1[qi] * inv;
    }
  }
}

void launch_attention_f32(const float* qkv, float* out, const int* meta, MetaLayout ml, int n_work,
                          int d_model, cudaStream_t s) {
  if (n_work <= 0) return;
  dim3 grid(n_work, d_model / kHeadDim);
  attention_f32_kernel<<<grid, 256, 0, s>>>(qkv, out, meta, ml, d_model);
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait every tensor-core kernel of the library relies on: one warp waits,
// with the same wait routine but a caller-chosen poll limit, on an mbarrier that nobody ever
// arrives on.  The wait must run out, raise the shared abort flag and return; the kernel then
// records role code 21 in the device error word and ends normally.  No TMA, no tensor memory.
__global__ void __launch_bounds__(32) wait_selftest_kernel(int* err_flag, uint32_t poll_limit) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncwarp();
  const bool ok = ptx::mbar_wait_limited(ptx::smem_u32(&bar), 0, &abort_flag, poll_limit);
  if (!__all_sync(0xffffffffu, ok) && threadIdx.x == 0) atomicExch(err_flag, 21);
}
void launch_wait_selftest(int* err_flag, unsigned poll_limit, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(err_flag, poll_limit);
}

// ---------------------------------------------------------------------------------------------
// Weight conversion at create time.
template <typename OutT>
__global__ void convert_kernel(const float* __restrict__ src, OutT* __restrict__ dst, long n) {
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n; i += (long)gridDim.x * blockDim.x)
    dst[i] = (OutT)src[i];
}
void launch_convert(const float* src, void* dst, long n, int dst_bf16, cudaStream_t s) {
  if (n <= 0) return;
  if (dst_bf16) convert_kernel<__nv_bfloat16><<<592, 256, 0, s>>>(src, (__nv_bfloat16*)dst, n);
  else convert_kernel<float><<<592, 256, 0, s>>>(src, (float*)dst, n);
}

// Conv kernel [out, in, 3] -> GEMM weight [out, 3 * in_ld] with column index tap * in_ld + channel,
// matching an activation row that is three consecutive time rows (of in_ld channels, the
// ones beyond `in` being zero) laid end to end.  dst is zeroed by the caller.
template <typename OutT>
__global__ void conv_weight_kernel(const float* __restrict__ src, OutT* __restrict__ dst, int c_out,
                                   int c_in, int in_ld) {
  long total = (long)c_out * c_in * 3;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    int j = (int)(i % 3);
    long rest = i / 3;
    int c = (int)(rest % c_in);
    long o = rest / c_in;
    dst[o * 3L * in_ld + (long)j * in_ld + c] = (OutT)src[i];
  }
}
void launch_conv_weight(const float* src, void* dst, int c_out, int c_in, int in_ld, int dst_bf16,
                        cudaStream_t s) {
  if (dst_bf16) conv_weight_kernel<__nv_bfloat16><<<592, 256, 0, s>>>(src, (__nv_bfloat16*)dst, c_out, c_in, in_ld);
  else conv_weight_kernel<float><<<592, 256, 0, s>>>(src, (float*)dst, c_out, c_in, in_ld);
}

__global__ void transpose_f32_kernel(const float* __restrict__ src, float* __restrict__ dst, int rows,
                                     int cols) {
  long total = (long)rows * cols;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    int r = (int)(i / cols), c = (int)(i % cols);
    dst[(long)c * rows + r] = src[i];
  }
}
void launch_transpose_f32(const float* src, float* dst, int rows, int cols, cudaStream_t s) {
  transpose_f32_kernel<<<64, 256, 0, s>>>(src, dst, rows, cols);
}

}  // namespace wf

// Dynamic time warping of token-by-frame cost matrices (token timestamping, Sec. 3.2 / Sec. 4.3.2).
//
// One CTA per problem.  D[i,j] = C[i,j] + min(D[i-1,j-1], D[i-1,j], D[i,j-1]) is swept along
// anti-diagonals (cells of one anti-diagonal are independent); only the last two diagonals of D
// live in shared memory, the arg-min of every cell goes to a byte matrix in global memory, and
// one thread walks it back from the last cell, recording the first frame of every token.
// Accumulation is float32 in the order written above; ties prefer the diagonal, then the step
// in the token index, then the step in the frame index.
#include "wf_internal.h"

namespace wf {

constexpr int kDtwThreads = 256;

// meta per problem: cost offset (cells), n_tok, n_frm, token offset
__global__ void __launch_bounds__(kDtwThreads) dtw_kernel(const float* __restrict__ cost,
                                                          const int* __restrict__ meta,
                                                          unsigned char* __restrict__ trace,
                                                          int* __restrict__ token_start,
                                                          float* __restrict__ total_cost) {
  extern __shared__ float diag[];  // 3 x n_tok floats
  const int b = blockIdx.x;
  const long off = meta[4 * b];
  const int N = meta[4 * b + 1], M = meta[4 * b + 2], tok0 = meta[4 * b + 3];
  const float* C = cost + off;
  unsigned char* T = trace + off;
  float* d0 = diag;            // diagonal k
  float* d1 = diag + N;        // diagonal k - 1
  float* d2 = diag + 2 * N;    // diagonal k - 2
  const float inf = __int_as_float(0x7f800000);
  for (int k = 0; k < N + M - 1; ++k) {
    const int i_lo = max(0, k - (M - 1)), i_hi = min(N - 1, k);
    for (int i = i_lo + threadIdx.x; i <= i_hi; i += blockDim.x) {
      const int j = k - i;
      float v;
      unsigned char s = 0;
      if (k == 0) {
        v = C[0];
      } else {
        float best = (i > 0 && j > 0) ? d2[i - 1] : inf;
        const float up = i > 0 ? d1[i - 1] : inf;      // (i-1, j) lies on diagonal k-1
        const float left = j > 0 ? d1[i] : inf;        // (i, j-1) lies on diagonal k-1
        if (up < best) { best = up; s = 1; }
        if (left < best) { best = left; s = 2; }
        v = C[(long)i * M + j] + best;
      }
      d0[i] = v;
      T[(long)i * M + j] = s;
    }
    __syncthreads();
    float* t = d2; d2 = d1; d1 = d0; d0 = t;  // rotate: every thread does the same swap
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    total_cost[b] = d1[N - 1];  // after the last rotation d1 holds the final diagonal
    int i = N - 1, j = M - 1;
    token_start[tok0 + i] = j;
    while (i > 0 || j > 0) {
      const unsigned char s = T[(long)i * M + j];
      if (s == 0) { --i; --j; }
      else if (s == 1) { --i; }
      else { --j; }
      token_start[tok0 + i] = j;  // walking backwards: the last write for a token is its first frame
    }
  }
}

cudaError_t launch_dtw(const float* cost, const int* meta, int B, int max_tok, unsigned char* trace,
                       int* token_start, float* total_cost, cudaStream_t s) {
  if (B <= 0) return cudaSuccess;
  const size_t smem = 3 * (size_t)max_tok * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(dtw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dtw_kernel<<<B, kDtwThreads, smem, s>>>(cost, meta, trace, token_start, total_cost);
  return cudaGetLastError();
}

}  // namespace wf

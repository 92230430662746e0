// Dynamic time warping of token-by-frame cost matrices (token timestamping, Sec. 3.2 / Sec. 4.3.2).
//
// One CTA per problem.  D[i,j] = C[i,j] + min(D[i-1,j-1], D[i-1,j], D[i,j-1]) is swept along
// anti-diagonals (cells of one anti-diagonal are independent); only the last two diagonals of D
// live in shared memory, the arg-min of every cell goes to a byte matrix (in shared memory when
// the problem fits, else in global memory), and
// one thread walks it back from the last cell, recording the first frame of every token.
// Accumulation is float32 in the order written above; ties prefer the diagonal, then the step
// in the token index, then the step in the frame index.
#include "wf_internal.h"

namespace wf {

constexpr int kDtwThreads = 256;
constexpr int kDtwPrefetch = 8;               // anti-diagonals whose costs are in flight ahead of the sweep
constexpr size_t kDtwSmemLimit = 220 * 1024;  // below this the arg-min bytes stay in shared memory

// meta per problem: cost offset (cells), n_tok, n_frm, token offset.
// Every thread's first cell of an anti-diagonal is fetched kDtwPrefetch diagonals ahead into
// registers, so the sweep's step time is one barrier plus a few shared-memory accesses instead of
// one global-memory round trip.  kSmemTrace keeps the arg-min bytes of the whole problem in
// shared memory (the walk back then never leaves the SM); otherwise they go to `trace`.
template <bool kSmemTrace>
__global__ void __launch_bounds__(kDtwThreads) dtw_kernel(const float* __restrict__ cost,
                                                          const int* __restrict__ meta,
                                                          unsigned char* __restrict__ trace,
                                                          int* __restrict__ token_start,
                                                          float* __restrict__ total_cost) {
  extern __shared__ float diag[];  // 3 x n_tok floats, then (kSmemTrace) n_tok x n_frm bytes
  const int b = blockIdx.x;
  const long off = meta[4 * b];
  const int N = meta[4 * b + 1], M = meta[4 * b + 2], tok0 = meta[4 * b + 3];
  const int K = N + M - 1;
  const float* C = cost + off;
  unsigned char* T = kSmemTrace ? reinterpret_cast<unsigned char*>(diag + 3 * N) : trace + off;
  float* d0 = diag;            // diagonal k
  float* d1 = diag + N;        // diagonal k - 1
  float* d2 = diag + 2 * N;    // diagonal k - 2
  const float inf = __int_as_float(0x7f800000);
  const int tid = threadIdx.x;
  auto first_cost = [&](int k) -> float {
    const int i = max(0, k - (M - 1)) + tid;
    return (k < K && i <= min(N - 1, k)) ? __ldg(C + (long)i * M + (k - i)) : 0.f;
  };
  float cur[kDtwPrefetch], nxt[kDtwPrefetch];
#pragma unroll
  for (int p = 0; p < kDtwPrefetch; ++p) cur[p] = first_cost(p);
  for (int k0 = 0; k0 < K; k0 += kDtwPrefetch) {
#pragma unroll
    for (int p = 0; p < kDtwPrefetch; ++p) nxt[p] = first_cost(k0 + kDtwPrefetch + p);
#pragma unroll
    for (int p = 0; p < kDtwPrefetch; ++p) {
      const int k = k0 + p;
      if (k >= K) break;  // the same for every thread
      const int i_lo = max(0, k - (M - 1)), i_hi = min(N - 1, k);
      for (int i = i_lo + tid; i <= i_hi; i += kDtwThreads) {
        const int j = k - i;
        const float c = (i == i_lo + tid) ? cur[p] : __ldg(C + (long)i * M + j);
        float v;
        unsigned char s = 0;
        if (k == 0) {
          v = c;
        } else {
          float best = (i > 0 && j > 0) ? d2[i - 1] : inf;
          const float up = i > 0 ? d1[i - 1] : inf;      // (i-1, j) lies on diagonal k-1
          const float left = j > 0 ? d1[i] : inf;        // (i, j-1) lies on diagonal k-1
          if (up < best) { best = up; s = 1; }
          if (left < best) { best = left; s = 2; }
          v = c + best;
        }
        d0[i] = v;
        T[(long)i * M + j] = s;
      }
      __syncthreads();
      float* t = d2; d2 = d1; d1 = d0; d0 = t;  // rotate: every thread does the same swap
    }
#pragma unroll
    for (int p = 0; p < kDtwPrefetch; ++p) cur[p] = nxt[p];
  }
  __syncthreads();
  if (tid == 0) {
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

cudaError_t launch_dtw(const float* cost, const int* meta, int B, int max_tok, long max_cells,
                       unsigned char* trace, int* token_start, float* total_cost, cudaStream_t s) {
  if (B <= 0) return cudaSuccess;
  const size_t diag_bytes = 3 * (size_t)max_tok * sizeof(float);
  const bool in_smem = diag_bytes + (size_t)max_cells <= kDtwSmemLimit;
  const size_t smem = diag_bytes + (in_smem ? (size_t)max_cells : 0);
  auto kernel = in_smem ? dtw_kernel<true> : dtw_kernel<false>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  kernel<<<B, kDtwThreads, smem, s>>>(cost, meta, trace, token_start, total_cost);
  return cudaGetLastError();
}

}  // namespace wf

// Log-mel front end: tables, framing + windowed DFT (as a folded real GEMM) + mel + log10,
// per-buffer normalisation, hush append and the padded-row layout the conv stem reads.
//
// The front end of Sec. 4.1.2 ("target level": 16 kHz audio -> 100 log-mel rows per second).
// All arithmetic is float32: the clamp at (max - 8) exposes 80 dB of dynamic range, which
// bfloat16 products cannot resolve.
#include "wf_internal.h"
#include "wf_ptx.cuh"

namespace wf {

// ---------------------------------------------------------------------------------------------
// Tables.  The periodic Hann window is symmetric (w[n] = w[400-n], w[0] = 0), so with
// e[n] = s[n] + s[400-n], o[n] = s[n] - s[400-n] (n = 1..199), e[200] = s[200]:
//   Re X[k] =  sum_{n=1}^{200} w[n] cos(2 pi k n / 400) e[n]
//   Im X[k] = -sum_{n=1}^{199} w[n] sin(2 pi k n / 400) o[n]
// basis[0][n-1][k] holds the cosine factors, basis[1][n-1][k] the sine factors (row 199 zero).
__global__ void build_tables_kernel(float* basis, float* pe, int n_ctx, int d) {
  const long n_basis = 2L * kFold * kBasisCols;
  const long n_pe = (long)n_ctx * d;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n_basis + n_pe;
       i += (long)gridDim.x * blockDim.x) {
    if (i < n_basis) {
      int which = (int)(i / (kFold * kBasisCols));
      int r = (int)(i % (kFold * kBasisCols));
      int n = r / kBasisCols + 1;
      int k = r % kBasisCols;
      double v = 0.0;
      if (k < kBins) {
        double w = 0.5 - 0.5 * cospi(2.0 * n / 400.0);
        int a = (k * n) % kNFft;  // exact angle reduction
        if (which == 0) v = w * cospi(2.0 * a / 400.0);
        else v = (n == kFold) ? 0.0 : w * sinpi(2.0 * a / 400.0);
      }
      basis[i] = (float)v;
    } else {
      long j = i - n_basis;
      int p = (int)(j / d), c = (int)(j % d);
      int half = d / 2;
      int ch = c < half ? c : c - half;
      double inv = exp(-log(10000.0) / (half - 1) * ch);
      double ang = (double)p * inv;
      pe[j] = (float)(c < half ? sin(ang) : cos(ang));
    }
  }
}

void launch_build_tables(float* dft_basis, float* pe, int n_ctx, int d, cudaStream_t s) {
  build_tables_kernel<<<296, 256, 0, s>>>(dft_basis, pe, n_ctx, d);
}

// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int float_to_ordered(float f) {
  int i = __float_as_int(f);
  return i >= 0 ? i : i ^ 0x7FFFFFFF;
}
__device__ __forceinline__ float ordered_to_float(int i) {
  return __int_as_float(i >= 0 ? i : i ^ 0x7FFFFFFF);
}

__global__ void fill_seq_max_kernel(int* seq_max, int B) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B) seq_max[i] = (int)0x80000000;
}
void launch_fill_seq_max(int* seq_max, int B, cudaStream_t s) {
  if (B > 0) fill_seq_max_kernel<<<(B + 255) / 256, 256, 0, s>>>(seq_max, B);
}

// One CTA = 64 consecutive frames of one buffer.  Phase 1 folds the reflected frames into
// shared memory; phase 2 is the [64 x 200] x [200 x 201] cosine and sine products with an
// 8-frame x 7-bin register tile per thread; phase 3 squares into shared memory; phase 4 is
// the mel projection, log10 and the per-buffer running maximum.
constexpr int kPStride = 204;
constexpr int kBasisChunk = 8;  // folded-DFT rows per staged chunk (a multiple of 4 that divides 200)
constexpr int kFeSpan = kHop * (kFeFrames - 1) + 399;  // samples one tile of frames touches
constexpr int kFeSmemFloats = kFeFrames * kPStride > 2 * kFeFrames * kFold ? kFeFrames * kPStride : 2 * kFeFrames * kFold;

__global__ void __launch_bounds__(256) frontend_kernel(
    const float* __restrict__ audio, const int* __restrict__ meta, MetaLayout ml, int B,
    const float* __restrict__ basis, const float* __restrict__ fbt, int n_mel,
    float* __restrict__ logmel, int* __restrict__ seq_max, const float* __restrict__ tail, int tail_len) {
  extern __shared__ __align__(16) float smem[];
  float* e_s = smem;                       // [64][200]
  float* o_s = smem + kFeFrames * kFold;   // [64][200]
  float* p_s = smem;                       // [64][204] after the DFT
  float* b_s = smem + kFeSmemFloats;       // [2 buffers][cos, sin][kBasisChunk][224] staged basis rows

  int seq, t0;
  if (ml.fe_tiles != 0) {  // explicit tile list (resident stream windows: only some frames are recomputed)
    seq = meta[ml.fe_tiles + 2 * blockIdx.x];
    t0 = meta[ml.fe_tiles + 2 * blockIdx.x + 1];
  } else {
    const int* tile_off = meta + ml.fe_tile_off;
    int tile = blockIdx.x;
    int lo = 0, hi = B - 1;
    while (lo < hi) {  // last sequence whose first tile is <= tile
      int mid = (lo + hi + 1) >> 1;
      if (tile_off[mid] <= tile) lo = mid; else hi = mid - 1;
    }
    seq = lo;
    t0 = (tile - tile_off[seq]) * kFeFrames;
  }
  const int T = meta[ml.frames + seq];
  const int s0 = meta[ml.sample_off + seq];
  const int L_audio = ml.fe_len != 0 ? meta[ml.fe_len + seq] : meta[ml.sample_off + seq + 1] - s0;
  const int L = L_audio + tail_len;  // the buffer followed by the raw-audio hush word, if any
  const float* x = audio + s0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // The tile's samples (with the reflected ends and the raw-audio hush word resolved) go to shared
  // memory once, coalesced; the fold then reads every sample twice from there instead of from
  // global memory.
  {
    float* span = smem + kFeSmemFloats + 2 * 2 * kBasisChunk * kBasisCols;
    const int p0 = kHop * t0 - 199;  // span[i] is sample p0 + i
#pragma unroll 4
    for (int i = tid; i < kFeSpan; i += 256) {
      int p = p0 + i;
      if (p < 0) p = -p;
      if (p >= L) p = 2 * (L - 1) - p;
      p = min(max(p, 0), L - 1);  // only for frames past the end of the buffer, which are not used
      span[i] = p < L_audio ? x[p] : tail[p - L_audio];
    }
    __syncthreads();
    for (int idx = tid; idx < kFeFrames * kFold; idx += 256) {
      const int f = idx / kFold, n = idx % kFold + 1;
      float e = 0.f, o = 0.f;
      if (t0 + f < T) {
        const float a = span[kHop * f - 1 + n];          // sample c - 200 + n, c = 160 (t0 + f)
        if (n == kFold) { e = a; }
        else { const float b = span[kHop * f + 399 - n]; e = a + b; o = a - b; }  // sample c + 200 - n
      }
      e_s[idx] = e;
      o_s[idx] = o;
    }
  }
  __syncthreads();

  float acc_r[8][7], acc_i[8][7];
#pragma unroll
  for (int f = 0; f < 8; ++f)
#pragma unroll
    for (int j = 0; j < 7; ++j) { acc_r[f][j] = 0.f; acc_i[f][j] = 0.f; }

  // The cosine / sine rows are staged through shared memory kBasisChunk at a time (cp.async, double
  // buffered): all eight warps read the same rows, and fetching them per warp through the L1 made
  // this loop wait on the L1 rather than on the FMA pipe.
  auto stage_basis = [&](int chunk, int buf) {
    float* dst = b_s + buf * (2 * kBasisChunk * kBasisCols);
    const int rows = min(kBasisChunk, kFold - chunk * kBasisChunk);
    const int vec_per_half = rows * kBasisCols / 4;  // 16-byte pieces of the cosine (or sine) rows
    for (int v = tid; v < 2 * vec_per_half; v += 256) {
      const int half = v >= vec_per_half ? 1 : 0, idx = v - half * vec_per_half;
      ptx::cp_async_16(ptx::smem_u32(dst + half * kBasisChunk * kBasisCols + 4 * idx),
                       basis + (size_t)half * kFold * kBasisCols + (size_t)chunk * kBasisChunk * kBasisCols + 4 * idx,
                       true);
    }
    ptx::cp_async_commit();
  };
  const float* er = e_s + warp * 8 * kFold;
  const float* orow = o_s + warp * 8 * kFold;
  constexpr int kChunks = (kFold + kBasisChunk - 1) / kBasisChunk;
  stage_basis(0, 0);
  for (int ch = 0; ch < kChunks; ++ch) {
    if (ch + 1 < kChunks) {
      stage_basis(ch + 1, (ch + 1) & 1);
      ptx::cp_async_wait<1>();
    } else {
      ptx::cp_async_wait<0>();
    }
    __syncthreads();  // chunk ch has landed for every thread
    const float* bc = b_s + (ch & 1) * (2 * kBasisChunk * kBasisCols) + lane;
    const float* bs = bc + kBasisChunk * kBasisCols;
    const int n_lo = ch * kBasisChunk, n_hi = min(kFold, n_lo + kBasisChunk);
    for (int n4 = n_lo; n4 < n_hi; n4 += 4) {
      float4 ev[8], ov[8];
#pragma unroll
      for (int f = 0; f < 8; ++f) {
        ev[f] = *reinterpret_cast<const float4*>(er + f * kFold + n4);
        ov[f] = *reinterpret_cast<const float4*>(orow + f * kFold + n4);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float c[7], s[7];
#pragma unroll
        for (int j = 0; j < 7; ++j) {
          c[j] = bc[(n4 - n_lo + u) * kBasisCols + 32 * j];
          s[j] = bs[(n4 - n_lo + u) * kBasisCols + 32 * j];
        }
#pragma unroll
        for (int f = 0; f < 8; ++f) {
          float e = u == 0 ? ev[f].x : u == 1 ? ev[f].y : u == 2 ? ev[f].z : ev[f].w;
          float o = u == 0 ? ov[f].x : u == 1 ? ov[f].y : u == 2 ? ov[f].z : ov[f].w;
#pragma unroll
          for (int j = 0; j < 7; ++j) {
            acc_r[f][j] = fmaf(e, c[j], acc_r[f][j]);
            acc_i[f][j] = fmaf(o, s[j], acc_i[f][j]);
          }
        }
      }
    }
    __syncthreads();  // everyone is done with this buffer before chunk ch + 2 overwrites it
  }
  __syncthreads();  // every warp is done with e_s / o_s before p_s overwrites them
#pragma unroll
  for (int f = 0; f < 8; ++f)
#pragma unroll
    for (int j = 0; j < 7; ++j) {
      int k = lane + 32 * j;
      if (k < kBins) p_s[(warp * 8 + f) * kPStride + k] = acc_r[f][j] * acc_r[f][j] + acc_i[f][j] * acc_i[f][j];
    }
  __syncwarp();  // a warp only reads back its own 8 rows

  float mel[8][4];
#pragma unroll
  for (int f = 0; f < 8; ++f)
#pragma unroll
    for (int j = 0; j < 4; ++j) mel[f][j] = 0.f;
  const float* pr = p_s + warp * 8 * kPStride;
  // Filterbanks are sparse (a channel is fed by a short run of neighbouring bins): the first and
  // last bin with a non-zero weight of every channel sit behind the transposed filterbank, and a
  // lane walks only its channels' runs, in ascending bin order as the full product would (the
  // skipped products would have added exact zeros; lanes past the end of their run add one).
  const int2* bin_range = reinterpret_cast<const int2*>(fbt + kBins * n_mel);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = lane + 32 * j;
    const int2 rg = m < n_mel ? __ldg(bin_range + m) : make_int2(0, 0);
    int len = rg.y - rg.x;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) len = max(len, __shfl_xor_sync(0xffffffffu, len, o));
    for (int kk = 0; kk < len; ++kk) {
      const int k = rg.x + kk;
      const bool in_run = k < rg.y;
      const int kc = in_run ? k : 0;
      const float wj = in_run ? __ldg(fbt + kc * n_mel + m) : 0.f;
#pragma unroll
      for (int f = 0; f < 8; ++f) mel[f][j] = fmaf(pr[f * kPStride + kc], wj, mel[f][j]);
    }
  }
  float mx = -INFINITY;
  const long frame0 = meta[ml.frame_off + seq];
#pragma unroll
  for (int f = 0; f < 8; ++f) {
    int t = t0 + warp * 8 + f;
    if (t < T) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int m = lane + 32 * j;
        if (m < n_mel) {
          float lg = log10f(fmaxf(mel[f][j], 1e-10f));
          logmel[(frame0 + t) * n_mel + m] = lg;
          mx = fmaxf(mx, lg);
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0 && mx > -INFINITY) atomicMax(seq_max + seq, float_to_ordered(mx));
}

constexpr int kFeSmemBytes = (kFeSmemFloats + 2 * 2 * kBasisChunk * kBasisCols + kFeSpan + 1) * (int)sizeof(float);  // 172,992 B

// Function attributes are per device: called by every create, on the device that is current then.
cudaError_t frontend_configure() {
  return cudaFuncSetAttribute(frontend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFeSmemBytes);
}

void launch_frontend(const float* audio, const int* meta, MetaLayout ml, int B, int n_tiles,
                     const float* dft_basis, const float* mel_fb_t, int n_mel, float* logmel,
                     int* seq_max, const float* tail, int tail_len, cudaStream_t s) {
  if (n_tiles > 0)
    frontend_kernel<<<n_tiles, 256, kFeSmemBytes, s>>>(audio, meta, ml, B, dft_basis, mel_fb_t, n_mel, logmel,
                                                seq_max, tail, tail_len);
}

// ---------------------------------------------------------------------------------------------
// Resident stream windows (the audio buffer of a stream grows at its end every round and is cut
// at its front now and then, Sec. 3.2): samples and un-normalised log-mel rows stay on the device
// between rounds, and only the frames whose 400 samples changed are recomputed.

// Drops `cut` floats at the front of a slice of `count` floats, in place.  One CTA per slice
// walks it front to back; a chunk is read completely (into registers) before it is written, and
// it is written to addresses below everything that is still to be read.
constexpr int kShiftPerThread = 32;
__global__ void __launch_bounds__(256) stream_shift_kernel(float* __restrict__ base_audio,
                                                           float* __restrict__ base_logmel,
                                                           const int* __restrict__ entries_audio,
                                                           const int* __restrict__ entries_logmel) {
  const int* en = (blockIdx.y == 0 ? entries_audio : entries_logmel) + 3 * blockIdx.x;
  float* a = (blockIdx.y == 0 ? base_audio : base_logmel) + en[0];
  const int cut = en[1], count = en[2];
  if (cut <= 0) return;
  const int keep = count - cut;
  for (int c0 = 0; c0 < keep; c0 += 256 * kShiftPerThread) {
    float v[kShiftPerThread];
#pragma unroll
    for (int u = 0; u < kShiftPerThread; ++u) {
      const int i = c0 + u * 256 + threadIdx.x;
      v[u] = i < keep ? a[cut + i] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kShiftPerThread; ++u) {
      const int i = c0 + u * 256 + threadIdx.x;
      if (i < keep) a[i] = v[u];
    }
  }
}

void launch_stream_shift(float* base_audio, float* base_logmel, const int* entries_audio, const int* entries_logmel,
                         int n, cudaStream_t s) {
  if (n > 0) stream_shift_kernel<<<dim3(n, 2), 256, 0, s>>>(base_audio, base_logmel, entries_audio, entries_logmel);
}

__global__ void stream_append_kernel(float* __restrict__ audio, const float* __restrict__ new_audio,
                                     const int* __restrict__ entries) {
  const int* en = entries + 3 * blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < en[2]) audio[en[0] + i] = new_audio[en[1] + i];
}

void launch_stream_append(float* audio, const float* new_audio, const int* entries, int n, int max_count,
                          cudaStream_t s) {
  if (n > 0 && max_count > 0)
    stream_append_kernel<<<dim3((max_count + 255) / 256, n), 256, 0, s>>>(audio, new_audio, entries);
}

// 32 frames per CTA
__global__ void __launch_bounds__(256) stream_max_kernel(const float* __restrict__ logmel,
                                                         const int* __restrict__ meta, MetaLayout ml, int n_mel,
                                                         int* __restrict__ seq_max) {
  const int seq = blockIdx.y;
  const int T = meta[ml.frames + seq];
  const int t0 = blockIdx.x * 32;
  if (t0 >= T) return;
  const float* src = logmel + ((long)meta[ml.frame_off + seq] + t0) * n_mel;
  const int count = min(32, T - t0) * n_mel;
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < count; i += 256) mx = fmaxf(mx, src[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0 && mx > -INFINITY) atomicMax(seq_max + seq, float_to_ordered(mx));
}

void launch_stream_max(const float* logmel, const int* meta, MetaLayout ml, int B, int max_frames, int n_mel,
                       int* seq_max, cudaStream_t s) {
  if (B > 0 && max_frames > 0)
    stream_max_kernel<<<dim3((max_frames + 31) / 32, B), 256, 0, s>>>(logmel, meta, ml, n_mel, seq_max);
}

// ---------------------------------------------------------------------------------------------
// Normalisation: max(lg, max_i - 8), (x + 4) / 4, written either packed (wf_logmel) or into
// the padded-row layout with the hush rows behind each buffer's rows (x (+) h at log-mel level).
// Padded-row layout of sequence i (R_i = 2 (n_i + 1) rows starting at the even row P_i):
//   row P_i            zero   (left conv padding)
//   rows P_i+1 ..      T_i audio rows, then H hush rows
//   remaining 1-2 rows zero   (right conv padding, rounds R_i up to even)
template <typename OutT>
__global__ void __launch_bounds__(256) normalise_kernel(
    const float* __restrict__ logmel, const int* __restrict__ seq_max,
    const float* __restrict__ mel_in, const int* __restrict__ meta, MetaLayout ml, int n_mel, int dst_ld,
    int hush_frames, const float* __restrict__ hush, OutT* __restrict__ dst, int mode) {
  const int seq = blockIdx.y;
  const int lr = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int T = meta[ml.frames + seq];
  const long frame0 = meta[ml.frame_off + seq];
  float floor_v = 0.f;
  if (logmel != nullptr) floor_v = ordered_to_float(seq_max[seq]) - 8.0f;
  if (mode == 0) {
    if (lr >= T) return;
    for (int m = lane; m < n_mel; m += 32) {
      float v = (fmaxf(logmel[(frame0 + lr) * n_mel + m], floor_v) + 4.0f) * 0.25f;
      dst[(frame0 + lr) * dst_ld + m] = (OutT)v;
    }
    return;
  }
  const int p0 = meta[ml.prow_off + seq];
  const int R = meta[ml.prow_off + seq + 1] - p0;
  if (lr >= R) return;
  const int t = lr - 1;
  for (int m = lane; m < n_mel; m += 32) {
    float v = 0.f;
    if (t >= 0 && t < T) {
      v = mel_in != nullptr ? mel_in[(frame0 + t) * n_mel + m]
                            : (fmaxf(logmel[(frame0 + t) * n_mel + m], floor_v) + 4.0f) * 0.25f;
    } else if (t >= T && t < T + hush_frames) {
      v = hush[(long)(t - T) * n_mel + m];
    }
    dst[(long)(p0 + lr) * dst_ld + m] = (OutT)v;
  }
}

void launch_normalise(const float* logmel, const int* seq_max, const float* mel_in, const int* meta,
                      MetaLayout ml, int B, int max_rows, int n_mel, int dst_ld, int hush_frames,
                      const float* hush, void* dst, int dst_bf16, int mode, cudaStream_t s) {
  if (B <= 0 || max_rows <= 0) return;
  dim3 grid((max_rows + 7) / 8, B);
  if (dst_bf16)
    normalise_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(logmel, seq_max, mel_in, meta, ml, n_mel, dst_ld,
                                                         hush_frames, hush, (__nv_bfloat16*)dst, mode);
  else
    normalise_kernel<float><<<grid, 256, 0, s>>>(logmel, seq_max, mel_in, meta, ml, n_mel, dst_ld,
                                                 hush_frames, hush, (float*)dst, mode);
}

// Row maps for the conv-stem epilogues: which padded rows hold data, and where each stride-2
// output row lands in the packed token matrix together with its position in its sequence.
__global__ void build_maps_kernel(const int* __restrict__ meta, MetaLayout ml, int hush_frames,
                                  int* __restrict__ row_valid, int2* __restrict__ row_dst) {
  const int seq = blockIdx.y;
  const int lr = blockIdx.x * blockDim.x + threadIdx.x;
  const int p0 = meta[ml.prow_off + seq];
  const int R = meta[ml.prow_off + seq + 1] - p0;
  if (lr >= R) return;
  const int rows = meta[ml.frames + seq] + hush_frames;
  row_valid[p0 + lr] = (lr >= 1 && lr <= rows) ? 1 : 0;
  if (lr < R / 2) {
    const int tok0 = meta[ml.tok_off + seq];
    const int n = meta[ml.tok_off + seq + 1] - tok0;
    row_dst[p0 / 2 + lr] = make_int2(lr < n ? tok0 + lr : -1, lr);
  }
}

void launch_build_maps(const int* meta, MetaLayout ml, int B, int max_rows, int hush_frames,
                       int* row_valid, int2* row_dst, cudaStream_t s) {
  if (B <= 0 || max_rows <= 0) return;
  dim3 grid((max_rows + 255) / 256, B);
  build_maps_kernel<<<grid, 256, 0, s>>>(meta, ml, hush_frames, row_valid, row_dst);
}

// Behind the transposed filterbank [201][n_mel]: per channel the half-open run of bins [first, last + 1)
// that holds all its non-zero weights (0, 0 for an all-zero channel).
__global__ void mel_bin_range_kernel(float* fbt, int n_mel) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= n_mel) return;
  int lo = 0, hi = 0;
  bool any = false;
  for (int k = 0; k < kBins; ++k)
    if (fbt[k * n_mel + m] != 0.f) {
      if (!any) lo = k;
      any = true;
      hi = k + 1;
    }
  reinterpret_cast<int2*>(fbt + kBins * n_mel)[m] = make_int2(lo, hi);
}
void launch_mel_bin_ranges(float* mel_fb_t, int n_mel, cudaStream_t s) {
  mel_bin_range_kernel<<<1, 128, 0, s>>>(mel_fb_t, n_mel);
}

}  // namespace wf

// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "../../include/wf_encoder.h"

namespace wf {

constexpr int kNFft = 400;
constexpr int kHop = 160;
constexpr int kBins = 201;
constexpr int kFold = 200;        // folded DFT length: 400-point real input, symmetric window
constexpr int kBasisCols = 224;   // 201 bins padded to 7 x 32 lanes
constexpr int kFeFrames = 64;     // frames per front-end CTA
constexpr int kHeadDim = 64;

// Epilogue selectors shared by the SIMT and the tcgen05 GEMM kernels.
enum Epilogue : int {
  kEpiBias = 0,       // out = acc + bias
  kEpiBiasGelu = 1,   // out = gelu(acc + bias)
  kEpiBiasResid = 2,  // resid(f32) += acc + bias
  kEpiConv1 = 3,      // out[row] = row_valid[row] ? gelu(acc + bias) : 0
  kEpiConv2 = 4,      // x[dst[row]] = gelu(acc + bias) + pe[pos[row]] (dst < 0: skip); x is f32 on the
                      // float32 path, the split bf16 residual stream (+ row statistics) on the bf16 path
  // bf16 path only.  The residual stream x is held as two bf16 planes, x = x_hi + x_lo with
  // x_hi = bf16(x) and x_lo = bf16(x - x_hi) (16 significant bits), so that x_hi is at once the
  // A operand of the GEMM that follows a LayerNorm.  That LayerNorm is folded into the GEMM:
  // with W' = W diag(gamma) (rounded to bf16), s[n] = sum_k W'[n,k], c[n] = bias[n] + sum_k W[n,k] beta[k],
  //   LN(x) W^T + bias = rstd (x W'^T - mean s) + c,
  // mean and rstd coming from per-row partial sums that the producer of x leaves behind.
  kEpiLnBias = 5,      // out = rstd (acc - mean s) + c
  kEpiLnBiasGelu = 6,  // out = gelu(rstd (acc - mean s) + c)
  kEpiResidSplit = 7   // (x_hi, x_lo) <- split(x_hi + x_lo + acc + bias); row statistics written
};

struct EpiParams {
  const float* bias;     // [N]
  void* out;             // element type of the path (kEpiBias, kEpiBiasGelu, kEpiConv1)
  float* resid;          // f32 (kEpiBiasResid, kEpiConv2)
  long ldc;              // leading dimension of out / resid (and of pe) in elements
  const int* row_valid;  // kEpiConv1: one int per GEMM row
  const int2* row_dst;   // kEpiConv2: (destination token row or -1, position in sequence)
  const float* pe;       // kEpiConv2: sinusoid table [n_ctx, N]
  // bf16 path, LayerNorm folded into the consumer / statistics left by the producer:
  const float* colsum;      // kEpiLn*: s[n]; `bias` then holds c[n]
  const float2* stats_in;   // kEpiLn*: [K / 128][stats_pitch] partial (sum, sum of squares) of 128 columns of x
  float2* stats_out;        // kEpiResidSplit, kEpiConv2 (bf16): the same layout over the N output columns
  long stats_pitch;         // rows per partial plane
  __nv_bfloat16* x_hi;      // kEpiConv2 (bf16): planes of the residual stream, row pitch ldc
  __nv_bfloat16* x_lo;
};

// Per-handle launch options of the bf16 path.
struct LaunchOpts {
  int pdl;          // launch with programmatic stream serialization (a kernel's set-up overlaps its predecessor's tail)
  int small_tiles;  // GEMMs too small to fill the CTA pairs run 128 x 128 tiles on single CTAs
  int tile;         // 0: the launcher chooses; 1 / 2 / 3: force 256 x 256 pair tiles / 128 x 128 / 128 x 256 single-CTA tiles
  int split_k;      // ... and, when even those leave half of the SMs idle and K has at least this many 64-wide
                    // blocks, split each tile's K range over a cluster of CTAs (0: never)
};

// Offsets (in ints) of the per-call metadata arrays inside one device int buffer.
struct MetaLayout {
  int sample_off;   // [B+1] first sample of each buffer in the packed audio
  int frames;       // [B]   audio frames T_i
  int frame_off;    // [B+1] prefix sums of T_i
  int prow_off;     // [B+1] first row of each sequence in the padded-row layout (even)
  int tok_off;      // [B+1] token prefix sums (cu_seqlens)
  int fe_tile_off;  // [B+1] prefix sums of front-end tiles
  int attn_work;    // [n_attn_work] pairs (sequence, first query row within the sequence)
  int total;
  // front end over resident stream windows (0 = absent: lengths come from sample_off differences
  // and tiles from fe_tile_off)
  int fe_len;       // [B] samples in each buffer
  int fe_tiles;     // [n_tiles] pairs (sequence, first frame of the tile)
};

// ---- kernel launch with optional cluster size and programmatic stream serialization.
// With the latter the kernel may begin (set up barriers, allocate tensor memory) while the kernel
// before it in the stream drains; it must call ptx::griddep_wait() before it touches global
// memory.
template <typename... P, typename... A>
inline cudaError_t launch_dependent(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    int cluster_x, bool pdl, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attrs[2];
  unsigned n = 0;
  if (cluster_x > 1) {
    attrs[n].id = cudaLaunchAttributeClusterDimension;
    attrs[n].val.clusterDim.x = (unsigned)cluster_x;
    attrs[n].val.clusterDim.y = 1;
    attrs[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl) {
    attrs[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attrs;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<A>(args)...);
}

// ---- tables (wf_frontend.cu)
void launch_build_tables(float* dft_basis /*[2][kFold][kBasisCols]*/, float* pe, int n_ctx, int d,
                         cudaStream_t s);

// ---- front end (wf_frontend.cu)
// mel_fb_t holds the transposed filterbank [201][n_mel] followed by n_mel int2 (launch_mel_bin_ranges):
// per channel, the run of bins [first, last + 1) that holds its non-zero weights.
void launch_mel_bin_ranges(float* mel_fb_t, int n_mel, cudaStream_t s);
cudaError_t frontend_configure();
void launch_frontend(const float* audio, const int* meta, MetaLayout ml, int B, int n_tiles,
                     const float* dft_basis, const float* mel_fb_t /*[201][n_mel]*/, int n_mel,
                     float* logmel /*[sum T, n_mel]*/, int* seq_max /*[B] ordered ints*/,
                     const float* tail /*tail_len samples that follow EVERY buffer, or NULL*/, int tail_len,
                     cudaStream_t s);
// mode 0: packed normalised mel (float) for wf_logmel; mode 1: padded-row layout + hush rows.
void launch_normalise(const float* logmel, const int* seq_max, const float* mel_in,
                      const int* meta, MetaLayout ml, int B, int max_rows, int n_mel, int dst_ld,
                      int hush_frames, const float* hush, void* dst, int dst_bf16, int mode, cudaStream_t s);
void launch_build_maps(const int* meta, MetaLayout ml, int B, int max_rows, int hush_frames,
                       int* row_valid, int2* row_dst, cudaStream_t s);
void launch_fill_seq_max(int* seq_max, int B, cudaStream_t s);

// ---- resident stream windows (wf_frontend.cu).  Lists live in one int buffer:
// shift entries (float offset of the array slice, floats to drop at its front, floats in it),
// append entries (destination float offset, source float offset, count).
void launch_stream_shift(float* base_audio, float* base_logmel, const int* entries_audio, const int* entries_logmel,
                         int n, cudaStream_t s);
void launch_stream_append(float* audio, const float* new_audio, const int* entries, int n, int max_count,
                          cudaStream_t s);
// seq_max[i] = max over the frames[i] x n_mel values at logmel + frame_off[i] * n_mel (ordered ints)
void launch_stream_max(const float* logmel, const int* meta, MetaLayout ml, int B, int max_frames, int n_mel,
                       int* seq_max, cudaStream_t s);

// ---- SIMT float32 kernels and element-wise kernels (wf_simt.cu)
void launch_gemm_f32(const float* A, long lda, const float* W, long ldw, long M, int N, int K,
                     int epi, const EpiParams& ep, cudaStream_t s);
void launch_layernorm(const float* x, const float* g, const float* b, float* out, long M, int d, cudaStream_t s);
void launch_attention_f32(const float* qkv, float* out, const int* meta, MetaLayout ml, int n_work,
                          int d_model, cudaStream_t s);
void launch_wait_selftest(int* err_flag, unsigned poll_limit, cudaStream_t s);
void launch_convert(const float* src, void* dst, long n, int dst_bf16, cudaStream_t s);
void launch_conv_weight(const float* src /*[out, in, 3]*/, void* dst /*[out, 3*in_ld], zeroed*/, int c_out,
                        int c_in, int in_ld, int dst_bf16, cudaStream_t s);
void launch_transpose_f32(const float* src, float* dst, int rows, int cols, cudaStream_t s);

// ---- tcgen05 bf16 GEMM (wf_gemm_tcgen05.cu)
struct TmaApi {
  void* encode_tiled;  // cuTensorMapEncodeTiled
};
bool tma_api_init(TmaApi* api);
// 2-D bf16 tensor map: inner extent `cols` (elements), outer extent `rows`, row pitch in
// elements, box = 64 x box_rows, 128 B swizzle.
bool make_tmap_bf16(const TmaApi& api, CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows,
                    uint64_t pitch_elems, uint32_t box_rows);
// Output tensor map for the epilogue's TMA stores: box of 32 rows x 128 bytes (64 bf16 or 32 f32).
bool make_tmap_out(const TmaApi& api, CUtensorMap* m, const void* base, int elem_bytes, uint64_t cols,
                   uint64_t rows);
cudaError_t gemm_bf16_configure();
// W tensor maps use 128-row boxes (both kernels stage 128 W rows per copy).
// a_cols: stored row length of A in elements (K for a plain GEMM; smaller when one GEMM row
// spans several consecutive stored rows, which must then be a multiple of 64).
// tc: bf16 output map (kEpiBias, kEpiBiasGelu, kEpiLn*, kEpiConv1); kEpiResidSplit: tc / tc2 are the
// maps of x_hi / x_lo (make_tmap_out, used for the fetch and for the store); unused by kEpiConv2.
// Rows of the output between M and the next multiple of 128 are written too when the map has
// them: outputs must be capacity-sized or exactly M rows.
void launch_gemm_bf16(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2,
                      long M, int N, int K, int a_cols, int epi, const EpiParams& ep, int* err_flag, int num_sms,
                      const LaunchOpts& opt, cudaStream_t s);
// Folds a LayerNorm's affine part into the weight that follows it (rows [0, N) of W [N, K] float32):
// wg = bf16(W diag(g)), colsum[n] = sum_k float(wg[n,k]), cbias[n] = bias[n] + sum_k W[n,k] b[k]
// (bias may be NULL = zeros).
void launch_ln_fold(const float* W, const float* g, const float* b, const float* bias, __nv_bfloat16* wg,
                    float* colsum, float* cbias, int N, int K, cudaStream_t s);
// Final LayerNorm of the bf16 path: reads the split residual stream.
void launch_layernorm_split(const __nv_bfloat16* x_hi, const __nv_bfloat16* x_lo, const float* g, const float* b,
                            __nv_bfloat16* out, long M, int d, bool pdl, cudaStream_t s);

// ---- bf16 attention on tcgen05 (wf_attention_tc.cu).  The work list at ml.attn_work holds
// n_entries triples (sequence, first query row | kind << 30, first item; kind 2 = one 128-row tile,
// one item per head, used for small batches): kind 0 = 256 consecutive
// query rows, one item per head; kind 1 = the odd last 128-row tile of a sequence, one item per
// pair of heads; behind the triples one int per item names its entry.  n_items is the total.
cudaError_t attention_bf16_configure();
// tmap_q / tmap_kv: bf16 [rows, 3 d_model] maps of the same buffer with 64 x 128 and 64 x 96 boxes
// (make_tmap_bf16 with box_rows 128 and 96)
void launch_attention_bf16(const CUtensorMap& tmap_q, const CUtensorMap& tmap_kv, __nv_bfloat16* out,
                           const int* meta, MetaLayout ml, int n_entries, int n_items, int d_model, int* err_flag,
                           int num_sms, bool pdl, cudaStream_t s);

// ---- dynamic time warping (wf_dtw.cu); meta holds 4 ints per problem:
// cost offset in cells, tokens, frames, offset into token_start
cudaError_t launch_dtw(const float* cost, const int* meta, int B, int max_tok, long max_cells,
                       unsigned char* trace,
                       int* token_start, float* total_cost, cudaStream_t s);

}  // namespace wf

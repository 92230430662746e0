// C ABI, host-side ragged planner and launch sequence of the encoder.
#include <algorithm>
#include <cstdarg>
#include <cstdlib>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "wf_internal.h"

using namespace wf;

namespace {
constexpr int kRing = 4;          // per-call metadata slots (pinned host + device)
constexpr int kMaxTailSamples = 16000;  // longest raw-audio hush word (1 s)
constexpr int kMinSamples = 401;  // reflect padding of 200 needs more than 200 samples on each side
}  // namespace

// float32 path: weights as given, LayerNorm parameters applied by the LayerNorm kernel.
// bf16 path: wqkv and w1 hold W diag(gamma) of the LayerNorm in front of them, bqkv / b1 the
// bias plus W beta, cs_qkv / cs_1 the row sums of the folded weights (see kEpiLnBias).
struct LayerW {
  float *ln1_g, *ln1_b, *ln2_g, *ln2_b;
  void *wqkv, *wo, *w1, *w2;
  float *bqkv, *bo, *b1, *b2;
  float *cs_qkv, *cs_1;
  CUtensorMap tm_wqkv, tm_wo, tm_w1, tm_w2;
};

struct ProfEvent {
  cudaEvent_t a, b;
  int cls;
};

struct wf_encoder {
  wf_config cfg;
  bool bf16;
  int num_sms;
  size_t esz;
  int mel_ld;      // channels per stored log-mel row (n_mel, rounded up to 64 on the bf16 path)
  long cap_prows;  // padded-row capacity
  long cap_frames; // log-mel rows the front-end scratch holds
  char err[512];
  std::vector<void*> allocs;
  std::vector<void*> pinned;
  TmaApi tma;

  float *dft_basis, *pe, *mel_fb_t;
  void *conv1_w, *conv2_w;
  float *conv1_b, *conv2_b, *lnp_g, *lnp_b;
  std::vector<LayerW> layers;
  CUtensorMap tm_conv1_w, tm_conv2_w, tm_zp, tm_c1p, tm_xh, tm_attn, tm_fc1;
  CUtensorMap tmo_c1p, tmo_qkv, tmo_fc1;         // epilogue outputs
  CUtensorMap tmx_hi, tmx_lo;                    // residual stream planes: fetched and stored by the residual epilogue
  CUtensorMap tm_qkv, tm_qkv_kv;                 // attention operand loads (128- and 96-row boxes)

  float* logmel;
  int* seq_max;
  void *zp_alloc, *c1p;
  int* row_valid;
  int2* row_dst;
  float* x;                 // float32 path: residual stream
  void* h;                  // float32 path: LayerNorm output
  __nv_bfloat16 *xh, *xl;   // bf16 path: residual stream x = xh + xl
  float2* stats;            // bf16 path: [d_model / 128][max_tokens] row partial (sum, sum of squares) of x
  void *qkv, *attn, *fc1;
  LaunchOpts opt;
  // host-buffer calls: two sets of staging buffers, so that the copies of one call overlap the
  // kernels of its neighbours (copies run on two streams of the library's own)
  float* audio_stage[2];
  void* out_stage[2];
  cudaStream_t copy_in, copy_out;
  cudaEvent_t host_ev_in[2], host_ev_comp[2], host_ev_out[2];
  bool host_used[2];
  long host_calls;
  int* err_flag;

  int meta_cap;
  int* meta_dev[kRing];
  int* meta_host[kRing];
  cudaEvent_t meta_ev[kRing];
  bool meta_used[kRing];
  int ring_pos;

  bool profile;
  std::vector<ProfEvent> prof;
  size_t prof_used;
};

// Resident windows of `n` streams: samples and un-normalised log-mel rows on the device, lengths
// on the host.
struct wf_streams {
  wf_encoder* enc;
  int n;
  long cap_samples;  // per stream, a multiple of the hop
  long cap_frames;   // cap_samples / hop
  float* audio;      // [n][cap_samples]
  float* logmel;     // [n][cap_frames][n_mel]  log10 mel power, before the max / clamp / scale
  int* scratch_max;  // [max_batch] sink for the front end's running maxima during a push
  std::vector<long> len;
};

namespace {

struct Plan {
  int B;
  long total_samples;
  int total_frames, total_prows, total_tokens;
  int n_fe_tiles, n_work, n_attn_items, max_prows_seq;
  MetaLayout ml;
};

wf_status fail(wf_encoder* e, wf_status st, const char* fmt, ...) {
  if (e) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(e->err, sizeof(e->err), fmt, ap);
    va_end(ap);
  }
  return st;
}

#define WF_CUDA(e, call)                                                                     \
  do {                                                                                       \
    cudaError_t _c = (call);                                                                 \
    if (_c != cudaSuccess)                                                                   \
      return fail((e), WF_ERR_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(_c),  \
                  __FILE__, __LINE__);                                                       \
  } while (0)

template <typename T>
wf_status dev_alloc(wf_encoder* e, T** p, size_t n_elems, bool zero = false) {
  void* q = nullptr;
  size_t bytes = std::max<size_t>(n_elems * sizeof(T), 256);
  WF_CUDA(e, cudaMalloc(&q, bytes));
  e->allocs.push_back(q);
  if (zero) WF_CUDA(e, cudaMemset(q, 0, bytes));
  *p = reinterpret_cast<T*>(q);
  return WF_OK;
}

wf_status dev_alloc_bytes(wf_encoder* e, void** p, size_t bytes, bool zero = false) {
  uint8_t* q = nullptr;
  wf_status st = dev_alloc<uint8_t>(e, &q, bytes, zero);
  *p = q;
  return st;
}

// Copies a float32 device vector into library-owned memory.
wf_status own_f32(wf_encoder* e, float** dst, const float* src, size_t n, cudaStream_t s) {
  if (!src) return fail(e, WF_ERR_INVALID_ARG, "a weight pointer is NULL");
  wf_status st = dev_alloc<float>(e, dst, n);
  if (st != WF_OK) return st;
  WF_CUDA(e, cudaMemcpyAsync(*dst, src, n * sizeof(float), cudaMemcpyDeviceToDevice, s));
  return WF_OK;
}

// Converts a float32 device matrix into the path's element type at dst (+ element offset).
wf_status own_mat(wf_encoder* e, void* dst, size_t elem_off, const float* src, size_t n, cudaStream_t s) {
  if (!src) return fail(e, WF_ERR_INVALID_ARG, "a weight pointer is NULL");
  launch_convert(src, (uint8_t*)dst + elem_off * e->esz, (long)n, e->bf16 ? 1 : 0, s);
  return WF_OK;
}

class Prof {
 public:
  Prof(wf_encoder* e, int cls, cudaStream_t s) : e_(e), s_(s), ev_(nullptr) {
    if (!e->profile) return;
    if (e->prof_used == e->prof.size()) {
      ProfEvent pe;
      if (cudaEventCreate(&pe.a) != cudaSuccess || cudaEventCreate(&pe.b) != cudaSuccess) return;
      pe.cls = cls;
      e->prof.push_back(pe);
    }
    ev_ = &e->prof[e->prof_used++];
    ev_->cls = cls;
    cudaEventRecord(ev_->a, s_);
  }
  ~Prof() {
    if (ev_) cudaEventRecord(ev_->b, s_);
  }

 private:
  wf_encoder* e_;
  cudaStream_t s_;
  ProfEvent* ev_;
};

// Attention work list for sequences in `order` (tok[i] .. tok[i+1] are sequence i's tokens), written
// at `dst`; returns the number of ints written.  float32 kernel: (sequence, first query row) pairs,
// one per 16 rows, *n_entries of them.  bf16 kernel: (sequence, first query row | kind << 30, first
// item) triples: per sequence the entries of 256 consecutive rows whose two 128-row tiles are both
// non-empty (kind 0, n_head items each), then one entry for its odd last tile if it has one
// (kind 1, two heads side by side: ceil(n_head / 2) items), then one int per item naming its entry.
// *n_items counts the bf16 items.
// With `num_sms` > 0 and few enough tokens that even one item per (128-row tile, head) gives no more
// items than SMs, the bf16 list is made of such single-tile items instead (kind 2).
int build_attn_work(const int* tok, const std::vector<int>& order, bool bf16, int n_head, int* dst, int* n_entries,
                    int* n_items, int num_sms = 0) {
  int nw = 0;
  *n_items = 0;
  if (!bf16) {
    for (int i : order)
      for (int q0 = 0; q0 < tok[i + 1] - tok[i]; q0 += 16) {
        dst[2 * nw] = i;
        dst[2 * nw + 1] = q0;
        ++nw;
      }
    *n_entries = nw;
    return 2 * nw;
  }
  int items = 0;
  long single = 0;
  for (int i : order) single += (long)((tok[i + 1] - tok[i] + 127) / 128) * n_head;
  if (num_sms > 0 && single <= num_sms) {
    for (int i : order)
      for (int q0 = 0; q0 < tok[i + 1] - tok[i]; q0 += 128) {
        dst[3 * nw] = i;
        dst[3 * nw + 1] = (int)((unsigned)q0 | (2u << 30));
        dst[3 * nw + 2] = items;
        items += n_head;
        ++nw;
      }
  } else
  for (int i : order) {
    const int n = tok[i + 1] - tok[i];
    for (int q0 = 0; q0 + 128 < n; q0 += 256) {
      dst[3 * nw] = i;
      dst[3 * nw + 1] = q0;
      dst[3 * nw + 2] = items;
      items += n_head;
      ++nw;
    }
    const int tiles = (n + 127) / 128;
    if (tiles & 1) {
      dst[3 * nw] = i;
      dst[3 * nw + 1] = ((tiles - 1) * 128) | (1 << 30);
      dst[3 * nw + 2] = items;
      items += (n_head + 1) / 2;
      ++nw;
    }
  }
  *n_entries = nw;
  *n_items = items;
  // one int per item: the entry it belongs to (saves the kernel a search)
  int* item_entry = dst + 3 * nw;
  for (int w = 0; w < nw; ++w) {
    const int end = w + 1 < nw ? dst[3 * (w + 1) + 2] : items;
    for (int it = dst[3 * w + 2]; it < end; ++it) item_entry[it] = w;
  }
  return 3 * nw + items;
}

// Builds prefix sums, the padded-row layout and the work lists for one call into `hm`
// (host ints), validating every length.  `frames_given`: `len` holds frame counts, not samples.
// `front_end_only`: the plan of wf_logmel (no hush rows, no token limits, no attention work list).
wf_status make_plan(wf_encoder* e, const long* len, bool frames_given, int B, Plan* p, int* hm,
                    bool front_end_only = false, long tail_samples = 0) {
  const wf_config& c = e->cfg;
  const bool build_work = !front_end_only;
  const long hush_rows = front_end_only ? 0 : c.hush_frames;
  const long n_ctx = front_end_only ? (1L << 28) : c.n_ctx;
  const long max_tokens = front_end_only ? (1L << 40) : c.max_tokens;
  if (B < 0 || (B > 0 && !len)) return fail(e, WF_ERR_INVALID_ARG, "bad batch size or NULL lengths");
  if (B > c.max_batch) return fail(e, WF_ERR_CAPACITY, "batch %d exceeds max_batch %d", B, c.max_batch);
  MetaLayout& ml = p->ml;
  int off = 0;
  ml.sample_off = off; off += B + 1;
  ml.frames = off; off += B + 1;
  ml.frame_off = off; off += B + 1;
  ml.prow_off = off; off += B + 1;
  ml.tok_off = off; off += B + 1;
  ml.fe_tile_off = off; off += B + 1;
  ml.attn_work = off;
  ml.fe_len = 0;
  ml.fe_tiles = 0;
  long samples = 0, frames = 0, prows = 0, tokens = 0, tiles = 0;
  int max_pr = 0;
  for (int i = 0; i < B; ++i) {
    long L = len[i], T;
    if (frames_given) {
      if (L < 1) return fail(e, WF_ERR_TOO_SHORT, "sequence %d has %ld frames", i, L);
      T = L;
      L = 0;
    } else {
      if (L < kMinSamples) return fail(e, WF_ERR_TOO_SHORT, "buffer %d has %ld samples (need >= %d)", i, L, kMinSamples);
      T = (L + tail_samples) / kHop;  // a raw-audio hush word lengthens every buffer
    }
    long rows = T + hush_rows;
    long n = (rows + 1) / 2;
    if (n > n_ctx) return fail(e, WF_ERR_TOO_LONG, "sequence %d would have %ld tokens (n_ctx %d)", i, n, c.n_ctx);
    hm[ml.sample_off + i] = (int)samples;
    hm[ml.frames + i] = (int)T;
    hm[ml.frame_off + i] = (int)frames;
    hm[ml.prow_off + i] = (int)prows;
    hm[ml.tok_off + i] = (int)tokens;
    hm[ml.fe_tile_off + i] = (int)tiles;
    samples += L;
    frames += T;
    prows += 2 * (n + 1);
    tokens += n;
    tiles += (T + kFeFrames - 1) / kFeFrames;
    max_pr = std::max<int>(max_pr, (int)(2 * (n + 1)));
    if (samples > c.max_samples) return fail(e, WF_ERR_CAPACITY, "more than max_samples=%ld samples", c.max_samples);
    if (tokens > max_tokens) return fail(e, WF_ERR_CAPACITY, "more than max_tokens=%ld tokens", c.max_tokens);
  }
  hm[ml.sample_off + B] = (int)samples;
  hm[ml.frames + B] = 0;
  hm[ml.frame_off + B] = (int)frames;
  hm[ml.prow_off + B] = (int)prows;
  hm[ml.tok_off + B] = (int)tokens;
  hm[ml.fe_tile_off + B] = (int)tiles;
  // attention work list, longest sequences first
  std::vector<int> order(B);
  for (int i = 0; i < B; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    return hm[ml.tok_off + a + 1] - hm[ml.tok_off + a] > hm[ml.tok_off + b + 1] - hm[ml.tok_off + b];
  });
  int nw = 0, n_items = 0, work_ints = 0;
  if (build_work) work_ints = build_attn_work(hm + ml.tok_off, order, e->bf16, c.n_head, hm + ml.attn_work, &nw, &n_items, e->num_sms);
  ml.total = ml.attn_work + work_ints;
  p->B = B;
  p->total_samples = samples;
  p->total_frames = (int)frames;
  p->total_prows = (int)prows;
  p->total_tokens = (int)tokens;
  p->n_fe_tiles = (int)tiles;
  p->n_work = nw;
  p->n_attn_items = n_items;
  p->max_prows_seq = max_pr;
  return WF_OK;
}

wf_status ring_acquire(wf_encoder* e, int* slot) {
  int s = e->ring_pos;
  e->ring_pos = (e->ring_pos + 1) % kRing;
  if (e->meta_used[s]) WF_CUDA(e, cudaEventSynchronize(e->meta_ev[s]));
  *slot = s;
  return WF_OK;
}

wf_status ring_upload(wf_encoder* e, int slot, const Plan& p, cudaStream_t s) {
  WF_CUDA(e, cudaMemcpyAsync(e->meta_dev[slot], e->meta_host[slot], (size_t)std::max(p.ml.total, 1) * sizeof(int),
                             cudaMemcpyHostToDevice, s));
  return WF_OK;
}

wf_status ring_release(wf_encoder* e, int slot, cudaStream_t s) {
  WF_CUDA(e, cudaEventRecord(e->meta_ev[slot], s));
  e->meta_used[slot] = true;
  return WF_OK;
}

// Everything after the log-mel rows sit in the padded-row layout, float32 path: SIMT GEMMs, a
// LayerNorm kernel in front of the QKV and FC1 GEMMs, float32 residual stream.
wf_status run_encoder_f32(wf_encoder* e, const Plan& p, const int* meta, void* hidden_out, cudaStream_t s) {
  const wf_config& c = e->cfg;
  const int d = c.d_model, F = c.d_mlp;
  const long M = p.total_tokens;
  const float* zp = (const float*)e->zp_alloc;
  {
    Prof pr(e, 1, s);
    launch_build_maps(meta, p.ml, p.B, p.max_prows_seq, c.hush_frames, e->row_valid, e->row_dst, s);
  }
  {
    Prof pr(e, 2, s);
    EpiParams ep{};
    ep.bias = e->conv1_b; ep.out = e->c1p; ep.ldc = d; ep.row_valid = e->row_valid;
    launch_gemm_f32(zp, e->mel_ld, (const float*)e->conv1_w, 3L * e->mel_ld, p.total_prows, d, 3 * e->mel_ld, kEpiConv1, ep, s);
  }
  {
    Prof pr(e, 2, s);
    EpiParams ep{};
    ep.bias = e->conv2_b; ep.resid = e->x; ep.ldc = d; ep.row_dst = e->row_dst; ep.pe = e->pe;
    launch_gemm_f32((const float*)e->c1p, 2L * d, (const float*)e->conv2_w, 3L * d, p.total_prows / 2, d, 3 * d, kEpiConv2, ep, s);
  }
  for (int l = 0; l < c.n_layer; ++l) {
    LayerW& w = e->layers[l];
    {
      Prof pr(e, 3, s);
      launch_layernorm(e->x, w.ln1_g, w.ln1_b, (float*)e->h, M, d, s);
    }
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.bqkv; ep.out = e->qkv; ep.ldc = 3L * d;
      launch_gemm_f32((const float*)e->h, d, (const float*)w.wqkv, d, M, 3 * d, d, kEpiBias, ep, s);
    }
    {
      Prof pr(e, 5, s);
      launch_attention_f32((const float*)e->qkv, (float*)e->attn, meta, p.ml, p.n_work, d, s);
    }
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.bo; ep.resid = e->x; ep.ldc = d;
      launch_gemm_f32((const float*)e->attn, d, (const float*)w.wo, d, M, d, d, kEpiBiasResid, ep, s);
    }
    {
      Prof pr(e, 3, s);
      launch_layernorm(e->x, w.ln2_g, w.ln2_b, (float*)e->h, M, d, s);
    }
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.b1; ep.out = e->fc1; ep.ldc = F;
      launch_gemm_f32((const float*)e->h, d, (const float*)w.w1, d, M, F, d, kEpiBiasGelu, ep, s);
    }
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.b2; ep.resid = e->x; ep.ldc = d;
      launch_gemm_f32((const float*)e->fc1, F, (const float*)w.w2, F, M, d, F, kEpiBiasResid, ep, s);
    }
  }
  {
    Prof pr(e, 3, s);
    launch_layernorm(e->x, e->lnp_g, e->lnp_b, (float*)hidden_out, M, d, s);
  }
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

// The same on the bf16 path: tcgen05 GEMMs; the residual stream is the pair of bf16 planes
// (xh, xl); its producers (conv2, out-projection, FC2) leave per-row partial sums in `stats`, from
// which the QKV and FC1 GEMMs, whose weights carry the LayerNorm's gain, finish the LayerNorm in
// their epilogues.  Only the final LayerNorm is a kernel of its own.
wf_status run_encoder_bf16(wf_encoder* e, const Plan& p, const int* meta, void* hidden_out, cudaStream_t s) {
  const wf_config& c = e->cfg;
  const int d = c.d_model, F = c.d_mlp;
  const long M = p.total_tokens;
  auto gemm = [&](const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2, long m,
                  int n, int k, int a_cols, int epi, const EpiParams& ep) {
    launch_gemm_bf16(ta, tb, tc, tc2, m, n, k, a_cols, epi, ep, e->err_flag, e->num_sms, e->opt, s);
  };
  {
    Prof pr(e, 1, s);
    launch_build_maps(meta, p.ml, p.B, p.max_prows_seq, c.hush_frames, e->row_valid, e->row_dst, s);
  }
  {
    Prof pr(e, 2, s);
    EpiParams ep{};
    ep.bias = e->conv1_b; ep.out = e->c1p; ep.ldc = d; ep.row_valid = e->row_valid;
    gemm(e->tm_zp, e->tm_conv1_w, e->tmo_c1p, e->tmo_c1p, p.total_prows, d, 3 * e->mel_ld, e->mel_ld, kEpiConv1, ep);
  }
  {
    Prof pr(e, 2, s);
    EpiParams ep{};
    ep.bias = e->conv2_b; ep.ldc = d; ep.row_dst = e->row_dst; ep.pe = e->pe;
    ep.x_hi = e->xh; ep.x_lo = e->xl; ep.stats_out = e->stats; ep.stats_pitch = c.max_tokens;
    gemm(e->tm_c1p, e->tm_conv2_w, e->tmx_hi, e->tmx_lo, p.total_prows / 2, d, 3 * d, 2 * d, kEpiConv2, ep);
  }
  for (int l = 0; l < c.n_layer; ++l) {
    LayerW& w = e->layers[l];
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.bqkv; ep.colsum = w.cs_qkv; ep.stats_in = e->stats; ep.stats_pitch = c.max_tokens;
      ep.out = e->qkv; ep.ldc = 3L * d;
      gemm(e->tm_xh, w.tm_wqkv, e->tmo_qkv, e->tmo_qkv, M, 3 * d, d, d, kEpiLnBias, ep);
    }
    {
      Prof pr(e, 5, s);
      launch_attention_bf16(e->tm_qkv, e->tm_qkv_kv, (__nv_bfloat16*)e->attn, meta, p.ml, p.n_work, p.n_attn_items, d,
                            e->err_flag, e->num_sms, e->opt.pdl != 0, s);
    }
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.bo; ep.ldc = d; ep.stats_out = e->stats; ep.stats_pitch = c.max_tokens;
      gemm(e->tm_attn, w.tm_wo, e->tmx_hi, e->tmx_lo, M, d, d, d, kEpiResidSplit, ep);
    }
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.b1; ep.colsum = w.cs_1; ep.stats_in = e->stats; ep.stats_pitch = c.max_tokens;
      ep.out = e->fc1; ep.ldc = F;
      gemm(e->tm_xh, w.tm_w1, e->tmo_fc1, e->tmo_fc1, M, F, d, d, kEpiLnBiasGelu, ep);
    }
    {
      Prof pr(e, 4, s);
      EpiParams ep{};
      ep.bias = w.b2; ep.ldc = d; ep.stats_out = e->stats; ep.stats_pitch = c.max_tokens;
      gemm(e->tm_fc1, w.tm_w2, e->tmx_hi, e->tmx_lo, M, d, F, F, kEpiResidSplit, ep);
    }
  }
  {
    Prof pr(e, 3, s);
    launch_layernorm_split(e->xh, e->xl, e->lnp_g, e->lnp_b, (__nv_bfloat16*)hidden_out, M, d, e->opt.pdl != 0, s);
  }
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

wf_status run_encoder(wf_encoder* e, const Plan& p, const int* meta, void* hidden_out, cudaStream_t s) {
  return e->bf16 ? run_encoder_bf16(e, p, meta, hidden_out, s) : run_encoder_f32(e, p, meta, hidden_out, s);
}

wf_status encode_impl(wf_encoder* e, const float* audio, const float* mel, const long* len, int B,
                      const float* hush, void* hidden_out, int* cu_out, cudaStream_t s,
                      const float* tail = nullptr, int tail_len = 0) {
  if (!e) return WF_ERR_INVALID_ARG;
  const wf_config& c = e->cfg;
  if (c.hush_frames > 0 && !hush) return fail(e, WF_ERR_INVALID_ARG, "hush_mel is NULL but hush_frames > 0");
  if (B > 0 && (!hidden_out || (!audio && !mel))) return fail(e, WF_ERR_INVALID_ARG, "NULL input or output");
  if (B > c.max_batch) return fail(e, WF_ERR_CAPACITY, "batch %d exceeds max_batch %d", B, c.max_batch);
  if (B < 0) return fail(e, WF_ERR_INVALID_ARG, "negative batch");
  int slot;
  wf_status st = ring_acquire(e, &slot);
  if (st != WF_OK) return st;
  Plan p;
  st = make_plan(e, len, mel != nullptr, B, &p, e->meta_host[slot], false, tail_len);
  if (st == WF_OK && (long)p.total_frames > e->cap_frames)
    st = fail(e, WF_ERR_CAPACITY, "more than %ld frames", e->cap_frames);
  if (st != WF_OK) return st;
  if (cu_out)
    for (int i = 0; i <= B; ++i) cu_out[i] = e->meta_host[slot][p.ml.tok_off + i];
  if (B == 0) return WF_OK;
  st = ring_upload(e, slot, p, s);
  if (st != WF_OK) return st;
  const int* meta = e->meta_dev[slot];
  void* zp = (uint8_t*)e->zp_alloc + (size_t)e->mel_ld * e->esz;  // row 0 sits behind one guard row
  if (audio) {
    {
      Prof pr(e, 0, s);
      launch_fill_seq_max(e->seq_max, B, s);
      launch_frontend(audio, meta, p.ml, B, p.n_fe_tiles, e->dft_basis, e->mel_fb_t, c.n_mel, e->logmel,
                      e->seq_max, tail, tail_len, s);
    }
    {
      Prof pr(e, 1, s);
      launch_normalise(e->logmel, e->seq_max, nullptr, meta, p.ml, B, p.max_prows_seq, c.n_mel, e->mel_ld,
                       c.hush_frames, hush, zp, e->bf16 ? 1 : 0, 1, s);
    }
  } else {
    Prof pr(e, 1, s);
    launch_normalise(nullptr, nullptr, mel, meta, p.ml, B, p.max_prows_seq, c.n_mel, e->mel_ld, c.hush_frames,
                     hush, zp, e->bf16 ? 1 : 0, 1, s);
  }
  st = run_encoder(e, p, meta, hidden_out, s);
  if (st != WF_OK) return st;
  return ring_release(e, slot, s);
}

}  // namespace

// ---------------------------------------------------------------------------------------------
extern "C" {

wf_status wf_encoder_create(const wf_config* cfg, const wf_weights* w, void* stream, wf_encoder** out) {
  if (!cfg || !w || !out) return WF_ERR_INVALID_ARG;
  *out = nullptr;
  cudaStream_t s = (cudaStream_t)stream;
  wf_encoder* e = new (std::nothrow) wf_encoder();
  if (!e) return WF_ERR_INVALID_ARG;
  e->cfg = *cfg;
  e->err[0] = 0;
  e->profile = false;
  e->prof_used = 0;
  e->ring_pos = 0;
  for (int i = 0; i < kRing; ++i) { e->meta_used[i] = false; e->meta_dev[i] = nullptr; e->meta_host[i] = nullptr; e->meta_ev[i] = nullptr; }
  e->copy_in = e->copy_out = nullptr;
  e->host_calls = 0;
  for (int i = 0; i < 2; ++i) { e->host_used[i] = false; e->host_ev_in[i] = e->host_ev_comp[i] = e->host_ev_out[i] = nullptr; }
  *out = e;  // returned even on failure so that the caller can read the message, then destroy
  const wf_config& c = e->cfg;
  if (c.n_mel <= 0 || c.n_mel % 8 || c.n_mel > 128 || c.d_model <= 0 || c.d_model % 128 || c.d_model > 1280 ||
      c.n_head * kHeadDim != c.d_model || c.d_mlp <= 0 || c.d_mlp % 128 || c.n_layer < 0 || c.n_ctx < 1 ||
      c.hush_frames < 0 || c.max_batch < 1 || c.max_tokens < 1 || c.max_samples < 0 ||
      c.max_samples >= (1L << 31) - 1 || c.max_tokens > (1L << 28) || (c.dtype != WF_F32 && c.dtype != WF_BF16))
    return fail(e, WF_ERR_INVALID_ARG, "unsupported configuration (see wf_config in wf_encoder.h)");
  int dev = 0;
  WF_CUDA(e, cudaGetDevice(&dev));
  cudaDeviceProp prop;
  WF_CUDA(e, cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return fail(e, WF_ERR_UNSUPPORTED_ARCH, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
  e->num_sms = prop.multiProcessorCount;
  e->bf16 = c.dtype == WF_BF16;
  e->esz = e->bf16 ? 2 : 4;
  e->mel_ld = e->bf16 ? (c.n_mel + 63) / 64 * 64 : c.n_mel;
  e->cap_prows = 2 * (c.max_tokens + c.max_batch);
  const int d = c.d_model, F = c.d_mlp;
  wf_status st;
#define WF_TRY(x) do { st = (x); if (st != WF_OK) return st; } while (0)

  if (e->bf16) {
    if (!tma_api_init(&e->tma)) return fail(e, WF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    WF_CUDA(e, gemm_bf16_configure());
    WF_CUDA(e, attention_bf16_configure());
  }
  WF_CUDA(e, frontend_configure());
  {
    // tuning switches, read once per handle
    const char* pdl_env = getenv("WF_PDL");
    e->opt.pdl = !(pdl_env != nullptr && pdl_env[0] == '0');
    const char* small_env = getenv("WF_GEMM_SMALL_TILES");
    e->opt.small_tiles = !(small_env != nullptr && small_env[0] == '0');
    const char* tile_env = getenv("WF_GEMM_TILE");
    e->opt.tile = tile_env != nullptr ? atoi(tile_env) : 0;
    const char* split_env = getenv("WF_GEMM_SPLIT_K");
    e->opt.split_k = split_env != nullptr ? atoi(split_env) : 64;
  }
  // tables
  WF_TRY(dev_alloc<float>(e, &e->dft_basis, 2L * kFold * kBasisCols));
  WF_TRY(dev_alloc<float>(e, &e->pe, (size_t)c.n_ctx * d));
  launch_build_tables(e->dft_basis, e->pe, c.n_ctx, d, s);
  if (!w->mel_fb) return fail(e, WF_ERR_INVALID_ARG, "mel_fb is NULL");
  WF_TRY(dev_alloc<float>(e, &e->mel_fb_t, (size_t)kBins * c.n_mel + 2 * c.n_mel));
  launch_transpose_f32(w->mel_fb, e->mel_fb_t, c.n_mel, kBins, s);
  launch_mel_bin_ranges(e->mel_fb_t, c.n_mel, s);
  // conv stem
  WF_TRY(dev_alloc_bytes(e, &e->conv1_w, (size_t)d * 3 * e->mel_ld * e->esz, true));
  WF_TRY(dev_alloc_bytes(e, &e->conv2_w, (size_t)d * 3 * d * e->esz, true));
  if (!w->conv1_w || !w->conv2_w) return fail(e, WF_ERR_INVALID_ARG, "conv weights are NULL");
  launch_conv_weight(w->conv1_w, e->conv1_w, d, c.n_mel, e->mel_ld, e->bf16, s);
  launch_conv_weight(w->conv2_w, e->conv2_w, d, d, d, e->bf16, s);
  WF_TRY(own_f32(e, &e->conv1_b, w->conv1_b, d, s));
  WF_TRY(own_f32(e, &e->conv2_b, w->conv2_b, d, s));
  WF_TRY(own_f32(e, &e->lnp_g, w->lnp_g, d, s));
  WF_TRY(own_f32(e, &e->lnp_b, w->lnp_b, d, s));
  // blocks
  e->layers.resize(c.n_layer);
  if (c.n_layer > 0 && (!w->ln1_g || !w->ln1_b || !w->wq || !w->bq || !w->wk || !w->wv || !w->bv || !w->wo ||
                        !w->bo || !w->ln2_g || !w->ln2_b || !w->w1 || !w->b1 || !w->w2 || !w->b2))
    return fail(e, WF_ERR_INVALID_ARG, "a per-layer weight array is NULL");
  for (int l = 0; l < c.n_layer; ++l) {
    LayerW& L = e->layers[l];
    if (!w->ln1_g[l] || !w->ln1_b[l] || !w->ln2_g[l] || !w->ln2_b[l] || !w->wq[l] || !w->wk[l] || !w->wv[l] ||
        !w->bq[l] || !w->bv[l] || !w->w1[l] || !w->b1[l])
      return fail(e, WF_ERR_INVALID_ARG, "a weight pointer of layer %d is NULL", l);
    WF_TRY(dev_alloc_bytes(e, &L.wqkv, (size_t)3 * d * d * e->esz));
    WF_TRY(dev_alloc<float>(e, &L.bqkv, 3 * d, true));  // float32 path: the key part stays zero
    WF_TRY(dev_alloc_bytes(e, &L.w1, (size_t)F * d * e->esz));
    if (e->bf16) {
      // LayerNorm 1 folded into the QKV weight, LayerNorm 2 into FC1's
      WF_TRY(dev_alloc<float>(e, &L.cs_qkv, 3 * d));
      WF_TRY(dev_alloc<float>(e, &L.cs_1, F));
      WF_TRY(dev_alloc<float>(e, &L.b1, F));
      __nv_bfloat16* wqkv = (__nv_bfloat16*)L.wqkv;
      launch_ln_fold(w->wq[l], w->ln1_g[l], w->ln1_b[l], w->bq[l], wqkv, L.cs_qkv, L.bqkv, d, d, s);
      launch_ln_fold(w->wk[l], w->ln1_g[l], w->ln1_b[l], nullptr, wqkv + (size_t)d * d, L.cs_qkv + d, L.bqkv + d, d, d, s);
      launch_ln_fold(w->wv[l], w->ln1_g[l], w->ln1_b[l], w->bv[l], wqkv + (size_t)2 * d * d, L.cs_qkv + 2 * d, L.bqkv + 2 * d, d, d, s);
      launch_ln_fold(w->w1[l], w->ln2_g[l], w->ln2_b[l], w->b1[l], (__nv_bfloat16*)L.w1, L.cs_1, L.b1, F, d, s);
    } else {
      WF_TRY(own_f32(e, &L.ln1_g, w->ln1_g[l], d, s));
      WF_TRY(own_f32(e, &L.ln1_b, w->ln1_b[l], d, s));
      WF_TRY(own_f32(e, &L.ln2_g, w->ln2_g[l], d, s));
      WF_TRY(own_f32(e, &L.ln2_b, w->ln2_b[l], d, s));
      WF_TRY(own_mat(e, L.wqkv, 0, w->wq[l], (size_t)d * d, s));
      WF_TRY(own_mat(e, L.wqkv, (size_t)d * d, w->wk[l], (size_t)d * d, s));
      WF_TRY(own_mat(e, L.wqkv, (size_t)2 * d * d, w->wv[l], (size_t)d * d, s));
      WF_CUDA(e, cudaMemcpyAsync(L.bqkv, w->bq[l], d * sizeof(float), cudaMemcpyDeviceToDevice, s));
      WF_CUDA(e, cudaMemcpyAsync(L.bqkv + 2 * d, w->bv[l], d * sizeof(float), cudaMemcpyDeviceToDevice, s));
      WF_TRY(own_mat(e, L.w1, 0, w->w1[l], (size_t)F * d, s));
      WF_TRY(own_f32(e, &L.b1, w->b1[l], F, s));
    }
    WF_TRY(dev_alloc_bytes(e, &L.wo, (size_t)d * d * e->esz));
    WF_TRY(own_mat(e, L.wo, 0, w->wo[l], (size_t)d * d, s));
    WF_TRY(own_f32(e, &L.bo, w->bo[l], d, s));
    WF_TRY(dev_alloc_bytes(e, &L.w2, (size_t)d * F * e->esz));
    WF_TRY(own_mat(e, L.w2, 0, w->w2[l], (size_t)d * F, s));
    WF_TRY(own_f32(e, &L.b2, w->b2[l], d, s));
  }
  // workspace
  const size_t mt = (size_t)c.max_tokens;
  e->cap_frames = c.max_samples / kHop + (long)c.max_batch * (kMaxTailSamples / kHop) + 1;
  WF_TRY(dev_alloc<float>(e, &e->logmel, (size_t)e->cap_frames * c.n_mel));
  WF_TRY(dev_alloc<int>(e, &e->seq_max, c.max_batch));
  WF_TRY(dev_alloc_bytes(e, &e->zp_alloc, (size_t)(e->cap_prows + 4) * e->mel_ld * e->esz, true));
  WF_TRY(dev_alloc_bytes(e, &e->c1p, (size_t)(e->cap_prows + 4) * d * e->esz, true));
  WF_TRY(dev_alloc<int>(e, &e->row_valid, (size_t)e->cap_prows + 4, true));
  WF_TRY(dev_alloc<int2>(e, &e->row_dst, (size_t)e->cap_prows / 2 + 4, true));
  if (e->bf16) {
    WF_TRY(dev_alloc<__nv_bfloat16>(e, &e->xh, mt * d, true));
    WF_TRY(dev_alloc<__nv_bfloat16>(e, &e->xl, mt * d, true));
    WF_TRY(dev_alloc<float2>(e, &e->stats, (size_t)(d / 128) * mt, true));
  } else {
    WF_TRY(dev_alloc<float>(e, &e->x, mt * d));
    WF_TRY(dev_alloc_bytes(e, &e->h, mt * d * e->esz, true));
  }
  WF_TRY(dev_alloc_bytes(e, &e->qkv, mt * 3 * d * e->esz, true));
  WF_TRY(dev_alloc_bytes(e, &e->attn, mt * d * e->esz, true));
  WF_TRY(dev_alloc_bytes(e, &e->fc1, mt * F * e->esz, true));
  for (int i = 0; i < 2; ++i) {
    WF_TRY(dev_alloc<float>(e, &e->audio_stage[i], (size_t)c.max_samples));
    WF_TRY(dev_alloc_bytes(e, &e->out_stage[i], mt * d * e->esz));
    WF_CUDA(e, cudaEventCreateWithFlags(&e->host_ev_in[i], cudaEventDisableTiming));
    WF_CUDA(e, cudaEventCreateWithFlags(&e->host_ev_comp[i], cudaEventDisableTiming));
    WF_CUDA(e, cudaEventCreateWithFlags(&e->host_ev_out[i], cudaEventDisableTiming));
  }
  WF_CUDA(e, cudaStreamCreateWithFlags(&e->copy_in, cudaStreamNonBlocking));
  WF_CUDA(e, cudaStreamCreateWithFlags(&e->copy_out, cudaStreamNonBlocking));
  WF_TRY(dev_alloc<int>(e, &e->err_flag, 1, true));
  e->meta_cap = 6 * (c.max_batch + 1) + 2 * (int)(c.max_tokens / 16 + c.max_batch) + 6 * c.max_batch + 16 +
                (e->bf16 ? (int)(c.max_tokens / 128 + 2 * c.max_batch) * c.n_head : 0);
  for (int i = 0; i < kRing; ++i) {
    WF_TRY(dev_alloc<int>(e, &e->meta_dev[i], e->meta_cap));
    void* hp = nullptr;
    WF_CUDA(e, cudaMallocHost(&hp, (size_t)e->meta_cap * sizeof(int)));
    e->pinned.push_back(hp);
    e->meta_host[i] = (int*)hp;
    WF_CUDA(e, cudaEventCreateWithFlags(&e->meta_ev[i], cudaEventDisableTiming));
  }
  if (e->bf16) {
    bool ok = true;
    ok &= make_tmap_bf16(e->tma, &e->tm_zp, e->zp_alloc, e->mel_ld, e->cap_prows + 4, e->mel_ld, 128);
    ok &= make_tmap_bf16(e->tma, &e->tm_c1p, e->c1p, 2 * d, (e->cap_prows + 4) / 2, 2 * d, 128);
    ok &= make_tmap_bf16(e->tma, &e->tm_xh, e->xh, d, mt, d, 128);
    ok &= make_tmap_bf16(e->tma, &e->tm_attn, e->attn, d, mt, d, 128);
    ok &= make_tmap_bf16(e->tma, &e->tm_fc1, e->fc1, F, mt, F, 128);
    ok &= make_tmap_bf16(e->tma, &e->tm_qkv, e->qkv, 3 * d, mt, 3 * d, 128);
    ok &= make_tmap_bf16(e->tma, &e->tm_qkv_kv, e->qkv, 3 * d, mt, 3 * d, 96);
    ok &= make_tmap_out(e->tma, &e->tmo_c1p, e->c1p, 2, d, e->cap_prows + 4);
    ok &= make_tmap_out(e->tma, &e->tmo_qkv, e->qkv, 2, 3 * d, mt);
    ok &= make_tmap_out(e->tma, &e->tmo_fc1, e->fc1, 2, F, mt);
    ok &= make_tmap_out(e->tma, &e->tmx_hi, e->xh, 2, d, mt);
    ok &= make_tmap_out(e->tma, &e->tmx_lo, e->xl, 2, d, mt);
    const uint32_t wbox = 128;
    ok &= make_tmap_bf16(e->tma, &e->tm_conv1_w, e->conv1_w, 3 * e->mel_ld, d, 3 * e->mel_ld, wbox);
    ok &= make_tmap_bf16(e->tma, &e->tm_conv2_w, e->conv2_w, 3 * d, d, 3 * d, wbox);
    for (int l = 0; l < c.n_layer; ++l) {
      LayerW& L = e->layers[l];
      ok &= make_tmap_bf16(e->tma, &L.tm_wqkv, L.wqkv, d, 3 * d, d, wbox);
      ok &= make_tmap_bf16(e->tma, &L.tm_wo, L.wo, d, d, d, wbox);
      ok &= make_tmap_bf16(e->tma, &L.tm_w1, L.w1, d, F, d, wbox);
      ok &= make_tmap_bf16(e->tma, &L.tm_w2, L.w2, F, d, F, wbox);
    }
    if (!ok) return fail(e, WF_ERR_CUDA, "cuTensorMapEncodeTiled rejected a tensor map");
  }
  WF_CUDA(e, cudaGetLastError());
  WF_CUDA(e, cudaStreamSynchronize(s));
#undef WF_TRY
  return WF_OK;
}

wf_status wf_encoder_destroy(wf_encoder* e) {
  if (!e) return WF_OK;
  cudaDeviceSynchronize();
  for (void* p : e->allocs) cudaFree(p);
  for (void* p : e->pinned) cudaFreeHost(p);
  for (int i = 0; i < kRing; ++i)
    if (e->meta_ev[i]) cudaEventDestroy(e->meta_ev[i]);
  for (auto& pe : e->prof) { cudaEventDestroy(pe.a); cudaEventDestroy(pe.b); }
  for (int i = 0; i < 2; ++i) {
    if (e->host_ev_in[i]) cudaEventDestroy(e->host_ev_in[i]);
    if (e->host_ev_comp[i]) cudaEventDestroy(e->host_ev_comp[i]);
    if (e->host_ev_out[i]) cudaEventDestroy(e->host_ev_out[i]);
  }
  if (e->copy_in) cudaStreamDestroy(e->copy_in);
  if (e->copy_out) cudaStreamDestroy(e->copy_out);
  delete e;
  return WF_OK;
}

const char* wf_last_error(const wf_encoder* e) { return e ? e->err : "null encoder"; }

wf_status wf_logmel(wf_encoder* e, const float* audio, const long* lengths, int B, float* mel_out,
                    long* frames_out, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (B > 0 && (!audio || !mel_out)) return fail(e, WF_ERR_INVALID_ARG, "NULL audio or output");
  if (B > e->cfg.max_batch) return fail(e, WF_ERR_CAPACITY, "batch %d exceeds max_batch %d", B, e->cfg.max_batch);
  if (B < 0) return fail(e, WF_ERR_INVALID_ARG, "negative batch");
  int slot;
  wf_status st = ring_acquire(e, &slot);
  if (st != WF_OK) return st;
  Plan p;
  // frame counts do not depend on the hush length; token limits do not apply to the front end
  st = make_plan(e, lengths, false, B, &p, e->meta_host[slot], true);
  if (st != WF_OK) return st;
  if (frames_out)
    for (int i = 0; i < B; ++i) frames_out[i] = e->meta_host[slot][p.ml.frames + i];
  if (B == 0) return WF_OK;
  p.ml.total = p.ml.attn_work;  // no attention work list needed
  st = ring_upload(e, slot, p, s);
  if (st != WF_OK) return st;
  const int* meta = e->meta_dev[slot];
  int max_T = 0;
  for (int i = 0; i < B; ++i) max_T = std::max(max_T, e->meta_host[slot][p.ml.frames + i]);
  {
    Prof pr(e, 0, s);
    launch_fill_seq_max(e->seq_max, B, s);
    launch_frontend(audio, meta, p.ml, B, p.n_fe_tiles, e->dft_basis, e->mel_fb_t, e->cfg.n_mel, e->logmel,
                    e->seq_max, nullptr, 0, s);
  }
  {
    Prof pr(e, 1, s);
    launch_normalise(e->logmel, e->seq_max, nullptr, meta, p.ml, B, max_T, e->cfg.n_mel, e->cfg.n_mel, 0, nullptr,
                     mel_out, 0, 0, s);
  }
  WF_CUDA(e, cudaGetLastError());
  return ring_release(e, slot, s);
}

wf_status wf_encode(wf_encoder* e, const float* audio, const long* lengths, int B, const float* hush_mel,
                    void* hidden_out, int* cu_seqlens_out, void* stream) {
  return encode_impl(e, audio, nullptr, lengths, B, hush_mel, hidden_out, cu_seqlens_out, (cudaStream_t)stream);
}

wf_status wf_encode_raw_hush(wf_encoder* e, const float* audio, const long* lengths, int B,
                             const float* hush_audio, int hush_samples, void* hidden_out, int* cu_seqlens_out,
                             void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  if (e->cfg.hush_frames != 0)
    return fail(e, WF_ERR_INVALID_ARG, "wf_encode_raw_hush needs an encoder created with hush_frames == 0");
  if (hush_samples < 0 || hush_samples > kMaxTailSamples || (hush_samples > 0 && !hush_audio))
    return fail(e, WF_ERR_INVALID_ARG, "hush_samples must be in [0, %d] with a non-NULL hush_audio", kMaxTailSamples);
  return encode_impl(e, audio, nullptr, lengths, B, nullptr, hidden_out, cu_seqlens_out, (cudaStream_t)stream,
                     hush_audio, hush_samples);
}

wf_status wf_encode_mel(wf_encoder* e, const float* mel, const long* frames, int B, const float* hush_mel,
                        void* hidden_out, int* cu_seqlens_out, void* stream) {
  return encode_impl(e, nullptr, mel, frames, B, hush_mel, hidden_out, cu_seqlens_out, (cudaStream_t)stream);
}

wf_status wf_encode_host_async(wf_encoder* e, const float* audio_host, const long* lengths, int B,
                               const float* hush_mel, void* hidden_out_host, int* cu_seqlens_out, void* stream,
                               long* ticket_out) {
  if (!e) return WF_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (B < 0 || !ticket_out || (B > 0 && (!audio_host || !lengths || !hidden_out_host)))
    return fail(e, WF_ERR_INVALID_ARG, "NULL input or output");
  long total = 0;
  for (int i = 0; i < B; ++i) {
    if (lengths[i] < 0) return fail(e, WF_ERR_INVALID_ARG, "negative length");
    total += lengths[i];
    if (total > e->cfg.max_samples) return fail(e, WF_ERR_CAPACITY, "more than max_samples=%ld samples", e->cfg.max_samples);
  }
  const int slot = (int)(e->host_calls & 1);
  // the call that used this slot two calls ago has delivered its result (and so finished its kernels)
  if (e->host_used[slot]) WF_CUDA(e, cudaEventSynchronize(e->host_ev_out[slot]));
  if (total > 0)
    WF_CUDA(e, cudaMemcpyAsync(e->audio_stage[slot], audio_host, (size_t)total * sizeof(float), cudaMemcpyHostToDevice, e->copy_in));
  WF_CUDA(e, cudaEventRecord(e->host_ev_in[slot], e->copy_in));
  WF_CUDA(e, cudaStreamWaitEvent(s, e->host_ev_in[slot], 0));
  std::vector<int> cu(B + 1, 0);
  wf_status st = encode_impl(e, e->audio_stage[slot], nullptr, lengths, B, hush_mel, e->out_stage[slot], cu.data(), s);
  if (st != WF_OK) return st;
  if (cu_seqlens_out) std::memcpy(cu_seqlens_out, cu.data(), (size_t)(B + 1) * sizeof(int));
  WF_CUDA(e, cudaEventRecord(e->host_ev_comp[slot], s));
  WF_CUDA(e, cudaStreamWaitEvent(e->copy_out, e->host_ev_comp[slot], 0));
  const size_t bytes = (size_t)cu[B] * e->cfg.d_model * e->esz;
  if (bytes) WF_CUDA(e, cudaMemcpyAsync(hidden_out_host, e->out_stage[slot], bytes, cudaMemcpyDeviceToHost, e->copy_out));
  WF_CUDA(e, cudaEventRecord(e->host_ev_out[slot], e->copy_out));
  e->host_used[slot] = true;
  *ticket_out = e->host_calls++;
  return WF_OK;
}

wf_status wf_encode_host_wait(wf_encoder* e, long ticket) {
  if (!e) return WF_ERR_INVALID_ARG;
  if (ticket < 0 || ticket >= e->host_calls) return fail(e, WF_ERR_INVALID_ARG, "unknown ticket %ld", ticket);
  if (ticket < e->host_calls - 2) return WF_OK;  // its slot has been reused, which waited for it
  WF_CUDA(e, cudaEventSynchronize(e->host_ev_out[ticket & 1]));
  return WF_OK;
}

wf_status wf_encode_host(wf_encoder* e, const float* audio_host, const long* lengths, int B,
                         const float* hush_mel, void* hidden_out_host, int* cu_seqlens_out, void* stream) {
  long ticket = 0;
  wf_status st = wf_encode_host_async(e, audio_host, lengths, B, hush_mel, hidden_out_host, cu_seqlens_out, stream, &ticket);
  if (st != WF_OK) return st;
  return wf_encode_host_wait(e, ticket);
}

wf_status wf_plan(const wf_config* cfg, const long* lengths, int B, int lengths_are_frames, long tail_samples,
                  int num_sms, int* cu_seqlens_out, long* totals_out, int* work_out, int work_cap) {
  if (!cfg || B < 0 || tail_samples < 0) return WF_ERR_INVALID_ARG;
  wf_encoder tmp{};  // the planner reads the configuration only; no CUDA call is made
  tmp.cfg = *cfg;
  tmp.bf16 = cfg->dtype == WF_BF16;
  tmp.num_sms = num_sms;
  tmp.err[0] = 0;
  if (B > cfg->max_batch) return WF_ERR_CAPACITY;
  const size_t cap = 6 * ((size_t)B + 1) + 2 * ((size_t)cfg->max_tokens / 16 + B) + 16 +
                     ((size_t)cfg->max_tokens / 128 + 2 * (size_t)B + 2) * (size_t)std::max(cfg->n_head, 1) * 2;
  std::vector<int> hm(cap);
  Plan p;
  wf_status st = make_plan(&tmp, lengths, lengths_are_frames != 0, B, &p, hm.data(), false, tail_samples);
  if (st != WF_OK) return st;
  if (cu_seqlens_out)
    for (int i = 0; i <= B; ++i) cu_seqlens_out[i] = hm[p.ml.tok_off + i];
  if (totals_out) {
    totals_out[0] = p.total_frames;
    totals_out[1] = p.total_prows;
    totals_out[2] = p.total_tokens;
    totals_out[3] = p.n_fe_tiles;
    totals_out[4] = p.n_work;
    totals_out[5] = p.n_attn_items;
  }
  if (work_out) {
    const int n = p.ml.total - p.ml.attn_work;
    if (n > work_cap) return WF_ERR_CAPACITY;
    for (int i = 0; i < n; ++i) work_out[i] = hm[p.ml.attn_work + i];
  }
  return WF_OK;
}

wf_status wf_check(wf_encoder* e, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  WF_CUDA(e, cudaStreamSynchronize(s));
  int flag = 0;
  WF_CUDA(e, cudaMemcpy(&flag, e->err_flag, sizeof(int), cudaMemcpyDeviceToHost));
  if (flag != 0) {
    cudaMemset(e->err_flag, 0, sizeof(int));
    return fail(e, WF_ERR_DEVICE_TIMEOUT, "a bounded wait inside a kernel gave up (role code %d: 1-6 GEMM, 11-13 attention, 21 self-test)", flag);
  }
  return WF_OK;
}

wf_status wf_selftest_wait_timeout(wf_encoder* e, unsigned poll_limit, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  if (poll_limit < 1 || poll_limit > (1u << 20)) return fail(e, WF_ERR_INVALID_ARG, "poll_limit must be in [1, 2^20]");
  launch_wait_selftest(e->err_flag, poll_limit, (cudaStream_t)stream);
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

wf_status wf_profile_enable(wf_encoder* e, int on) {
  if (!e) return WF_ERR_INVALID_ARG;
  e->profile = on != 0;
  return WF_OK;
}

wf_status wf_profile_read(wf_encoder* e, long* launches, double* millis) {
  if (!e || !launches || !millis) return WF_ERR_INVALID_ARG;
  WF_CUDA(e, cudaDeviceSynchronize());
  for (int c = 0; c < WF_N_KERNEL_CLASSES; ++c) { launches[c] = 0; millis[c] = 0.0; }
  for (size_t i = 0; i < e->prof_used; ++i) {
    float ms = 0.f;
    WF_CUDA(e, cudaEventElapsedTime(&ms, e->prof[i].a, e->prof[i].b));
    launches[e->prof[i].cls] += 1;
    millis[e->prof[i].cls] += ms;
  }
  e->prof_used = 0;
  return WF_OK;
}

wf_status wf_gemm_bf16(wf_encoder* e, const void* A, const void* W, const float* bias, void* C, long M, int N,
                       int K, int mode, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  if (!e->bf16) return fail(e, WF_ERR_INVALID_ARG, "wf_gemm_bf16 needs an encoder created with WF_BF16");
  if (!A || !W || !bias || !C || M < 0 || N <= 0 || K <= 0 || N % 8 || K % 8 || mode < 0 || mode > 1 ||
      ((uintptr_t)A & 15) || ((uintptr_t)W & 15) || ((uintptr_t)C & 15) || ((uintptr_t)bias & 15))
    return fail(e, WF_ERR_INVALID_ARG, "wf_gemm_bf16: bad pointer, size or mode");
  if (M == 0) return WF_OK;
  CUtensorMap ta, tb, tc;
  if (!make_tmap_bf16(e->tma, &ta, A, K, M, K, 128) || !make_tmap_bf16(e->tma, &tb, W, K, N, K, 128) ||
      !make_tmap_out(e->tma, &tc, C, 2, N, M))
    return fail(e, WF_ERR_CUDA, "cuTensorMapEncodeTiled rejected a tensor map");
  EpiParams ep{};
  ep.bias = bias;
  ep.ldc = N;
  ep.out = C;
  launch_gemm_bf16(ta, tb, tc, tc, M, N, K, K, mode == 0 ? kEpiBias : kEpiBiasGelu, ep, e->err_flag, e->num_sms, e->opt,
                   (cudaStream_t)stream);
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

wf_status wf_gemm_resid_bf16(wf_encoder* e, const void* A, const void* W, const float* bias, void* x_hi, void* x_lo,
                             float* stats, long M, int N, int K, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  if (!e->bf16) return fail(e, WF_ERR_INVALID_ARG, "wf_gemm_resid_bf16 needs an encoder created with WF_BF16");
  if (!A || !W || !bias || !x_hi || !x_lo || !stats || M < 0 || N <= 0 || K <= 0 || N % 128 || K % 8 ||
      ((uintptr_t)A & 15) || ((uintptr_t)W & 15) || ((uintptr_t)x_hi & 15) || ((uintptr_t)x_lo & 15) ||
      ((uintptr_t)bias & 15) || ((uintptr_t)stats & 7))
    return fail(e, WF_ERR_INVALID_ARG, "wf_gemm_resid_bf16: bad pointer or size (N must be a multiple of 128)");
  if (M == 0) return WF_OK;
  CUtensorMap ta, tb, th, tl;
  if (!make_tmap_bf16(e->tma, &ta, A, K, M, K, 128) || !make_tmap_bf16(e->tma, &tb, W, K, N, K, 128) ||
      !make_tmap_out(e->tma, &th, x_hi, 2, N, M) || !make_tmap_out(e->tma, &tl, x_lo, 2, N, M))
    return fail(e, WF_ERR_CUDA, "cuTensorMapEncodeTiled rejected a tensor map");
  EpiParams ep{};
  ep.bias = bias;
  ep.ldc = N;
  ep.stats_out = (float2*)stats;
  ep.stats_pitch = M;
  launch_gemm_bf16(ta, tb, th, tl, M, N, K, K, kEpiResidSplit, ep, e->err_flag, e->num_sms, e->opt, (cudaStream_t)stream);
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

wf_status wf_ln_fold(wf_encoder* e, const float* W, const float* ln_g, const float* ln_b, const float* bias, void* Wg,
                     float* colsum, float* cbias, int N, int K, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  if (!W || !ln_g || !ln_b || !Wg || !colsum || !cbias || N <= 0 || K <= 0)
    return fail(e, WF_ERR_INVALID_ARG, "wf_ln_fold: bad pointer or size");
  launch_ln_fold(W, ln_g, ln_b, bias, (__nv_bfloat16*)Wg, colsum, cbias, N, K, (cudaStream_t)stream);
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

wf_status wf_gemm_ln_bf16(wf_encoder* e, const void* x_hi, const float* stats, const void* Wg, const float* colsum,
                          const float* cbias, void* C, long M, int N, int K, int gelu, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  if (!e->bf16) return fail(e, WF_ERR_INVALID_ARG, "wf_gemm_ln_bf16 needs an encoder created with WF_BF16");
  if (!x_hi || !stats || !Wg || !colsum || !cbias || !C || M < 0 || N <= 0 || K <= 0 || N % 8 || K % 128 ||
      ((uintptr_t)x_hi & 15) || ((uintptr_t)Wg & 15) || ((uintptr_t)C & 15) || ((uintptr_t)colsum & 15) ||
      ((uintptr_t)cbias & 15) || ((uintptr_t)stats & 7))
    return fail(e, WF_ERR_INVALID_ARG, "wf_gemm_ln_bf16: bad pointer or size (K must be a multiple of 128)");
  if (M == 0) return WF_OK;
  CUtensorMap ta, tb, tc;
  if (!make_tmap_bf16(e->tma, &ta, x_hi, K, M, K, 128) || !make_tmap_bf16(e->tma, &tb, Wg, K, N, K, 128) ||
      !make_tmap_out(e->tma, &tc, C, 2, N, M))
    return fail(e, WF_ERR_CUDA, "cuTensorMapEncodeTiled rejected a tensor map");
  EpiParams ep{};
  ep.bias = cbias;
  ep.colsum = colsum;
  ep.stats_in = (const float2*)stats;
  ep.stats_pitch = M;
  ep.ldc = N;
  ep.out = C;
  launch_gemm_bf16(ta, tb, tc, tc, M, N, K, K, gelu ? kEpiLnBiasGelu : kEpiLnBias, ep, e->err_flag, e->num_sms, e->opt,
                   (cudaStream_t)stream);
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

wf_status wf_streams_create(wf_encoder* e, int n_streams, long max_window_samples, wf_streams** out) {
  if (!e || !out) return WF_ERR_INVALID_ARG;
  *out = nullptr;
  const long cap = (max_window_samples + kHop - 1) / kHop * kHop;
  if (n_streams < 1 || max_window_samples < kMinSamples || (double)n_streams * (double)cap * e->cfg.n_mel / kHop >= 2147483647.0 ||
      (double)n_streams * (double)cap >= 2147483647.0)
    return fail(e, WF_ERR_INVALID_ARG, "wf_streams_create: bad stream count or window size");
  wf_streams* st = new (std::nothrow) wf_streams();
  if (!st) return fail(e, WF_ERR_CUDA, "out of host memory");
  st->enc = e;
  st->n = n_streams;
  st->cap_samples = cap;
  st->cap_frames = cap / kHop;
  st->audio = nullptr;
  st->logmel = nullptr;
  st->scratch_max = nullptr;
  st->len.assign(n_streams, 0);
  if (cudaMalloc(&st->audio, (size_t)n_streams * cap * sizeof(float)) != cudaSuccess ||
      cudaMalloc(&st->logmel, (size_t)n_streams * st->cap_frames * e->cfg.n_mel * sizeof(float)) != cudaSuccess ||
      cudaMalloc(&st->scratch_max, (size_t)e->cfg.max_batch * sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(st->audio);
    cudaFree(st->logmel);
    cudaFree(st->scratch_max);
    delete st;
    return fail(e, WF_ERR_CUDA, "wf_streams_create: out of device memory");
  }
  *out = st;
  return WF_OK;
}

wf_status wf_streams_destroy(wf_streams* st) {
  if (!st) return WF_OK;
  cudaDeviceSynchronize();
  cudaFree(st->audio);
  cudaFree(st->logmel);
  cudaFree(st->scratch_max);
  delete st;
  return WF_OK;
}

wf_status wf_streams_length(const wf_streams* st, int stream_id, long* samples) {
  if (!st || !samples || stream_id < 0 || stream_id >= st->n) return WF_ERR_INVALID_ARG;
  *samples = st->len[stream_id];
  return WF_OK;
}

wf_status wf_streams_push(wf_streams* st, const int* ids, int B, const float* new_audio, const long* n_new,
                          const long* trim, void* stream) {
  if (!st) return WF_ERR_INVALID_ARG;
  wf_encoder* e = st->enc;
  cudaStream_t s = (cudaStream_t)stream;
  if (B < 0 || (B > 0 && (!ids || !n_new))) return fail(e, WF_ERR_INVALID_ARG, "wf_streams_push: NULL argument");
  if (B > e->cfg.max_batch) return fail(e, WF_ERR_CAPACITY, "batch %d exceeds max_batch %d", B, e->cfg.max_batch);
  if (B == 0) return WF_OK;
  // validate everything before any state changes
  std::vector<char> seen(st->n, 0);
  long total_new = 0, max_new = 0;
  int n_shift = 0, n_tiles = 0;
  for (int i = 0; i < B; ++i) {
    const int id = ids[i];
    if (id < 0 || id >= st->n || seen[id]) return fail(e, WF_ERR_INVALID_ARG, "wf_streams_push: stream id %d out of range or repeated", id);
    seen[id] = 1;
    const long cut = trim ? trim[i] : 0, add = n_new[i], len = st->len[id];
    if (cut < 0 || cut % kHop != 0 || cut > len || add < 0)
      return fail(e, WF_ERR_INVALID_ARG, "wf_streams_push: stream %d: trim %ld (window %ld) or new sample count %ld", id, cut, len, add);
    if (add > 0 && !new_audio) return fail(e, WF_ERR_INVALID_ARG, "wf_streams_push: new_audio is NULL");
    const long nl = len - cut + add;
    if (nl > st->cap_samples) return fail(e, WF_ERR_CAPACITY, "stream %d would hold %ld samples (capacity %ld)", id, nl, st->cap_samples);
    if (nl < kMinSamples) return fail(e, WF_ERR_TOO_SHORT, "stream %d would hold %ld samples (need >= %d)", id, nl, kMinSamples);
    total_new += add;
    max_new = std::max(max_new, add);
    if (cut > 0 && cut < len) ++n_shift;
    // frames to compute: the two at the old end (their reflected tail is now real audio) and all
    // new ones; after a cut also the first two (their reflected head changed)
    const long T_new = nl / kHop, kept = (len - cut) / kHop;
    const long from = std::max(0L, kept - 2);
    if (cut > 0 && from > 0) ++n_tiles;
    n_tiles += (int)((T_new - from + kFeFrames - 1) / kFeFrames);
  }
  const int need = 4 * (B + 1) + 2 * n_tiles + 6 * n_shift + 3 * B + 8;
  if (need > e->meta_cap) return fail(e, WF_ERR_CAPACITY, "wf_streams_push: metadata capacity exceeded");
  int slot;
  wf_status rc = ring_acquire(e, &slot);
  if (rc != WF_OK) return rc;
  int* hm = e->meta_host[slot];
  MetaLayout ml{};
  ml.sample_off = 0;
  ml.frames = B + 1;
  ml.frame_off = 2 * (B + 1);
  ml.fe_len = 3 * (B + 1);
  ml.fe_tiles = 4 * (B + 1);
  const int off_shift_a = ml.fe_tiles + 2 * n_tiles, off_shift_m = off_shift_a + 3 * n_shift;
  const int off_append = off_shift_m + 3 * n_shift;
  ml.total = off_append + 3 * B;
  int it = 0, is = 0;
  long src = 0;
  const int n_mel = e->cfg.n_mel;
  for (int i = 0; i < B; ++i) {
    const int id = ids[i];
    const long cut = trim ? trim[i] : 0, add = n_new[i], len = st->len[id];
    const long nl = len - cut + add, T_new = nl / kHop, kept = (len - cut) / kHop;
    hm[ml.sample_off + i] = (int)(id * st->cap_samples);
    hm[ml.frames + i] = (int)T_new;
    hm[ml.frame_off + i] = (int)(id * st->cap_frames);
    hm[ml.fe_len + i] = (int)nl;
    if (cut > 0 && cut < len) {
      hm[off_shift_a + 3 * is] = (int)(id * st->cap_samples);
      hm[off_shift_a + 3 * is + 1] = (int)cut;
      hm[off_shift_a + 3 * is + 2] = (int)len;
      hm[off_shift_m + 3 * is] = (int)(id * st->cap_frames * n_mel);
      hm[off_shift_m + 3 * is + 1] = (int)(cut / kHop * n_mel);
      hm[off_shift_m + 3 * is + 2] = (int)(len / kHop * n_mel);
      ++is;
    }
    hm[off_append + 3 * i] = (int)(id * st->cap_samples + len - cut);
    hm[off_append + 3 * i + 1] = (int)src;
    hm[off_append + 3 * i + 2] = (int)add;
    src += add;
    const long from = std::max(0L, kept - 2);
    if (cut > 0 && from > 0) {
      hm[ml.fe_tiles + 2 * it] = i;
      hm[ml.fe_tiles + 2 * it + 1] = 0;  // recomputes frames 0..63: the first two are the ones that changed
      ++it;
    }
    for (long t0 = from; t0 < T_new; t0 += kFeFrames) {
      hm[ml.fe_tiles + 2 * it] = i;
      hm[ml.fe_tiles + 2 * it + 1] = (int)t0;
      ++it;
    }
  }
  hm[ml.sample_off + B] = hm[ml.frames + B] = hm[ml.frame_off + B] = 0;
  Plan p{};
  p.ml = ml;
  rc = ring_upload(e, slot, p, s);
  if (rc != WF_OK) return rc;
  const int* meta = e->meta_dev[slot];
  {
    Prof pr(e, 0, s);
    launch_stream_shift(st->audio, st->logmel, meta + off_shift_a, meta + off_shift_m, n_shift, s);
    launch_stream_append(st->audio, new_audio, meta + off_append, B, (int)max_new, s);
    launch_frontend(st->audio, meta, ml, B, it, e->dft_basis, e->mel_fb_t, n_mel, st->logmel, st->scratch_max, nullptr, 0, s);
  }
  WF_CUDA(e, cudaGetLastError());
  for (int i = 0; i < B; ++i) st->len[ids[i]] += n_new[i] - (trim ? trim[i] : 0);
  return ring_release(e, slot, s);
}

wf_status wf_encode_streams(wf_streams* st, const int* ids, int B, const float* hush, void* hidden_out,
                            int* cu_out, void* stream) {
  if (!st) return WF_ERR_INVALID_ARG;
  wf_encoder* e = st->enc;
  const wf_config& c = e->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  if (c.hush_frames > 0 && !hush) return fail(e, WF_ERR_INVALID_ARG, "hush_mel is NULL but hush_frames > 0");
  if (B < 0 || (B > 0 && (!ids || !hidden_out))) return fail(e, WF_ERR_INVALID_ARG, "NULL input or output");
  if (B > c.max_batch) return fail(e, WF_ERR_CAPACITY, "batch %d exceeds max_batch %d", B, c.max_batch);
  std::vector<long> frames(std::max(B, 1));
  for (int i = 0; i < B; ++i) {
    if (ids[i] < 0 || ids[i] >= st->n) return fail(e, WF_ERR_INVALID_ARG, "stream id %d out of range", ids[i]);
    if (st->len[ids[i]] < kMinSamples) return fail(e, WF_ERR_TOO_SHORT, "stream %d holds %ld samples", ids[i], st->len[ids[i]]);
    frames[i] = st->len[ids[i]] / kHop;
  }
  int slot;
  wf_status rc = ring_acquire(e, &slot);
  if (rc != WF_OK) return rc;
  Plan p;
  rc = make_plan(e, frames.data(), true, B, &p, e->meta_host[slot]);
  if (rc != WF_OK) return rc;
  int* hm = e->meta_host[slot];
  if (cu_out)
    for (int i = 0; i <= B; ++i) cu_out[i] = hm[p.ml.tok_off + i];
  if (B == 0) return WF_OK;
  int max_T = 0;
  for (int i = 0; i < B; ++i) {
    hm[p.ml.frame_off + i] = (int)(ids[i] * st->cap_frames);  // rows are read from the resident windows
    max_T = std::max(max_T, (int)frames[i]);
  }
  rc = ring_upload(e, slot, p, s);
  if (rc != WF_OK) return rc;
  const int* meta = e->meta_dev[slot];
  void* zp = (uint8_t*)e->zp_alloc + (size_t)e->mel_ld * e->esz;
  {
    Prof pr(e, 1, s);
    launch_fill_seq_max(e->seq_max, B, s);
    launch_stream_max(st->logmel, meta, p.ml, B, max_T, c.n_mel, e->seq_max, s);
    launch_normalise(st->logmel, e->seq_max, nullptr, meta, p.ml, B, p.max_prows_seq, c.n_mel, e->mel_ld,
                     c.hush_frames, hush, zp, e->bf16 ? 1 : 0, 1, s);
  }
  rc = run_encoder(e, p, meta, hidden_out, s);
  if (rc != WF_OK) return rc;
  return ring_release(e, slot, s);
}

wf_status wf_cross_kv(wf_encoder* e, const void* hidden, const void* W_kv, const float* b_kv, long M,
                      int n_dec_layers, void* kv, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  const int d = e->cfg.d_model;
  if (M < 0 || n_dec_layers < 1 || (long)n_dec_layers * 2 * d > (1L << 30) || !W_kv || !b_kv ||
      (M > 0 && (!hidden || !kv)))
    return fail(e, WF_ERR_INVALID_ARG, "wf_cross_kv: bad pointer or size");
  if (M == 0) return WF_OK;
  const int N = n_dec_layers * 2 * d;
  EpiParams ep{};
  ep.bias = b_kv;
  ep.ldc = N;
  ep.out = kv;
  if (e->bf16) {
    if (((uintptr_t)hidden & 15) || ((uintptr_t)W_kv & 15) || ((uintptr_t)kv & 15) || ((uintptr_t)b_kv & 15))
      return fail(e, WF_ERR_INVALID_ARG, "wf_cross_kv: pointers must be 16-byte aligned");
    CUtensorMap ta, tb, tc;
    if (!make_tmap_bf16(e->tma, &ta, hidden, d, M, d, 128) ||
        !make_tmap_bf16(e->tma, &tb, W_kv, d, N, d, 128) ||
        !make_tmap_out(e->tma, &tc, kv, 2, N, M))
      return fail(e, WF_ERR_CUDA, "cuTensorMapEncodeTiled rejected a tensor map");
    launch_gemm_bf16(ta, tb, tc, tc, M, N, d, d, kEpiBias, ep, e->err_flag, e->num_sms, e->opt, (cudaStream_t)stream);
  } else {
    launch_gemm_f32((const float*)hidden, d, (const float*)W_kv, d, M, N, d, kEpiBias, ep, (cudaStream_t)stream);
  }
  WF_CUDA(e, cudaGetLastError());
  return WF_OK;
}

wf_status wf_dtw(wf_encoder* e, const float* cost, const int* n_tokens, const int* n_frames, int B,
                 unsigned char* trace_ws, int* token_start, float* total_cost, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (B < 0 || (B > 0 && (!cost || !n_tokens || !n_frames || !trace_ws || !token_start || !total_cost)))
    return fail(e, WF_ERR_INVALID_ARG, "wf_dtw: NULL argument");
  if (B == 0) return WF_OK;
  if (4 * B > e->meta_cap) return fail(e, WF_ERR_CAPACITY, "wf_dtw: batch %d exceeds the metadata capacity", B);
  int slot;
  wf_status st = ring_acquire(e, &slot);
  if (st != WF_OK) return st;
  int* hm = e->meta_host[slot];
  long cells = 0, toks = 0;
  int max_tok = 0;
  long max_cells = 0;
  for (int b = 0; b < B; ++b) {
    if (n_tokens[b] < 1 || n_frames[b] < 1 || n_tokens[b] > 16384)
      return fail(e, WF_ERR_INVALID_ARG, "wf_dtw: problem %d has %d tokens x %d frames", b, n_tokens[b], n_frames[b]);
    if (cells + (long)n_tokens[b] * n_frames[b] >= (1L << 31))
      return fail(e, WF_ERR_CAPACITY, "wf_dtw: more than 2^31 cells in one call");
    hm[4 * b] = (int)cells;
    hm[4 * b + 1] = n_tokens[b];
    hm[4 * b + 2] = n_frames[b];
    hm[4 * b + 3] = (int)toks;
    cells += (long)n_tokens[b] * n_frames[b];
    toks += n_tokens[b];
    max_tok = std::max(max_tok, n_tokens[b]);
    max_cells = std::max(max_cells, (long)n_tokens[b] * n_frames[b]);
  }
  Plan p{};
  p.ml.total = 4 * B;
  st = ring_upload(e, slot, p, s);
  if (st != WF_OK) return st;
  WF_CUDA(e, launch_dtw(cost, e->meta_dev[slot], B, max_tok, max_cells, trace_ws, token_start, total_cost, s));
  return ring_release(e, slot, s);
}

wf_status wf_attention(wf_encoder* e, const void* qkv, const int* cu_seqlens, int B, void* out, void* stream) {
  if (!e) return WF_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (B < 0 || (B > 0 && (!qkv || !cu_seqlens || !out))) return fail(e, WF_ERR_INVALID_ARG, "NULL argument");
  if (B > e->cfg.max_batch) return fail(e, WF_ERR_CAPACITY, "batch %d exceeds max_batch %d", B, e->cfg.max_batch);
  if (B == 0) return WF_OK;
  if (cu_seqlens[0] != 0) return fail(e, WF_ERR_INVALID_ARG, "cu_seqlens[0] must be 0");
  for (int i = 0; i < B; ++i)
    if (cu_seqlens[i + 1] <= cu_seqlens[i]) return fail(e, WF_ERR_INVALID_ARG, "cu_seqlens must increase strictly");
  if (cu_seqlens[B] > e->cfg.max_tokens) return fail(e, WF_ERR_CAPACITY, "more than max_tokens tokens");
  int slot;
  wf_status st = ring_acquire(e, &slot);
  if (st != WF_OK) return st;
  int* hm = e->meta_host[slot];
  MetaLayout ml{};
  ml.tok_off = 0;
  ml.attn_work = B + 1;
  for (int i = 0; i <= B; ++i) hm[i] = cu_seqlens[i];
  std::vector<int> order(B);
  for (int i = 0; i < B; ++i) order[i] = i;
  int nw = 0, n_items = 0;
  ml.total = ml.attn_work + build_attn_work(hm, order, e->bf16, e->cfg.n_head, hm + ml.attn_work, &nw, &n_items, e->num_sms);
  Plan p{};
  p.ml = ml;
  st = ring_upload(e, slot, p, s);
  if (st != WF_OK) return st;
  {
    Prof pr(e, 5, s);
    if (e->bf16) {
      CUtensorMap tq, tkv;
      if (!make_tmap_bf16(e->tma, &tq, qkv, 3 * e->cfg.d_model, cu_seqlens[B], 3 * e->cfg.d_model, 128) ||
          !make_tmap_bf16(e->tma, &tkv, qkv, 3 * e->cfg.d_model, cu_seqlens[B], 3 * e->cfg.d_model, 96))
        return fail(e, WF_ERR_CUDA, "cuTensorMapEncodeTiled rejected the qkv tensor map");
      launch_attention_bf16(tq, tkv, (__nv_bfloat16*)out, e->meta_dev[slot], ml, nw, n_items, e->cfg.d_model, e->err_flag, e->num_sms,
                            e->opt.pdl != 0, s);
    }
    else launch_attention_f32((const float*)qkv, (float*)out, e->meta_dev[slot], ml, nw, e->cfg.d_model, s);
  }
  WF_CUDA(e, cudaGetLastError());
  return ring_release(e, slot, s);
}

}  // extern "C"

/*
 * wf_encoder.h -- C ABI of the ragged, hush-terminated speech-encoder library (sm_100a).
 *
 * The library implements the encoding stage of a streaming speech pipeline in which each
 * audio buffer x is followed by a short fixed "hush" segment h instead of being padded to
 * 30 s (paper Sec. 4.1.2, "New paradigm: hush word": x (+) h), so that the encoder --
 * the 1,500-token, tens-of-layers cost named in Sec. 1.1 and Sec. 2.3 -- runs over real
 * tokens only.  Buffers of different lengths are batched without padding (the
 * variable-length batching problem raised in Sec. 3.3): every activation is a packed
 * [sum of rows, channels] matrix plus prefix sums.
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers on the device that was current when the
 *     encoder was created; "host" pointers are ordinary host memory.
 *   - All work is enqueued on the `stream` argument (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream).  Calls return without synchronising unless stated.
 *     Host arrays are read or written before the call returns.
 *   - The caller owns every buffer it passes.  The library owns its converted weights,
 *     tables and workspace, sized at create time and released by wf_encoder_destroy.
 *   - Errors are return codes; nothing aborts.  After a non-zero return the outputs are
 *     undefined.  wf_last_error gives a human-readable message for the last failure on a
 *     handle.  A handle is not thread-safe; distinct handles are independent.
 *   - Calls on one handle share its workspace: enqueue them on one stream, or order the streams
 *     yourself so that two calls never run on the GPU at the same time.
 *   - Row counts: a buffer of L samples has T = floor(L/160) frames (L >= 401 required);
 *     with the hush segment of H frames it has T' = T + H rows and n = ceil(T'/2) tokens.
 */
#ifndef WF_ENCODER_H
#define WF_ENCODER_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wf_encoder wf_encoder;

typedef enum {
  WF_OK = 0,
  WF_ERR_INVALID_ARG = 1,
  WF_ERR_TOO_SHORT = 2,      /* a buffer has fewer than 401 samples                        */
  WF_ERR_TOO_LONG = 3,       /* a sequence would have more than n_ctx tokens               */
  WF_ERR_CAPACITY = 4,       /* batch, samples or tokens exceed what create() sized        */
  WF_ERR_CUDA = 5,           /* a CUDA runtime/driver call failed                          */
  WF_ERR_DEVICE_TIMEOUT = 6, /* a bounded wait inside a kernel gave up                     */
  WF_ERR_UNSUPPORTED_ARCH = 7,
  WF_ERR_UNIMPLEMENTED = 8
} wf_status;

typedef enum { WF_F32 = 0, WF_BF16 = 1 } wf_dtype;

/* Model and capacity description.  d_model / n_head must be 64; d_model and d_mlp multiples
 * of 128 (d_model <= 1280); n_mel a multiple of 8, at most 128.  dtype selects the arithmetic
 * of the encoder body: WF_F32 = float32 SIMT kernels, WF_BF16 = bfloat16 tensor-core kernels
 * with float32 accumulation, a residual stream held to 16 significant bits (two bfloat16
 * planes), each LayerNorm's gain folded into the weight that follows it (the product is
 * rounded to bfloat16), bfloat16 output.  The front end is float32 in both. */
typedef struct {
  int n_mel, d_model, n_layer, n_head, d_mlp;
  int n_ctx;          /* most tokens one sequence may have (positions are a closed form)   */
  int hush_frames;    /* H; 0 = no hush segment (e.g. a 30 s padded run)                    */
  int dtype;          /* wf_dtype                                                           */
  int max_batch;      /* most sequences per call                                            */
  long max_tokens;    /* most tokens per call (sum over sequences)                          */
  long max_samples;   /* most audio samples per call (sum over sequences), below 2^31       */
} wf_config;

/* Weights: float32, device memory, read (and converted) once inside wf_encoder_create.
 * Linear weights are [out, in] row-major, conv kernels [out, in, 3].  The per-layer members
 * are HOST arrays of n_layer DEVICE pointers.  The key projection has no bias. */
typedef struct {
  const float *mel_fb;                 /* [n_mel, 201] non-negative filterbank               */
  const float *conv1_w, *conv1_b;      /* [d, n_mel, 3], [d]                                 */
  const float *conv2_w, *conv2_b;      /* [d, d, 3], [d]                                     */
  const float *const *ln1_g, *const *ln1_b;
  const float *const *wq, *const *bq, *const *wk, *const *wv, *const *bv;
  const float *const *wo, *const *bo;
  const float *const *ln2_g, *const *ln2_b;
  const float *const *w1, *const *b1;  /* [d_mlp, d], [d_mlp]                                */
  const float *const *w2, *const *b2;  /* [d, d_mlp], [d]                                    */
  const float *lnp_g, *lnp_b;          /* final LayerNorm                                    */
} wf_weights;

/* Builds an encoder on the current device: converts weights to the layouts the kernels
 * read, builds the windowed-DFT and sinusoid tables on the device, allocates workspace for
 * the stated capacities.  Synchronises `stream` before returning.  Fails with
 * WF_ERR_UNSUPPORTED_ARCH on a device that is not compute capability 10.x.
 * (Operation: the encoder of Sec. 1.1 / Sec. 2.3; weights are caller-provided.)
 * Four tuning switches of the WF_BF16 path are read from the environment here and kept in the
 * handle (a later create with another environment does not change this one):
 *   WF_PDL=0               launch kernels plainly instead of with programmatic stream
 *                          serialization (on by default: a kernel's set-up overlaps the tail of
 *                          the kernel before it);
 *   WF_GEMM_SMALL_TILES=0  never use 128 x 128 single-CTA tiles for small GEMMs;
 *   WF_GEMM_TILE=1|2|3     force 256 x 256 CTA-pair tiles, 128 x 128 or 128 x 256 single-CTA tiles for the
 *                          block GEMMs instead of letting the launcher choose by the problem's size;
 *   WF_GEMM_SPLIT_K=n      split the K range of a GEMM with few tiles over a cluster of CTAs when K
 *                          has at least n blocks of 64 (default 64; 0 = never).
 * None of them changes what is computed beyond float32 rounding order (which is fixed for a
 * given setting).  Results are bit-reproducible from call to call: no kernel of
 * the encoder combines partial results in an order that varies. */
wf_status wf_encoder_create(const wf_config *cfg, const wf_weights *w, void *stream,
                            wf_encoder **out);

/* Log-mel front end alone (Sec. 4.1.2, "target level": 16 kHz audio -> 100 rows per second):
 * reflect-padded 400-point periodic-Hann DFT every 160 samples, power, mel projection,
 * log10 with floor 1e-10, clamp to (per-buffer maximum - 8), (x + 4) / 4.
 *   audio       dev  float32, the B buffers back to back (sum of lengths samples)
 *   lengths     host B sample counts
 *   mel_out     dev  float32 [sum T_i, n_mel], rows of buffer i start at sum_{j<i} T_j
 *   frames_out  host B frame counts T_i (may be NULL) */
wf_status wf_logmel(wf_encoder *enc, const float *audio, const long *lengths, int B,
                    float *mel_out, long *frames_out, void *stream);

/* The whole path: front end, hush rows appended to each buffer's log-mel rows (x (+) h of
 * Sec. 4.1.2 at the log-mel level), conv stem, sinusoid positions restarting at 0 for every
 * sequence, n_layer pre-LN blocks whose attention sees one sequence's tokens only, final
 * LayerNorm.
 *   hush_mel        dev  float32 [hush_frames, n_mel] in normalised log-mel units;
 *                        may be NULL iff hush_frames == 0
 *   hidden_out      dev  [sum n_i, d_model]; float32 for WF_F32, bfloat16 for WF_BF16
 *   cu_seqlens_out  host B+1 token prefix sums (may be NULL) */
wf_status wf_encode(wf_encoder *enc, const float *audio, const long *lengths, int B,
                    const float *hush_mel, void *hidden_out, int *cu_seqlens_out, void *stream);

/* The paper's own variant of the method (Sec. 4.1.2 "Hush word target level", Sec. 5): the hush
 * word is a raw-audio segment (8000 samples = 0.5 s) that follows the buffer BEFORE the front
 * end, x (+) h, so frames at the junction straddle both and the per-buffer maximum sees the
 * hush frames too.  The samples are never copied: the front end reads index i >= L_i of buffer i
 * from hush_audio[i - L_i].  Needs an encoder created with hush_frames == 0.
 *   hush_audio    dev  float32 [hush_samples], shared by all buffers; hush_samples <= 16000
 *   row counts         T_i = floor((L_i + hush_samples) / 160), n_i = ceil(T_i / 2)
 * Everything else as wf_encode. */
wf_status wf_encode_raw_hush(wf_encoder *enc, const float *audio, const long *lengths, int B,
                             const float *hush_audio, int hush_samples, void *hidden_out,
                             int *cu_seqlens_out, void *stream);

/* Same as wf_encode but starting from normalised log-mel rows (e.g. from wf_logmel, or a
 * raw-audio-level hush word already concatenated by the caller with hush_frames == 0).
 *   mel     dev  float32 [sum T_i, n_mel] packed;   frames  host B row counts T_i >= 1 */
wf_status wf_encode_mel(wf_encoder *enc, const float *mel, const long *frames, int B,
                        const float *hush_mel, void *hidden_out, int *cu_seqlens_out,
                        void *stream);

/* wf_encode with HOST audio and HOST output: copies the samples to a library-owned device
 * buffer, encodes, copies the hidden states back, and synchronises `stream`.
 * `audio_host` and `hidden_out_host` should be pinned for the copies to run at full rate. */
wf_status wf_encode_host(wf_encoder *enc, const float *audio_host, const long *lengths, int B,
                         const float *hush_mel, void *hidden_out_host, int *cu_seqlens_out,
                         void *stream);

/* The same without the wait, for a caller that encodes buffer after buffer (every round of the
 * streaming pipeline re-encodes the stream's buffer, Sec. 4.3.2): the call returns once its work
 * is enqueued, and the library's two sets of staging buffers let the host-to-device copy of one
 * call and the device-to-host copy of the previous one run (on two streams of the library's own)
 * under the kernels in between.  hidden_out_host holds the result, and audio_host may be reused,
 * once wf_encode_host_wait(ticket) has returned; pass pinned memory, and do not reuse an output
 * buffer before its ticket has been waited for.  At most two calls are in flight: a third call
 * first waits for the oldest.  cu_seqlens_out is written before the call returns. */
wf_status wf_encode_host_async(wf_encoder *enc, const float *audio_host, const long *lengths, int B,
                               const float *hush_mel, void *hidden_out_host, int *cu_seqlens_out,
                               void *stream, long *ticket_out);
wf_status wf_encode_host_wait(wf_encoder *enc, long ticket);

/* The host-side planner of wf_encode / wf_encode_mel alone: no device, no encoder handle, no CUDA
 * call.  Row arithmetic of the method (Sec. 4.1.2: 100 log-mel rows per second, the hush segment
 * appended; Sec. 2.1: two rows per encoder token) and the ragged work lists, with the same
 * validation and status codes as the encoding calls.
 *   lengths             host  B sample counts, or frame counts if lengths_are_frames != 0
 *   tail_samples              raw-audio hush samples that follow every buffer (wf_encode_raw_hush), else 0
 *   num_sms                   SM count the attention work list is planned for (0: never use single-tile items)
 *   cu_seqlens_out      host  B+1 token prefix sums (may be NULL)
 *   totals_out          host  6 values: log-mel frames, rows of the padded-row layout, tokens,
 *                             front-end tiles, attention work-list entries, attention items (may be NULL)
 *   work_out, work_cap  host  the attention work list as the kernels read it (may be NULL): WF_F32 pairs
 *                             (sequence, first query row) per 16 rows; WF_BF16 triples (sequence, first query
 *                             row | kind << 30, first item) followed by one entry index per item */
wf_status wf_plan(const wf_config *cfg, const long *lengths, int B, int lengths_are_frames,
                  long tail_samples, int num_sms, int *cu_seqlens_out, long *totals_out,
                  int *work_out, int work_cap);

/* Synchronises `stream` and reports WF_ERR_DEVICE_TIMEOUT if any kernel's bounded wait gave
 * up since the last check, WF_ERR_CUDA if the stream is in error, else WF_OK. */
wf_status wf_check(wf_encoder *enc, void *stream);

/* Exercises the failure path behind WF_ERR_DEVICE_TIMEOUT without any fault: enqueues a one-warp
 * kernel that waits, through the same bounded wait as the GEMM and attention kernels but with
 * `poll_limit` polls (1 .. 2^20), on a barrier that is never signalled.  The wait runs out, the
 * kernel records it and ends normally; the next wf_check on this handle returns
 * WF_ERR_DEVICE_TIMEOUT (and clears the record), and the handle stays fully usable.
 * (Every wait of the paper's encoding stage as built here, Sec. 3.2 "Operations", is of this kind.) */
wf_status wf_selftest_wait_timeout(wf_encoder *enc, unsigned poll_limit, void *stream);

wf_status wf_encoder_destroy(wf_encoder *enc);
const char *wf_last_error(const wf_encoder *enc);

/* Per-kernel-class timing.  When enabled, every launch inside wf_encode* is bracketed by
 * CUDA events on the caller's stream.  wf_profile_read synchronises, then writes for class c
 * (0 front end, 1 layout/maps, 2 conv stem GEMMs, 3 LayerNorm kernels (WF_BF16: the final one
 * only), 4 block GEMMs, 5 attention)
 * the number of launches and their summed milliseconds since the last read, and resets. */
#define WF_N_KERNEL_CLASSES 6
wf_status wf_profile_enable(wf_encoder *enc, int on);
wf_status wf_profile_read(wf_encoder *enc, long *launches, double *millis);

/* Component entry points (used by the parity tests and for profiling one kernel alone).
 *
 * wf_gemm_bf16: C = epilogue(A W^T + bias) with the tcgen05 kernel the encoder blocks use
 * (the four GEMMs of a transformer block, Sec. 1.1).  Needs a WF_BF16 encoder.
 *   A dev bf16 [M, K] row-major, W dev bf16 [N, K] row-major, bias dev float32 [N];
 *   mode 0: C bf16 [M, N] = acc + bias;  1: C bf16 = gelu(acc + bias).
 *   K and N must be multiples of 8. */
wf_status wf_gemm_bf16(wf_encoder *enc, const void *A, const void *W, const float *bias, void *C,
                       long M, int N, int K, int mode, void *stream);

/* The three pieces with which the WF_BF16 path runs a pre-LN block (x += Wo attn(LN1 x) + bo;
 * x += W2 gelu(W1 LN2 x + b1) + b2, the blocks of the encoder of Sec. 1.1 / Sec. 2.3) without a
 * LayerNorm kernel: the residual stream x is stored as two bf16 planes, x = x_hi + x_lo with
 * x_hi = bf16(x) and x_lo = bf16(x - x_hi); x_hi doubles as the A operand of the GEMM behind a
 * LayerNorm, whose gain and shift are folded into that GEMM's weight and bias.
 *
 * wf_gemm_resid_bf16: (x_hi, x_lo) <- split(x_hi + x_lo + A W^T + bias), in place, each element
 *   by one thread (bit-reproducible).  Also writes, for every row and every 128 columns, the sum
 *   and the sum of squares of the new x:
 *   A dev bf16 [M, K], W dev bf16 [N, K], bias dev float32 [N], x_hi / x_lo dev bf16 [M, N],
 *   stats dev float32 [N / 128][M][2];  N a multiple of 128, K of 8.
 * wf_ln_fold: W dev float32 [N, K], ln_g / ln_b dev float32 [K], bias dev float32 [N] or NULL ->
 *   Wg dev bf16 [N, K] = bf16(W diag(ln_g)), colsum dev float32 [N] = row sums of Wg,
 *   cbias dev float32 [N] = bias + W ln_b.
 * wf_gemm_ln_bf16: C bf16 [M, N] = LayerNorm(x; ln_g, ln_b) W^T + bias (gelu of it if `gelu`),
 *   computed as rstd (x_hi Wg^T - mean colsum) + cbias with mean and rstd (biased variance,
 *   eps 1e-5) from `stats` [K / 128][M][2] as wf_gemm_resid_bf16 leaves them for an x of K columns.
 *   K a multiple of 128, N of 8. */
wf_status wf_gemm_resid_bf16(wf_encoder *enc, const void *A, const void *W, const float *bias,
                             void *x_hi, void *x_lo, float *stats, long M, int N, int K, void *stream);
wf_status wf_ln_fold(wf_encoder *enc, const float *W, const float *ln_g, const float *ln_b,
                     const float *bias, void *Wg, float *colsum, float *cbias, int N, int K,
                     void *stream);
wf_status wf_gemm_ln_bf16(wf_encoder *enc, const void *x_hi, const float *stats, const void *Wg,
                          const float *colsum, const float *cbias, void *C, long M, int N, int K,
                          int gelu, void *stream);

/* wf_attention: non-causal attention over packed tokens, one softmax per (sequence, head)
 * over that sequence's keys only (no padded token is computed).  qkv dev [M, 3 d_model]
 * (q | k | v, head h at columns 64 h), out dev [M, d_model]; element type follows the
 * encoder's dtype.  cu_seqlens host B+1. */
wf_status wf_attention(wf_encoder *enc, const void *qkv, const int *cu_seqlens, int B, void *out,
                       void *stream);

/* Resident stream windows (Sec. 3.2: every round a stream's audio buffer is extended at its end
 * by the newly arrived audio and now and then cut at its front once a transcript segment is
 * confirmed; Sec. 4.3.2: the buffer is re-encoded every round).  The library keeps each stream's
 * window (samples and un-normalised log-mel rows) on the device, so that a round frames only the
 * audio that is new: wf_streams_push recomputes just the frames whose 400 samples changed (the
 * new ones, the two at the old end whose reflected tail became real audio and, after a cut, the
 * first two), and wf_encode_streams runs the max / clamp / scale over the cached rows, appends the
 * hush segment and encodes.  Results are identical, bit for bit, to wf_encode on the same windows.
 *
 * wf_streams_create: windows for n_streams streams of up to max_window_samples samples each
 *   (rounded up to a multiple of 160); all windows start empty.  Device memory is allocated
 *   here and released by wf_streams_destroy (which synchronises the device first).
 * wf_streams_push: for each listed stream (ids host, B distinct ids), drop trim[i] samples at the
 *   front (a multiple of 160, at most the window; trim may be NULL), then append n_new[i]
 *   samples taken back to back from new_audio (dev float32).  The window must end up with at
 *   least 401 samples (WF_ERR_TOO_SHORT) and at most its capacity (WF_ERR_CAPACITY); on an
 *   error nothing is changed.
 * wf_streams_length: samples currently in a stream's window (host bookkeeping, no sync).
 * wf_encode_streams: as wf_encode, on the current windows of the listed streams, in the order
 *   listed. */
typedef struct wf_streams wf_streams;
wf_status wf_streams_create(wf_encoder *enc, int n_streams, long max_window_samples, wf_streams **out);
wf_status wf_streams_destroy(wf_streams *st);
wf_status wf_streams_length(const wf_streams *st, int stream_id, long *samples);
wf_status wf_streams_push(wf_streams *st, const int *ids, int B, const float *new_audio,
                          const long *n_new, const long *trim, void *stream);
wf_status wf_encode_streams(wf_streams *st, const int *ids, int B, const float *hush_mel,
                            void *hidden_out, int *cu_seqlens_out, void *stream);

/* wf_cross_kv: the cross-attention key and value projections of the encoder's output for every
 * decoder layer in one GEMM, kv = hidden W_kv^T + b_kv: the first thing prompt prefill (Sec. 3.2
 * "Operations", Sec. 4.3.2) needs from the encoding stage, and the same for every later decoding
 * round on this buffer.  Runs on the encoder's path (tcgen05 for WF_BF16, float32 SIMT else).
 *   hidden  dev  [M, d_model]                   path dtype (what wf_encode wrote)
 *   W_kv    dev  [n_dec_layers * 2 d_model, d_model] path dtype, row-major: rows
 *                [2 l d, 2 l d + d) are layer l's key weight, the next d rows its value weight
 *   b_kv    dev  float32 [n_dec_layers * 2 d_model] (the architecture's key projection has no
 *                bias: those slices are zero)
 *   kv      dev  [M, n_dec_layers * 2 d_model]  path dtype; layer l's keys are columns
 *                [2 l d, 2 l d + d) of every row, its values the next d columns
 * On the bf16 path all pointers must be 16-byte aligned. */
wf_status wf_cross_kv(wf_encoder *enc, const void *hidden, const void *W_kv, const float *b_kv,
                      long M, int n_dec_layers, void *kv, void *stream);

/* wf_dtw: dynamic time warping of B token-by-frame cost matrices (token timestamping from the
 * decoder's cross-attention, Sec. 3.2 "Workload mapping" and Sec. 4.3.2, which name DTW and give
 * no further detail: this is the classic recurrence D[i,j] = C[i,j] + min(D[i-1,j-1], D[i-1,j],
 * D[i,j-1]) with the path traced back from the last cell; float32; ties prefer the diagonal,
 * then the token step, then the frame step).
 *   cost         dev  float32, problem b is a row-major [n_tokens[b], n_frames[b]] matrix, the
 *                     problems back to back
 *   n_tokens, n_frames  host  B sizes (tokens <= 16384; fewer than 2^31 cells in total)
 *   trace_ws     dev  scratch, one byte per cost cell (caller-owned)
 *   token_start  dev  int32, sum of n_tokens entries: first frame of every token on the path
 *   total_cost   dev  float32 [B]: D at the last cell */
wf_status wf_dtw(wf_encoder *enc, const float *cost, const int *n_tokens, const int *n_frames, int B,
                 unsigned char *trace_ws, int *token_start, float *total_cost, void *stream);

/* Beam-pruning state machine (Sec. 4.2.2, "New design in beam pruning"): host-side integer logic
 * that tells a beam-search decoder which beam size to use in its next round, given the top-1
 * token of the current round and the previous round's transcript as a reference.  Decoding
 * starts with beam 1; the first comparable top-1 token is searched through the reference
 * (alignment; the aligned token counts as matched); afterwards a comparable token must equal the
 * next reference token; tokens flagged special (punctuation, timestamps, other special ids) are
 * never compared and leave the state unchanged; a failed search, a mismatch or an exhausted
 * reference restores `full_beam` until the session ends.
 *   reference   host  n_reference token ids (copied);  is_special  host  vocab_size flags (copied)
 *   wf_beam_pruner_step returns the beam size for the NEXT round, or -1 on a bad argument. */
typedef struct wf_beam_pruner wf_beam_pruner;
wf_status wf_beam_pruner_create(const int *reference, int n_reference, const unsigned char *is_special,
                                int vocab_size, int full_beam, wf_beam_pruner **out);
int wf_beam_pruner_step(wf_beam_pruner *p, int top1_token);
/* reference_index: next position to compare with (-1 before alignment); any pointer may be NULL */
wf_status wf_beam_pruner_state(const wf_beam_pruner *p, long *reference_index, int *fallen_back,
                               long *rounds, long *rounds_at_one);
wf_status wf_beam_pruner_destroy(wf_beam_pruner *p);

/* wf_attention_f32_static: wf_attention for float32 activations without an encoder handle and
 * without any allocation (the paper has no counterpart; this exists for integration only).
 * It is meant for callers that cannot call cudaMalloc: code running inside a process whose
 * device memory is owned and fully handed out by another allocator, or a plug-in that is
 * given pointers and must not grow its host's footprint.  Such callers cannot create an
 * encoder, because create() allocates workspace.  Here the per-call index arrays (token prefix
 * sums and query-tile list) live in a fixed 35 KB array inside the library image, held by
 * every GPU that loads the library until the process exits.
 *   qkv dev float32 [M, 3 d_model] (q | k | v, head h at columns 64 h), out dev float32
 *   [M, d_model], cu_seqlens host B+1 strictly increasing from 0; d_model a multiple of 64.
 * Limits: B <= 256 and M <= 65,536, else WF_ERR_CAPACITY.  No cudaMalloc, cudaFree or other
 * allocating call is made.  The first call on a device looks up the array's device address
 * (once per device, with that device current); make that first call outside any stream
 * capture.  A call on a stream that is being captured is rejected (WF_ERR_INVALID_ARG): the
 * index arrays are copied from the call's own stack frame.  That copy makes the host wait for
 * earlier work on the stream, so unlike the other entry points this one does not return early.
 * All calls on a device share the array and each overwrites what it reads, so calls are safe
 * back to back on one stream, but calls that may overlap on the GPU (different streams without
 * ordering between them) race on it.  Not thread-safe: call it from one host thread at a time. */
wf_status wf_attention_f32_static(const float *qkv, const int *cu_seqlens, int B, int d_model,
                                  float *out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* WF_ENCODER_H */

// An attention entry point for callers that may not allocate device memory.
//
// The regular entry points keep their per-call index arrays (token prefix sums and the
// list of query tiles) in workspace that wf_encoder_create obtained with cudaMalloc.  Code
// that runs where cudaMalloc is off limits -- inside a process whose memory pool is owned and
// fully handed out by another allocator, or in a plug-in that is only given pointers and
// must not grow the footprint of its host -- cannot create an encoder at all.  For those
// callers the index arrays of this one entry point live in a fixed array that is part of
// the library image on every GPU that loads it.
#include "wf_internal.h"

namespace {

constexpr int kStaticMaxBatch = 256;      // most sequences per call
constexpr int kStaticMaxTokens = 65536;   // most tokens per call
constexpr int kStaticQueryTile = 16;      // query rows per CTA of the float32 attention kernel
constexpr int kStaticMaxWork = kStaticMaxTokens / kStaticQueryTile + kStaticMaxBatch;
constexpr int kStaticInts = (kStaticMaxBatch + 1) + 2 * kStaticMaxWork;   // 8,961 ints, 35 KB

// Scratch shared by every call on a device.  Nothing in it has to start at zero: each call
// overwrites the part it reads (prefix sums, then work list) before its kernel runs.
static __device__ __align__(256) int g_static_meta[kStaticInts];

// Device address of the array on each device, looked up on first use.  Plain host state: calls
// from several host threads at once are not supported.
constexpr int kMaxDevices = 64;
int* g_static_meta_ptr[kMaxDevices] = {nullptr};

}  // namespace

extern "C" wf_status wf_attention_f32_static(const float* qkv, const int* cu_seqlens, int B, int d_model,
                                             float* out, void* stream) {
  if (B < 0 || d_model <= 0 || d_model % wf::kHeadDim != 0) return WF_ERR_INVALID_ARG;
  if (B == 0) return WF_OK;
  if (!qkv || !cu_seqlens || !out) return WF_ERR_INVALID_ARG;
  if (B > kStaticMaxBatch) return WF_ERR_CAPACITY;
  if (cu_seqlens[0] != 0) return WF_ERR_INVALID_ARG;
  for (int i = 0; i < B; ++i)
    if (cu_seqlens[i + 1] <= cu_seqlens[i]) return WF_ERR_INVALID_ARG;
  if (cu_seqlens[B] > kStaticMaxTokens) return WF_ERR_CAPACITY;

  cudaStream_t s = (cudaStream_t)stream;
  // The index arrays are uploaded from this call's stack frame: a captured copy would outlive it.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) return WF_ERR_CUDA;
  if (cap != cudaStreamCaptureStatusNone) return WF_ERR_INVALID_ARG;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return WF_ERR_CUDA;
  if (g_static_meta_ptr[dev] == nullptr) {
    // The array's name is only a handle on the host; the kernel needs its device address.
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_static_meta) != cudaSuccess || p == nullptr) return WF_ERR_CUDA;
    g_static_meta_ptr[dev] = p;
  }
  int* meta_dev = g_static_meta_ptr[dev];

  int host_meta[kStaticInts];  // on the stack: no host allocation either
  wf::MetaLayout ml{};
  ml.tok_off = 0;
  ml.attn_work = B + 1;
  for (int i = 0; i <= B; ++i) host_meta[i] = cu_seqlens[i];
  int nw = 0;
  for (int i = 0; i < B; ++i)
    for (int q0 = 0; q0 < cu_seqlens[i + 1] - cu_seqlens[i]; q0 += kStaticQueryTile) {
      host_meta[ml.attn_work + 2 * nw] = i;
      host_meta[ml.attn_work + 2 * nw + 1] = q0;
      ++nw;
    }
  ml.total = ml.attn_work + 2 * nw;
  // Pageable source: the runtime has taken its copy of host_meta when this call returns (which
  // makes the host wait for earlier work on the stream).
  if (cudaMemcpyAsync(meta_dev, host_meta, (size_t)ml.total * sizeof(int), cudaMemcpyHostToDevice, s) != cudaSuccess)
    return WF_ERR_CUDA;
  cudaGetLastError();  // an error left behind by earlier work is not this launch's
  wf::launch_attention_f32(qkv, out, meta_dev, ml, nw, d_model, s);
  return cudaGetLastError() == cudaSuccess ? WF_OK : WF_ERR_CUDA;
}

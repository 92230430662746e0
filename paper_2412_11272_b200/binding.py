"""ctypes binding of libwf_encoder.so: argument marshalling only.

Every step of the encoding path runs inside the library's CUDA kernels; this module turns
torch tensors into pointers, keeps them alive, and raises on error codes.  PyTorch is used
for device memory and streams, nothing else.  There is no CPU fallback: if the shared
library is missing or cannot be loaded, importing the handle raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwf_encoder.so")

WF_F32, WF_BF16 = 0, 1
STATUS = {0: "WF_OK", 1: "WF_ERR_INVALID_ARG", 2: "WF_ERR_TOO_SHORT", 3: "WF_ERR_TOO_LONG",
          4: "WF_ERR_CAPACITY", 5: "WF_ERR_CUDA", 6: "WF_ERR_DEVICE_TIMEOUT",
          7: "WF_ERR_UNSUPPORTED_ARCH", 8: "WF_ERR_UNIMPLEMENTED"}
N_KERNEL_CLASSES = 6
KERNEL_CLASSES = ("front_end", "layout", "conv_gemm", "layernorm", "block_gemm", "attention")


class WfError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"{STATUS.get(code, code)}: {message}")
        self.code = code
        self.status = STATUS.get(code, str(code))


class wf_config(C.Structure):
    _fields_ = [("n_mel", C.c_int), ("d_model", C.c_int), ("n_layer", C.c_int), ("n_head", C.c_int),
                ("d_mlp", C.c_int), ("n_ctx", C.c_int), ("hush_frames", C.c_int), ("dtype", C.c_int),
                ("max_batch", C.c_int), ("max_tokens", C.c_long), ("max_samples", C.c_long)]


_PP = C.POINTER(C.c_void_p)


class wf_weights(C.Structure):
    _fields_ = [("mel_fb", C.c_void_p), ("conv1_w", C.c_void_p), ("conv1_b", C.c_void_p),
                ("conv2_w", C.c_void_p), ("conv2_b", C.c_void_p),
                ("ln1_g", _PP), ("ln1_b", _PP), ("wq", _PP), ("bq", _PP), ("wk", _PP), ("wv", _PP),
                ("bv", _PP), ("wo", _PP), ("bo", _PP), ("ln2_g", _PP), ("ln2_b", _PP),
                ("w1", _PP), ("b1", _PP), ("w2", _PP), ("b2", _PP),
                ("lnp_g", C.c_void_p), ("lnp_b", C.c_void_p)]


_PER_LAYER = ("ln1_g", "ln1_b", "wq", "bq", "wk", "wv", "bv", "wo", "bo", "ln2_g", "ln2_b",
              "w1", "b1", "w2", "b2")

EXPORTS = ("wf_encoder_create", "wf_logmel", "wf_encode", "wf_encode_raw_hush", "wf_encode_mel", "wf_encode_host", "wf_encode_host_async", "wf_encode_host_wait", "wf_check",
           "wf_encoder_destroy", "wf_last_error", "wf_profile_enable", "wf_profile_read",
           "wf_plan", "wf_gemm_bf16", "wf_gemm_resid_bf16", "wf_ln_fold", "wf_gemm_ln_bf16", "wf_selftest_wait_timeout", "wf_attention", "wf_cross_kv", "wf_dtw",
           "wf_streams_create", "wf_streams_destroy", "wf_streams_length", "wf_streams_push", "wf_encode_streams", "wf_attention_f32_static",
           "wf_beam_pruner_create", "wf_beam_pruner_step", "wf_beam_pruner_state", "wf_beam_pruner_destroy")

_lib = None


def load_library() -> C.CDLL:
    """Loads the shared library (building it is the job of ``paper_2412_11272_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2412_11272_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, ip, lp = C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_long)
    lib.wf_encoder_create.argtypes = [C.POINTER(wf_config), C.POINTER(wf_weights), vp, C.POINTER(vp)]
    lib.wf_logmel.argtypes = [vp, vp, lp, C.c_int, vp, lp, vp]
    lib.wf_encode.argtypes = [vp, vp, lp, C.c_int, vp, vp, ip, vp]
    lib.wf_encode_mel.argtypes = [vp, vp, lp, C.c_int, vp, vp, ip, vp]
    lib.wf_encode_raw_hush.argtypes = [vp, vp, lp, C.c_int, vp, C.c_int, vp, ip, vp]
    lib.wf_encode_host.argtypes = [vp, vp, lp, C.c_int, vp, vp, ip, vp]
    lib.wf_encode_host_async.argtypes = [vp, vp, lp, C.c_int, vp, vp, ip, vp, lp]
    lib.wf_encode_host_wait.argtypes = [vp, C.c_long]
    lib.wf_check.argtypes = [vp, vp]
    lib.wf_encoder_destroy.argtypes = [vp]
    lib.wf_last_error.argtypes = [vp]
    lib.wf_last_error.restype = C.c_char_p
    lib.wf_plan.argtypes = [C.POINTER(wf_config), lp, C.c_int, C.c_int, C.c_long, C.c_int, ip, lp, ip, C.c_int]
    lib.wf_selftest_wait_timeout.argtypes = [vp, C.c_uint, vp]
    lib.wf_profile_enable.argtypes = [vp, C.c_int]
    lib.wf_profile_read.argtypes = [vp, lp, C.POINTER(C.c_double)]
    lib.wf_gemm_bf16.argtypes = [vp, vp, vp, vp, vp, C.c_long, C.c_int, C.c_int, C.c_int, vp]
    lib.wf_gemm_resid_bf16.argtypes = [vp, vp, vp, vp, vp, vp, vp, C.c_long, C.c_int, C.c_int, vp]
    lib.wf_ln_fold.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, C.c_int, C.c_int, vp]
    lib.wf_gemm_ln_bf16.argtypes = [vp, vp, vp, vp, vp, vp, vp, C.c_long, C.c_int, C.c_int, C.c_int, vp]
    lib.wf_attention.argtypes = [vp, vp, ip, C.c_int, vp, vp]
    lib.wf_cross_kv.argtypes = [vp, vp, vp, vp, C.c_long, C.c_int, vp, vp]
    lib.wf_streams_create.argtypes = [vp, C.c_int, C.c_long, C.POINTER(vp)]
    lib.wf_streams_destroy.argtypes = [vp]
    lib.wf_streams_length.argtypes = [vp, C.c_int, lp]
    lib.wf_streams_push.argtypes = [vp, ip, C.c_int, vp, lp, lp, vp]
    lib.wf_encode_streams.argtypes = [vp, ip, C.c_int, vp, vp, ip, vp]
    lib.wf_dtw.argtypes = [vp, vp, ip, ip, C.c_int, vp, vp, vp, vp]
    lib.wf_attention_f32_static.argtypes = [vp, ip, C.c_int, C.c_int, vp, vp]
    lib.wf_beam_pruner_create.argtypes = [ip, C.c_int, C.POINTER(C.c_ubyte), C.c_int, C.c_int, C.POINTER(vp)]
    lib.wf_beam_pruner_step.argtypes = [vp, C.c_int]
    lib.wf_beam_pruner_state.argtypes = [vp, lp, ip, lp, lp]
    lib.wf_beam_pruner_destroy.argtypes = [vp]
    for name in EXPORTS:
        if name != "wf_last_error":
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _stream_ptr(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _longs(values):
    arr = np.ascontiguousarray(np.asarray(values, dtype=np.int64))
    return arr, arr.ctypes.data_as(C.POINTER(C.c_long))


class Encoder:
    """Owns one ``wf_encoder`` handle.  ``weights`` maps the names of
    ``inputs.encoder_weights`` to float32 arrays (numpy or torch); they are moved to the
    current CUDA device and may be released by the caller afterwards."""

    def __init__(self, shape, weights: dict, mel_fb, max_batch: int, max_tokens: int, max_samples: int,
                 hush_frames: int | None = None, n_ctx: int | None = None, dtype: str | None = None,
                 device="cuda:0"):
        self.lib = load_library()
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.shape = shape
        self.dtype = dtype or shape.dtype
        self.hush_frames = shape.hush_frames if hush_frames is None else hush_frames
        self.n_ctx = shape.n_ctx if n_ctx is None else n_ctx
        self.d_model = shape.d_model
        self.n_mel = shape.n_mel
        self.out_dtype = torch.bfloat16 if self.dtype == "bf16" else torch.float32
        cfg = wf_config(shape.n_mel, shape.d_model, shape.n_layer, shape.n_head, shape.d_mlp, self.n_ctx,
                        self.hush_frames, WF_BF16 if self.dtype == "bf16" else WF_F32,
                        int(max_batch), int(max_tokens), int(max_samples))
        dev = {}

        def put(a):
            t = torch.as_tensor(np.ascontiguousarray(a) if isinstance(a, np.ndarray) else a)
            return t.to(device=self.device, dtype=torch.float32).contiguous()

        w = wf_weights()
        for name in ("conv1_w", "conv1_b", "conv2_w", "conv2_b", "lnp_g", "lnp_b"):
            dev[name] = put(weights[name])
            setattr(w, name, dev[name].data_ptr())
        dev["mel_fb"] = put(mel_fb)
        w.mel_fb = dev["mel_fb"].data_ptr()
        arrays = {}
        for name in _PER_LAYER:
            arr = (C.c_void_p * max(shape.n_layer, 1))()
            for l in range(shape.n_layer):
                dev[f"{name}.{l}"] = put(weights[f"{name}.{l}"])
                arr[l] = dev[f"{name}.{l}"].data_ptr()
            arrays[name] = arr
            setattr(w, name, C.cast(arr, _PP))
        handle = C.c_void_p()
        st = self.lib.wf_encoder_create(C.byref(cfg), C.byref(w), _stream_ptr(), C.byref(handle))
        self.handle = handle
        if st != 0:
            msg = self.lib.wf_last_error(handle).decode() if handle else "create failed"
            if handle:
                self.lib.wf_encoder_destroy(handle)
            self.handle = None
            raise WfError(st, msg)
        torch.cuda.synchronize()
        del dev, arrays  # the library holds its own converted copies

    # -- helpers
    def _check(self, st: int):
        if st != 0:
            raise WfError(st, self.lib.wf_last_error(self.handle).decode())

    def close(self):
        if getattr(self, "handle", None):
            self.lib.wf_encoder_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- entry points (same names as the C ABI)
    def wf_logmel(self, audio: torch.Tensor, lengths, stream=None):
        """audio: float32 CUDA tensor of packed samples.  Returns (mel [sum T, n_mel] f32, frames)."""
        arr, ptr = _longs(lengths)
        B = len(arr)
        total_frames = int((arr // 160).sum())
        mel = torch.empty((total_frames, self.n_mel), dtype=torch.float32, device=self.device)
        frames = np.zeros(max(B, 1), dtype=np.int64)
        self._check(self.lib.wf_logmel(self.handle, audio.data_ptr() if B else None, ptr, B, mel.data_ptr(),
                                       frames.ctypes.data_as(C.POINTER(C.c_long)), _stream_ptr(stream)))
        return mel, frames[:B]

    def _tokens(self, frames):
        return (np.asarray(frames, dtype=np.int64) + self.hush_frames + 1) // 2

    def wf_encode(self, audio: torch.Tensor, lengths, hush_mel: torch.Tensor | None, out=None, stream=None):
        """Returns (hidden [sum n_i, d_model], cu_seqlens int32 numpy [B+1]).  No host sync."""
        arr, ptr = _longs(lengths)
        B = len(arr)
        M = int(self._tokens(arr // 160).sum())
        if out is None:
            out = torch.empty((M, self.d_model), dtype=self.out_dtype, device=self.device)
        cu = np.zeros(B + 1, dtype=np.int32)
        self._check(self.lib.wf_encode(self.handle, audio.data_ptr() if B else None, ptr, B,
                                       hush_mel.data_ptr() if hush_mel is not None else None,
                                       out.data_ptr(), cu.ctypes.data_as(C.POINTER(C.c_int)),
                                       _stream_ptr(stream)))
        return out, cu

    def wf_encode_raw_hush(self, audio: torch.Tensor, lengths, hush_audio: torch.Tensor, out=None, stream=None):
        """Hush word at raw-audio level: float32 CUDA samples appended (virtually) to every buffer."""
        arr, ptr = _longs(lengths)
        B = len(arr)
        hs = int(hush_audio.numel())
        M = int(self._tokens((arr + hs) // 160).sum())
        if out is None:
            out = torch.empty((M, self.d_model), dtype=self.out_dtype, device=self.device)
        cu = np.zeros(B + 1, dtype=np.int32)
        self._check(self.lib.wf_encode_raw_hush(self.handle, audio.data_ptr() if B else None, ptr, B,
                                                hush_audio.data_ptr(), hs, out.data_ptr(),
                                                cu.ctypes.data_as(C.POINTER(C.c_int)), _stream_ptr(stream)))
        return out, cu

    def wf_encode_mel(self, mel: torch.Tensor, frames, hush_mel, out=None, stream=None):
        arr, ptr = _longs(frames)
        B = len(arr)
        M = int(self._tokens(arr).sum())
        if out is None:
            out = torch.empty((M, self.d_model), dtype=self.out_dtype, device=self.device)
        cu = np.zeros(B + 1, dtype=np.int32)
        self._check(self.lib.wf_encode_mel(self.handle, mel.data_ptr() if B else None, ptr, B,
                                           hush_mel.data_ptr() if hush_mel is not None else None,
                                           out.data_ptr(), cu.ctypes.data_as(C.POINTER(C.c_int)),
                                           _stream_ptr(stream)))
        return out, cu

    def wf_encode_host(self, audio_host: torch.Tensor, lengths, hush_mel, out_host: torch.Tensor, stream=None):
        """audio_host / out_host: (pinned) CPU tensors.  Copies in, encodes, copies out, synchronises."""
        arr, ptr = _longs(lengths)
        B = len(arr)
        cu = np.zeros(B + 1, dtype=np.int32)
        self._check(self.lib.wf_encode_host(self.handle, audio_host.data_ptr(), ptr, B,
                                            hush_mel.data_ptr() if hush_mel is not None else None,
                                            out_host.data_ptr(), cu.ctypes.data_as(C.POINTER(C.c_int)),
                                            _stream_ptr(stream)))
        return out_host, cu

    def wf_encode_host_async(self, audio_host: torch.Tensor, lengths, hush_mel, out_host: torch.Tensor, stream=None):
        """As wf_encode_host without the wait: returns (ticket, cu_seqlens); out_host is valid after
        wf_encode_host_wait(ticket)."""
        arr, ptr = _longs(lengths)
        B = len(arr)
        cu = np.zeros(B + 1, dtype=np.int32)
        ticket = C.c_long(0)
        self._check(self.lib.wf_encode_host_async(self.handle, audio_host.data_ptr(), ptr, B,
                                                  hush_mel.data_ptr() if hush_mel is not None else None,
                                                  out_host.data_ptr(), cu.ctypes.data_as(C.POINTER(C.c_int)),
                                                  _stream_ptr(stream), C.byref(ticket)))
        return int(ticket.value), cu

    def wf_encode_host_wait(self, ticket: int):
        self._check(self.lib.wf_encode_host_wait(self.handle, ticket))

    def wf_check(self, stream=None):
        self._check(self.lib.wf_check(self.handle, _stream_ptr(stream)))

    def wf_selftest_wait_timeout(self, poll_limit: int = 4096, stream=None):
        self._check(self.lib.wf_selftest_wait_timeout(self.handle, poll_limit, _stream_ptr(stream)))

    def wf_profile_enable(self, on: bool):
        self._check(self.lib.wf_profile_enable(self.handle, 1 if on else 0))

    def wf_profile_read(self) -> dict:
        n = (C.c_long * N_KERNEL_CLASSES)()
        ms = (C.c_double * N_KERNEL_CLASSES)()
        self._check(self.lib.wf_profile_read(self.handle, n, ms))
        return {KERNEL_CLASSES[i]: {"launches": int(n[i]), "ms": float(ms[i])} for i in range(N_KERNEL_CLASSES)}

    def wf_gemm_bf16(self, A: torch.Tensor, W: torch.Tensor, bias: torch.Tensor, mode: int, C_out=None,
                     stream=None):
        M, K = A.shape
        N = W.shape[0]
        if C_out is None:
            C_out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
        self._check(self.lib.wf_gemm_bf16(self.handle, A.data_ptr(), W.data_ptr(), bias.data_ptr(),
                                          C_out.data_ptr(), M, N, K, mode, _stream_ptr(stream)))
        return C_out

    def wf_gemm_resid_bf16(self, A: torch.Tensor, W: torch.Tensor, bias: torch.Tensor, x_hi: torch.Tensor,
                           x_lo: torch.Tensor, stream=None):
        """(x_hi, x_lo) <- split(x_hi + x_lo + A W^T + bias) in place; returns the row statistics
        [N / 128, M, 2] (sum and sum of squares of every 128 columns of the new x)."""
        M, K = A.shape
        N = W.shape[0]
        stats = torch.empty((max(N // 128, 1), M, 2), dtype=torch.float32, device=A.device)
        self._check(self.lib.wf_gemm_resid_bf16(self.handle, A.data_ptr(), W.data_ptr(), bias.data_ptr(), x_hi.data_ptr(),
                                                x_lo.data_ptr(), stats.data_ptr(), M, N, K, _stream_ptr(stream)))
        return stats

    def wf_ln_fold(self, W: torch.Tensor, ln_g: torch.Tensor, ln_b: torch.Tensor, bias: torch.Tensor | None, stream=None):
        """W float32 [N, K] -> (Wg bf16 [N, K], colsum float32 [N], cbias float32 [N])."""
        N, K = W.shape
        Wg = torch.empty((N, K), dtype=torch.bfloat16, device=W.device)
        colsum = torch.empty(N, dtype=torch.float32, device=W.device)
        cbias = torch.empty(N, dtype=torch.float32, device=W.device)
        self._check(self.lib.wf_ln_fold(self.handle, W.data_ptr(), ln_g.data_ptr(), ln_b.data_ptr(),
                                        bias.data_ptr() if bias is not None else None, Wg.data_ptr(), colsum.data_ptr(),
                                        cbias.data_ptr(), N, K, _stream_ptr(stream)))
        return Wg, colsum, cbias

    def wf_gemm_ln_bf16(self, x_hi: torch.Tensor, stats: torch.Tensor, Wg: torch.Tensor, colsum: torch.Tensor,
                        cbias: torch.Tensor, gelu: bool, stream=None):
        """C bf16 [M, N] = (gelu of) LayerNorm(x) W^T + bias from x_hi, the row statistics of x and folded weights."""
        M, K = x_hi.shape
        N = Wg.shape[0]
        out = torch.empty((M, N), dtype=torch.bfloat16, device=x_hi.device)
        self._check(self.lib.wf_gemm_ln_bf16(self.handle, x_hi.data_ptr(), stats.data_ptr(), Wg.data_ptr(), colsum.data_ptr(),
                                             cbias.data_ptr(), out.data_ptr(), M, N, K, 1 if gelu else 0, _stream_ptr(stream)))
        return out

    def wf_cross_kv(self, hidden: torch.Tensor, W_kv: torch.Tensor, b_kv: torch.Tensor, kv_out=None, stream=None):
        """hidden [M, d], W_kv [n_dec * 2 d, d] (path dtype), b_kv float32 [n_dec * 2 d] -> kv [M, n_dec * 2 d]."""
        M, d = hidden.shape
        n_dec = W_kv.shape[0] // (2 * d)
        if kv_out is None:
            kv_out = torch.empty((M, W_kv.shape[0]), dtype=hidden.dtype, device=hidden.device)
        self._check(self.lib.wf_cross_kv(self.handle, hidden.data_ptr(), W_kv.data_ptr(), b_kv.data_ptr(), M, n_dec,
                                         kv_out.data_ptr(), _stream_ptr(stream)))
        return kv_out

    def wf_dtw(self, cost: torch.Tensor, n_tokens, n_frames, stream=None):
        """cost: float32 CUDA tensor holding the B matrices back to back.  Returns
        (token_start int32 [sum n_tokens], total_cost float32 [B]) as CUDA tensors."""
        nt = np.ascontiguousarray(np.asarray(n_tokens, dtype=np.int32))
        nf = np.ascontiguousarray(np.asarray(n_frames, dtype=np.int32))
        B = len(nt)
        cells = int((nt.astype(np.int64) * nf).sum())
        trace = torch.empty(max(cells, 1), dtype=torch.uint8, device=cost.device)
        start = torch.empty(max(int(nt.sum()), 1), dtype=torch.int32, device=cost.device)
        total = torch.empty(max(B, 1), dtype=torch.float32, device=cost.device)
        ip = C.POINTER(C.c_int)
        self._check(self.lib.wf_dtw(self.handle, cost.data_ptr(), nt.ctypes.data_as(ip), nf.ctypes.data_as(ip), B,
                                    trace.data_ptr(), start.data_ptr(), total.data_ptr(), _stream_ptr(stream)))
        return start[:int(nt.sum())], total[:B]

    def wf_attention(self, qkv: torch.Tensor, cu_seqlens, stream=None):
        cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
        out = torch.empty((qkv.shape[0], self.d_model), dtype=qkv.dtype, device=qkv.device)
        self._check(self.lib.wf_attention(self.handle, qkv.data_ptr(), cu.ctypes.data_as(C.POINTER(C.c_int)),
                                          len(cu) - 1, out.data_ptr(), _stream_ptr(stream)))
        return out


def wf_plan(shape, lengths, hush_frames: int, max_batch: int, max_tokens: int, max_samples: int, frames_given=False,
            tail_samples: int = 0, num_sms: int = 148, n_ctx=None):
    """The host-side planner alone (no GPU): returns (cu_seqlens, totals dict, attention work list)."""
    lib = load_library()
    cfg = wf_config(shape.n_mel, shape.d_model, shape.n_layer, shape.n_head, shape.d_mlp, n_ctx or shape.n_ctx, hush_frames,
                    1 if shape.dtype == "bf16" else 0, max_batch, max_tokens, max_samples)
    B = len(lengths)
    arr, ptr = _longs(lengths)
    cu = (C.c_int * (B + 1))()
    totals = (C.c_long * 6)()
    cap = 8 * (max_tokens // 16 + B + 4) + 4 * (max_tokens // 128 + 2 * B + 2) * max(shape.n_head, 1)
    work = (C.c_int * cap)()
    st = lib.wf_plan(C.byref(cfg), ptr, B, 1 if frames_given else 0, tail_samples, num_sms, cu, totals, work, cap)
    if st != 0:
        raise WfError(st, "wf_plan rejected the batch")
    names = ("frames", "padded_rows", "tokens", "front_end_tiles", "attention_entries", "attention_items")
    t = dict(zip(names, [int(v) for v in totals]))
    n = (2 * t["attention_entries"]) if shape.dtype != "bf16" else (3 * t["attention_entries"] + t["attention_items"])
    return np.array(cu[:B + 1]), t, np.array(work[:n])


def wf_attention_f32_static(qkv: torch.Tensor, cu_seqlens, d_model: int, out: torch.Tensor, stream=None):
    """Handle-free float32 attention that makes no allocation of its own: the caller passes the
    output tensor too.  For code that may not call cudaMalloc (see the header).  Raises WfError."""
    lib = load_library()
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    st = lib.wf_attention_f32_static(qkv.data_ptr(), cu.ctypes.data_as(C.POINTER(C.c_int)), len(cu) - 1,
                                     int(d_model), out.data_ptr(), _stream_ptr(stream))
    if st != 0:
        raise WfError(st, "wf_attention_f32_static rejected its arguments or a CUDA call failed")
    return out


class Streams:
    """Resident windows of ``n_streams`` audio streams on an encoder's device (``wf_streams_*``)."""

    def __init__(self, enc: Encoder, n_streams: int, max_window_samples: int):
        self.enc = enc
        self.handle = C.c_void_p()
        enc._check(enc.lib.wf_streams_create(enc.handle, n_streams, max_window_samples, C.byref(self.handle)))

    def close(self):
        if self.handle:
            self.enc.lib.wf_streams_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def wf_streams_length(self, stream_id: int) -> int:
        n = C.c_long()
        self.enc._check(self.enc.lib.wf_streams_length(self.handle, stream_id, C.byref(n)))
        return n.value

    def wf_streams_push(self, ids, new_audio: torch.Tensor | None, n_new, trim=None, stream=None):
        """Drops ``trim[i]`` samples at the front of stream ``ids[i]`` and appends ``n_new[i]`` samples
        taken back to back from ``new_audio`` (float32 CUDA)."""
        idv = np.ascontiguousarray(np.asarray(ids, dtype=np.int32))
        nn, nn_ptr = _longs(n_new)
        tr_ptr = None
        if trim is not None:
            tr, tr_ptr = _longs(trim)
        self.enc._check(self.enc.lib.wf_streams_push(
            self.handle, idv.ctypes.data_as(C.POINTER(C.c_int)), len(idv),
            new_audio.data_ptr() if new_audio is not None and new_audio.numel() else None, nn_ptr, tr_ptr,
            _stream_ptr(stream)))

    def wf_encode_streams(self, ids, hush_mel: torch.Tensor | None, out=None, stream=None):
        """Encodes the current windows of the listed streams; returns (hidden, cu_seqlens)."""
        enc = self.enc
        idv = np.ascontiguousarray(np.asarray(ids, dtype=np.int32))
        B = len(idv)
        frames = np.array([self.wf_streams_length(int(i)) // 160 for i in idv], dtype=np.int64)
        M = int(enc._tokens(frames).sum()) if B else 0
        if out is None:
            out = torch.empty((M, enc.d_model), dtype=enc.out_dtype, device=enc.device)
        cu = np.zeros(B + 1, dtype=np.int32)
        enc._check(enc.lib.wf_encode_streams(self.handle, idv.ctypes.data_as(C.POINTER(C.c_int)), B,
                                             hush_mel.data_ptr() if hush_mel is not None else None, out.data_ptr(),
                                             cu.ctypes.data_as(C.POINTER(C.c_int)), _stream_ptr(stream)))
        return out, cu


class BeamPruner:
    """Marshals the host-side beam-pruning state machine (wf_beam_pruner_*)."""

    def __init__(self, reference, is_special, full_beam: int = 5):
        self.lib = load_library()
        ref = np.ascontiguousarray(np.asarray(reference, dtype=np.int32))
        flags = np.ascontiguousarray(np.asarray(is_special, dtype=np.uint8))
        h = C.c_void_p()
        st = self.lib.wf_beam_pruner_create(ref.ctypes.data_as(C.POINTER(C.c_int)), len(ref),
                                            flags.ctypes.data_as(C.POINTER(C.c_ubyte)), len(flags), int(full_beam),
                                            C.byref(h))
        if st != 0:
            raise WfError(st, "wf_beam_pruner_create rejected its arguments")
        self.handle = h

    def step(self, top1: int) -> int:
        r = self.lib.wf_beam_pruner_step(self.handle, int(top1))
        if r < 0:
            raise WfError(1, "wf_beam_pruner_step: token id outside the vocabulary")
        return r

    def state(self):
        idx, rounds, ones, fb = C.c_long(), C.c_long(), C.c_long(), C.c_int()
        self.lib.wf_beam_pruner_state(self.handle, C.byref(idx), C.byref(fb), C.byref(rounds), C.byref(ones))
        return {"reference_index": idx.value, "fallen_back": bool(fb.value), "rounds": rounds.value,
                "rounds_at_one": ones.value}

    def close(self):
        if getattr(self, "handle", None):
            self.lib.wf_beam_pruner_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

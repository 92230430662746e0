"""fp64 CPU oracle for the hush-terminated encoding stage.  TEST INFRASTRUCTURE ONLY.

This file is the yardstick the CUDA library is checked against.  It is imported by the
tests, by the smoke check and by the benchmark's CPU-baseline leg, never by the
library or its Python binding, and it shares no code with them.

What it computes (one sequence at a time; a batch is a Python loop over sequences):

* the method itself -- Sec. 4.1.2 ("New paradigm: hush word"): the buffer x is followed by
  a short fixed hush segment h (x (+) h) and the encoder then runs over the real tokens
  only, with no padding to 30 s.  Sec. 4.1.2 ("Hush word target level") names two levels at
  which the segment can be attached, raw audio and log-mel; both are here
  (``hush_level='audio'`` concatenates samples before framing, ``'mel'`` concatenates
  rows after the log-mel normalisation);
* the front end -- Sec. 4.1.2 states 16 kHz audio and a log-mel matrix of shape (100, 80) per
  second; Sec. 1.1 / Sec. 2.1 state 30 s -> 1500 encoder tokens.  The paper gives no further
  arithmetic (it builds on the Whisper architecture), so every step below is the plain
  textbook definition of that architecture's operator, written with explicit sums or one
  library matmul per step, in float64, with no blocking, fusion or reordering.

Readings where the paper is silent (window, padding, epsilon, ...) are stated in the
docstrings of the functions that take them.

Every function is pinned by tests that do not re-use its own formula
(tests/test_oracle_pins.py): paper shape facts, closed forms of the DFT of a sine,
Parseval, convolution identities, attention/LayerNorm invariants, batch invariance, and a
second scalar evaluation of the whole path on tiny dimensions.  Nothing here is
"parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf as _erf

SAMPLE_RATE = 16000
N_FFT = 400
HOP = 160
N_BINS = 201


# --------------------------------------------------------------------------- front end

def n_frames(n_samples: int) -> int:
    """Frames of a buffer: one per hop, T = floor(L / 160) (Sec. 4.1.2: 1 s -> 100 rows).
    Frames are centred on multiples of the hop; the frame that would be centred on the
    last hop boundary is dropped."""
    return n_samples // HOP


def reflect_pad(x: np.ndarray, pad: int = N_FFT // 2) -> np.ndarray:
    """xp[j] = x[reflect(j - pad)] with reflect(-k) = k and reflect(L-1+k) = L-1-k
    (mirror without repeating the edge sample).  Needs L > pad."""
    x = np.asarray(x, dtype=np.float64)
    L = x.shape[0]
    if L <= pad:
        raise ValueError("buffer shorter than the reflect padding")
    out = np.empty(L + 2 * pad, dtype=np.float64)
    for j in range(L + 2 * pad):
        i = j - pad
        if i < 0:
            i = -i
        elif i > L - 1:
            i = 2 * (L - 1) - i
        out[j] = x[i]
    return out


def hann_window(n: int = N_FFT) -> np.ndarray:
    """Periodic Hann window w[i] = 0.5 - 0.5 cos(2 pi i / n)."""
    i = np.arange(n, dtype=np.float64)
    return 0.5 - 0.5 * np.cos(2.0 * math.pi * i / n)


def dft_power(x: np.ndarray) -> np.ndarray:
    """Power spectrum of every frame, P[t, k] = |sum_n w[n] xp[160 t + n] e^{-2 pi i k n / 400}|^2,
    k = 0..200, by the direct O(N^2) sum (angles reduced as (k n) mod 400 so the table is exact)."""
    xp = reflect_pad(x)
    T = n_frames(len(x))
    w = hann_window()
    k = np.arange(N_BINS).reshape(-1, 1)
    n = np.arange(N_FFT).reshape(1, -1)
    ang = 2.0 * math.pi * ((k * n) % N_FFT).astype(np.float64) / N_FFT
    cos_t, sin_t = np.cos(ang), np.sin(ang)
    P = np.empty((T, N_BINS), dtype=np.float64)
    for t in range(T):
        seg = w * xp[HOP * t: HOP * t + N_FFT]
        re = cos_t @ seg
        im = -(sin_t @ seg)
        P[t] = re * re + im * im
    return P


def log_mel(x: np.ndarray, mel_fb: np.ndarray) -> np.ndarray:
    """Normalised log-mel rows of one buffer, shape [T, n_mel]:
    Mel = P F^T;  Lg = log10(max(Mel, 1e-10));  Lg = max(Lg, max(Lg) - 8) with the maximum
    taken over this buffer's frames and channels only;  A = (Lg + 4) / 4."""
    P = dft_power(x)
    F = np.asarray(mel_fb, dtype=np.float64)
    mel = P @ F.T
    lg = np.log10(np.maximum(mel, 1e-10))
    lg = np.maximum(lg, lg.max() - 8.0)
    return (lg + 4.0) / 4.0


def append_hush_mel(A: np.ndarray, hush: np.ndarray | None) -> np.ndarray:
    """x (+) h at the log-mel level: the hush rows follow the buffer's rows (Sec. 4.1.2)."""
    if hush is None or len(hush) == 0:
        return np.asarray(A, dtype=np.float64)
    return np.concatenate([np.asarray(A, np.float64), np.asarray(hush, np.float64)], axis=0)


def append_hush_audio(x: np.ndarray, hush: np.ndarray | None) -> np.ndarray:
    """x (+) h at the raw-audio level, the level the paper settles on (Sec. 4.1.2, Sec. 5)."""
    if hush is None or len(hush) == 0:
        return np.asarray(x, dtype=np.float64)
    return np.concatenate([np.asarray(x, np.float64), np.asarray(hush, np.float64)])


# --------------------------------------------------------------------------- encoder pieces

def gelu(u: np.ndarray) -> np.ndarray:
    """Exact GELU, 0.5 u (1 + erf(u / sqrt 2))."""
    return 0.5 * u * (1.0 + _erf(u / math.sqrt(2.0)))


def n_tokens(n_rows: int) -> int:
    """Tokens after the stride-2 convolution: floor((T' - 1) / 2) + 1 (3000 -> 1500)."""
    return (n_rows - 1) // 2 + 1 if n_rows > 0 else 0


def conv1d_k3(Z: np.ndarray, W: np.ndarray, b: np.ndarray, stride: int) -> np.ndarray:
    """1-D convolution over time, kernel 3, zero padding 1 on both sides of THIS sequence:
    out[p, o] = b[o] + sum_{c, j in 0..2} W[o, c, j] Z[stride p + j - 1, c], rows outside
    [0, T') read as zero.  Z is [T', C_in], W is [C_out, C_in, 3]; returns [n_out, C_out]."""
    Z = np.asarray(Z, np.float64)
    W = np.asarray(W, np.float64)
    Tp = Z.shape[0]
    n_out = (Tp - 1) // stride + 1
    out = np.tile(np.asarray(b, np.float64), (n_out, 1))
    p = np.arange(n_out)
    for j in range(3):
        r = stride * p + j - 1
        inside = (r >= 0) & (r < Tp)
        out[inside] += Z[r[inside]] @ W[:, :, j].T
    return out


def sinusoid_positions(n: int, d: int) -> np.ndarray:
    """PE[p, j] = sin(p r^j), PE[p, d/2 + j] = cos(p r^j), r = 10000^(-1/(d/2 - 1)), j < d/2."""
    half = d // 2
    inv = np.exp(-math.log(10000.0) / (half - 1) * np.arange(half, dtype=np.float64))
    ang = np.arange(n, dtype=np.float64).reshape(-1, 1) * inv.reshape(1, -1)
    return np.concatenate([np.sin(ang), np.cos(ang)], axis=1)


def layer_norm(u: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float = 1e-5) -> np.ndarray:
    """Row-wise LayerNorm with biased variance: g (u - mean) / sqrt(var + eps) + b."""
    u = np.asarray(u, np.float64)
    mu = u.mean(axis=-1, keepdims=True)
    var = ((u - mu) ** 2).mean(axis=-1, keepdims=True)
    return np.asarray(g, np.float64) * (u - mu) / np.sqrt(var + eps) + np.asarray(b, np.float64)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, n_head: int) -> np.ndarray:
    """Non-causal multi-head attention over ONE sequence's tokens: per head,
    softmax(q k^T / sqrt(d_head)) v with the row maximum subtracted before exponentiation."""
    n, d = q.shape
    dh = d // n_head
    out = np.empty((n, d), dtype=np.float64)
    for h in range(n_head):
        sl = slice(h * dh, (h + 1) * dh)
        s = (q[:, sl] @ k[:, sl].T) / math.sqrt(dh)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, sl] = p @ v[:, sl]
    return out


def _w(weights: dict, name: str) -> np.ndarray:
    return np.asarray(weights[name], dtype=np.float64)


def encoder_block(x: np.ndarray, weights: dict, l: int, n_head: int) -> np.ndarray:
    """Pre-LN transformer block: x += Wo attn(LN1 x) + bo;  x += W2 gelu(W1 LN2 x + b1) + b2.
    The key projection has no bias (a key bias shifts every logit of a row equally and
    cancels in the softmax)."""
    hN = layer_norm(x, _w(weights, f"ln1_g.{l}"), _w(weights, f"ln1_b.{l}"))
    q = hN @ _w(weights, f"wq.{l}").T + _w(weights, f"bq.{l}")
    k = hN @ _w(weights, f"wk.{l}").T
    v = hN @ _w(weights, f"wv.{l}").T + _w(weights, f"bv.{l}")
    a = attention(q, k, v, n_head)
    x = x + a @ _w(weights, f"wo.{l}").T + _w(weights, f"bo.{l}")
    h2 = layer_norm(x, _w(weights, f"ln2_g.{l}"), _w(weights, f"ln2_b.{l}"))
    m = gelu(h2 @ _w(weights, f"w1.{l}").T + _w(weights, f"b1.{l}"))
    return x + m @ _w(weights, f"w2.{l}").T + _w(weights, f"b2.{l}")


def conv_stem(Z: np.ndarray, weights: dict) -> np.ndarray:
    """gelu(conv k3 s1) then gelu(conv k3 s2), then the sinusoid table is added with the
    position index starting at 0 for this sequence."""
    c1 = gelu(conv1d_k3(Z, _w(weights, "conv1_w"), _w(weights, "conv1_b"), 1))
    c2 = gelu(conv1d_k3(c1, _w(weights, "conv2_w"), _w(weights, "conv2_b"), 2))
    return c2 + sinusoid_positions(c2.shape[0], c2.shape[1])


def encode_rows(Z: np.ndarray, weights: dict, n_layer: int, n_head: int) -> np.ndarray:
    """Encoder over one sequence given its (hush-terminated) log-mel rows Z [T', n_mel]."""
    x = conv_stem(Z, weights)
    for l in range(n_layer):
        x = encoder_block(x, weights, l, n_head)
    return layer_norm(x, _w(weights, "lnp_g"), _w(weights, "lnp_b"))


def encode_sequence(x: np.ndarray, mel_fb: np.ndarray, hush, weights: dict,
                    n_layer: int, n_head: int, hush_level: str = "mel") -> np.ndarray:
    """Final hidden states [n, d] of one buffer followed by its hush segment."""
    if hush_level == "audio":
        Z = log_mel(append_hush_audio(x, hush), mel_fb)
    elif hush_level == "mel":
        Z = append_hush_mel(log_mel(x, mel_fb), hush)
    else:
        raise ValueError(hush_level)
    return encode_rows(Z, weights, n_layer, n_head)


def encode_batch(seqs, mel_fb, hush, weights, n_layer, n_head, hush_level="mel"):
    """Ragged batch = independent sequences.  Returns (packed [sum n_i, d], cu_seqlens)."""
    outs = [encode_sequence(s, mel_fb, hush, weights, n_layer, n_head, hush_level) for s in seqs]
    cu = np.concatenate([[0], np.cumsum([o.shape[0] for o in outs])]).astype(np.int64)
    d = np.asarray(weights["lnp_g"]).shape[0]
    packed = np.concatenate(outs, axis=0) if outs else np.zeros((0, d))
    return packed, cu


def cross_kv(hidden, wk, wv, bv):
    """Cross-attention keys and values the decoder's layers read from the encoder output
    (the step right after the encoding stage, Sec. 3.2 "Operations"): for decoder layer l,
    K_l = hidden wk[l]^T (no bias) and V_l = hidden wv[l]^T + bv[l].
    hidden [n, d]; wk, wv [L, d, d] as [out, in]; bv [L, d].  Returns (K, V), each [L, n, d]."""
    h = np.asarray(hidden, dtype=np.float64)
    K = np.stack([h @ np.asarray(w, dtype=np.float64).T for w in wk])
    V = np.stack([h @ np.asarray(w, dtype=np.float64).T + np.asarray(b, dtype=np.float64) for w, b in zip(wv, bv)])
    return K, V

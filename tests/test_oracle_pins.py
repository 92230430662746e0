"""Pins for the fp64 oracle: facts the paper states, closed forms, invariants and a second,
independently written scalar evaluation.  None of these re-uses an oracle formula as its
own expected value."""
import json
import math
import os

import numpy as np
import pytest

from oracle import wf_oracle as O
from paper_2412_11272_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


# ----- shape facts printed in the paper (tests/golden/paper_shape_facts.json) ---------------

def test_paper_shape_facts():
    facts = json.load(open(os.path.join(GOLDEN, "paper_shape_facts.json")))["facts"]
    for f in facts:
        frames = O.n_frames(f["samples"]) if "samples" in f else f["frames"]
        if "frames_expected" in f:
            assert frames == f["frames_expected"], f
        if "tokens_expected" in f:
            assert O.n_tokens(frames + f.get("extra_frames", 0)) == f["tokens_expected"], f


def test_one_second_gives_100_by_80():
    x = I.synth_audio(7, 0, 16000)
    A = O.log_mel(x, I.mel_filterbank(80))
    assert A.shape == (100, 80)       # Sec. 4.1.2: 1 s of 16 kHz audio -> (100, 80)


def test_conv_stem_3000_frames_to_1500_tokens():
    rng = _rng(0)
    W1, b1 = rng.normal(size=(4, 3, 3)), rng.normal(size=4)
    W2, b2 = rng.normal(size=(4, 4, 3)), rng.normal(size=4)
    Z = rng.normal(size=(3000, 3))
    c1 = O.conv1d_k3(Z, W1, b1, 1)
    c2 = O.conv1d_k3(c1, W2, b2, 2)
    assert c1.shape == (3000, 4) and c2.shape == (1500, 4)   # Sec. 2.1: 30 s -> 1500 tokens


# ----- front end -----------------------------------------------------------------------------

def test_reflect_pad_mirror():
    x = np.arange(10, 310, dtype=np.float64)
    xp = O.reflect_pad(x)
    assert len(xp) == 300 + 400
    assert xp[200] == 10 and xp[199] == 11 and xp[0] == 210       # x[200]
    assert xp[200 + 299] == 309 and xp[200 + 300] == 308 and xp[-1] == 309 - 200


def test_hann_is_periodic():
    w = O.hann_window()
    assert w[0] == 0.0 and abs(w[200] - 1.0) < 1e-15
    assert np.allclose(w[1:], w[1:][::-1], atol=1e-15)           # w[n] = w[400 - n]
    assert abs(w.sum() - 200.0) < 1e-10                           # mean of a periodic Hann is 1/2


@pytest.mark.parametrize("k0", [5, 37, 100, 150])
def test_pure_sine_on_bin_centre_has_three_lines(k0):
    """sin(2 pi f t) with f = 40 k0 Hz: a Hann-windowed DFT has |X[k0]| = A N/4 and
    |X[k0 +- 1]| = A N/8, nothing elsewhere (interior frames only)."""
    amp = 0.7
    f = 40.0 * k0
    t = np.arange(16000)
    x = amp * np.sin(2 * math.pi * f * t / 16000 + 0.3)
    P = O.dft_power(x)
    inner = P[5:-5]
    assert np.allclose(inner[:, k0], (amp * 400 / 4) ** 2, rtol=1e-9)
    assert np.allclose(inner[:, k0 - 1], (amp * 400 / 8) ** 2, rtol=1e-9)
    assert np.allclose(inner[:, k0 + 1], (amp * 400 / 8) ** 2, rtol=1e-9)
    mask = np.ones(201, bool)
    mask[k0 - 1:k0 + 2] = False
    assert inner[:, mask].max() < 1e-18 * (amp * 100) ** 2 * 1e6
    # the arg-max mel channel is the filter whose peak frequency is nearest f
    F = I.mel_filterbank(80)
    A = O.log_mel(x, F)
    centre = np.argmax(F, axis=1) * 40.0
    assert np.argmax(A[50]) == np.argmin(np.abs(centre - f))


def test_parseval_and_dc():
    rng = _rng(3)
    x = rng.normal(size=4000)
    P = O.dft_power(x)
    xp = O.reflect_pad(x)
    w = O.hann_window()
    for t in (0, 7, 24):
        seg = w * xp[160 * t:160 * t + 400]
        full = P[t, 0] + P[t, 200] + 2 * P[t, 1:200].sum()       # conjugate-symmetric spectrum
        assert abs(full - 400 * (seg ** 2).sum()) < 1e-8 * full
    Pdc = O.dft_power(np.full(2000, 2.0))
    assert np.allclose(Pdc[:, 0], (2.0 * 200) ** 2) and np.allclose(Pdc[:, 1], (2.0 * 100) ** 2)
    assert Pdc[:, 2:].max() < 1e-18


def test_dft_matches_library_fft():
    """Special case that reduces to a library routine: numpy's real FFT of the windowed frame."""
    x = I.synth_audio(11, 2, 3200).astype(np.float64)
    P = O.dft_power(x)
    xp = np.pad(x, 200, mode="reflect")
    w = np.hanning(401)[:-1]
    for t in range(20):
        ref = np.abs(np.fft.rfft(w * xp[160 * t:160 * t + 400])) ** 2
        assert np.allclose(P[t], ref, rtol=1e-9, atol=1e-12)


def test_log_mel_range_and_silence():
    F = I.mel_filterbank(80)
    A = O.log_mel(I.synth_audio(5, 1, 8000), F)
    assert A.max() - A.min() <= 2.0 + 1e-12
    x = np.zeros(1600)
    assert np.allclose(O.log_mel(x, F), (-10.0 + 4.0) / 4.0)      # floor 1e-10 -> log10 = -10
    # scaling the audio by 10 raises every unclamped log-mel value by 2 (power x100) -> A + 0.5
    y = I.synth_audio(5, 2, 4000).astype(np.float64)
    A1, A2 = O.log_mel(y, F), O.log_mel(10 * y, F)
    assert np.allclose(A2 - A1, 0.5, atol=1e-9)
    # a loud frame clamps quiet ones: values sit at exactly (max - 8 + 4) / 4 where clamped
    z = np.concatenate([1e-7 * y[:2000], 100 * y[2000:]])
    Az = O.log_mel(z, F)
    assert np.isclose(Az.min(), Az.max() - 2.0)


def test_hush_append_levels():
    F = I.mel_filterbank(80)
    x = I.synth_audio(9, 0, 3200)
    h_mel = I.hush_mel(9, 80)
    Z = O.append_hush_mel(O.log_mel(x, F), h_mel)
    assert Z.shape == (20 + 50, 80) and np.array_equal(Z[20:], h_mel.astype(np.float64))
    # Sec. 1.2 / Sec. 5: the 0.5 s hush word is 8000 samples and costs about 25 tokens
    h_audio = I.hush_audio(9)
    xa = O.append_hush_audio(x, h_audio)
    assert len(xa) == 3200 + 8000 and O.n_tokens(O.n_frames(len(xa))) == 10 + 25
    # x (+) h: the buffer first, the hush word behind it (Sec. 4.1.2), sample for sample
    assert np.array_equal(xa[:3200], x.astype(np.float64)) and np.array_equal(xa[3200:], h_audio.astype(np.float64))
    assert not np.array_equal(xa[:8000], h_audio.astype(np.float64))
    # at the raw-audio level the junction frames mix buffer and hush samples, so the rows before the
    # junction differ from the buffer's own log-mel rows only near it (frame t reads samples
    # 160 t - 200 .. 160 t + 199) and through the shared maximum
    lone, joint = O.dft_power(x), O.dft_power(xa)
    assert np.allclose(joint[:19], lone[:19], rtol=1e-12, atol=1e-18)      # frames 0..18 end at sample 3079
    assert not np.allclose(joint[19], lone[19], rtol=1e-3)                  # frame 19 reaches into the hush word


# ----- encoder pieces ------------------------------------------------------------------------

def test_conv_identity_impulse_edges():
    rng = _rng(1)
    C = 5
    for Tp in (6, 7):
        Z = rng.normal(size=(Tp, C))
        W = np.zeros((C, C, 3))
        W[np.arange(C), np.arange(C), 1] = 1.0
        assert np.array_equal(O.conv1d_k3(Z, W, np.zeros(C), 1), Z)          # centre tap = copy
        assert np.array_equal(O.conv1d_k3(Z, W, np.zeros(C), 2), Z[0::2])    # stride 2 keeps even rows
        assert O.conv1d_k3(Z, W, np.zeros(C), 2).shape[0] == (Tp + 1) // 2
    # impulse at row 3, channel 2: output rows 2,3,4 carry taps 2,1,0 of W[:, 2, :]
    W = rng.normal(size=(4, C, 3))
    Z = np.zeros((8, C))
    Z[3, 2] = 1.0
    out = O.conv1d_k3(Z, W, np.zeros(4), 1)
    assert np.allclose(out[2], W[:, 2, 2]) and np.allclose(out[3], W[:, 2, 1])
    assert np.allclose(out[4], W[:, 2, 0]) and np.allclose(out[[0, 1, 5, 6, 7]], 0)
    # edges: first row has no left neighbour, last row no right neighbour
    Z = rng.normal(size=(5, C))
    out = O.conv1d_k3(Z, W, np.zeros(4), 1)
    assert np.allclose(out[0], W[:, :, 1] @ Z[0] + W[:, :, 2] @ Z[1])
    assert np.allclose(out[4], W[:, :, 0] @ Z[3] + W[:, :, 1] @ Z[4])
    # against a library routine: np.convolve per channel pair (correlation = convolve with flipped taps)
    b = rng.normal(size=4)
    ref = np.tile(b, (5, 1))
    for o in range(4):
        for c in range(C):
            ref[:, o] += np.convolve(Z[:, c], W[o, c, ::-1], mode="same")
    assert np.allclose(out + b, ref)


def test_gelu_identities():
    u = np.linspace(-6, 6, 241)
    g = O.gelu(u)
    assert O.gelu(np.array([0.0]))[0] == 0.0
    assert np.allclose(g - O.gelu(-u), u, atol=1e-14)
    assert abs(O.gelu(np.array([12.0]))[0] - 12.0) < 1e-12
    assert abs(O.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15   # Phi(1)
    # derivative at 0 is 1/2
    assert abs((O.gelu(np.array([1e-6]))[0] - O.gelu(np.array([-1e-6]))[0]) / 2e-6 - 0.5) < 1e-9


def test_sinusoid_table():
    pe = O.sinusoid_positions(40, 16)
    assert np.array_equal(pe[0], np.r_[np.zeros(8), np.ones(8)])
    assert np.allclose(pe[:, :8] ** 2 + pe[:, 8:] ** 2, 1.0)
    assert np.allclose(pe[:, 0], np.sin(np.arange(40)))
    assert np.allclose(pe[:, 7], np.sin(np.arange(40) / 10000.0))           # slowest channel
    assert np.allclose(pe[:, 8 + 7], np.cos(np.arange(40) / 10000.0))
    # timescales are geometric
    assert np.allclose(np.arcsin(pe[1, 1:8]) / np.arcsin(pe[1, 0:7]), 10000 ** (-1 / 7))


def test_layer_norm_invariants():
    rng = _rng(2)
    u = rng.normal(size=(9, 64)) * 3 + 1.5
    y = O.layer_norm(u, np.ones(64), np.zeros(64))
    assert np.allclose(y.mean(axis=1), 0, atol=1e-13)
    assert np.allclose(y.var(axis=1), 1.0, atol=1e-5)                         # 1 - O(eps)
    assert np.allclose(O.layer_norm(7.0 * u, np.ones(64), np.zeros(64)), y, atol=1e-5)
    g, b = rng.normal(size=64), rng.normal(size=64)
    assert np.allclose(O.layer_norm(u, g, b), g * y + b)
    # eps really is 1e-5 and the variance really is biased: a two-element row [-a, a]
    a = 1e-3
    y2 = O.layer_norm(np.array([[-a, a]]), np.ones(2), np.zeros(2))
    assert np.allclose(y2, np.array([[-a, a]]) / math.sqrt(a * a + 1e-5))


def test_attention_closed_forms():
    rng = _rng(4)
    n, H, dh = 11, 2, 4
    d = H * dh
    q = rng.normal(size=(n, d))
    v = rng.normal(size=(n, d))
    k_same = np.tile(rng.normal(size=(1, d)), (n, 1))
    assert np.allclose(O.attention(q, k_same, v, H), np.tile(v.mean(axis=0), (n, 1)))
    # one key with a dominant logit: returns that key's value
    k = rng.normal(size=(n, d)) * 1e-3
    q1 = np.tile(np.r_[np.ones(dh), np.ones(dh)] * 50.0, (n, 1))
    k[6] = 50.0
    assert np.allclose(O.attention(q1, k, v, H), np.tile(v[6], (n, 1)), atol=1e-12)
    # n = 1 returns v
    assert np.allclose(O.attention(q[:1], k[:1], v[:1], H), v[:1])
    # key bias cancels
    k2 = rng.normal(size=(n, d))
    bias = rng.normal(size=d)
    assert np.allclose(O.attention(q, k2 + bias, v, H), O.attention(q, k2, v, H), atol=1e-12)
    # scale is 1/sqrt(d_head): two keys, logits differ by q.(k0-k1)/sqrt(dh)
    qq = np.zeros((1, dh)); qq[0, 0] = 2.0
    kk = np.zeros((2, dh)); kk[0, 0] = 1.0
    vv = np.array([[1.0] + [0] * (dh - 1), [0.0] * dh])
    out = O.attention(qq, kk, vv, 1)
    assert abs(out[0, 0] - 1.0 / (1.0 + math.exp(-2.0 / math.sqrt(dh)))) < 1e-14
    # heads are independent: changing head 1's q/k/v leaves head 0's output alone
    q3, k3, v3 = q.copy(), k2.copy(), v.copy()
    q3[:, dh:] += 1.0; k3[:, dh:] *= 2.0; v3[:, dh:] -= 1.0
    assert np.array_equal(O.attention(q3, k3, v3, H)[:, :dh], O.attention(q, k2, v, H)[:, :dh])


def _tiny_shape(**kw):
    base = dict(name="t", n_mel=4, d_model=8, n_layer=1, n_head=2, d_mlp=16, dtype="f32",
                n_ctx=64, hush_frames=3)
    base.update(kw)
    return I.EncoderShape(**base)


def test_residual_wiring_with_zero_weights():
    shape = _tiny_shape(n_layer=2)
    W = I.encoder_weights(3, shape, bf16=False)
    W = {k: v.astype(np.float64) * 10 for k, v in W.items()}
    rng = _rng(5)
    Z = rng.normal(size=(9, 4))
    stem = O.conv_stem(Z, W)
    ref = O.layer_norm(stem, W["lnp_g"], W["lnp_b"])
    W0 = dict(W)
    for l in range(2):
        W0[f"wo.{l}"] = np.zeros_like(W[f"wo.{l}"]); W0[f"bo.{l}"] = np.zeros(8)
        W0[f"w2.{l}"] = np.zeros_like(W[f"w2.{l}"]); W0[f"b2.{l}"] = np.zeros(8)
    assert np.allclose(O.encode_rows(Z, W0, 2, 2), ref, atol=1e-14)
    assert not np.allclose(O.encode_rows(Z, W, 2, 2), ref, atol=1e-3)


def test_block_is_permutation_equivariant():
    shape = _tiny_shape()
    W = {k: v.astype(np.float64) * 20 for k, v in I.encoder_weights(4, shape, bf16=False).items()}
    x = _rng(6).normal(size=(7, 8))
    perm = np.array([3, 0, 6, 1, 5, 2, 4])
    assert np.allclose(O.encoder_block(x[perm], W, 0, 2), O.encoder_block(x, W, 0, 2)[perm], atol=1e-13)


def test_batch_invariance():
    shape = _tiny_shape(n_mel=8, d_model=16, d_mlp=32)
    W = I.encoder_weights(5, shape, bf16=False)
    F = I.mel_filterbank(8)
    hush = I.hush_mel(5, 8, 3)
    seqs = [I.synth_audio(5, i, n) for i, n in enumerate((800, 1120, 480))]
    packed, cu = O.encode_batch(seqs, F, hush, W, 1, 2)
    assert list(cu) == [0, 4, 9, 12]
    for order in ([2, 0, 1], [1], [0, 2]):
        p2, cu2 = O.encode_batch([seqs[i] for i in order], F, hush, W, 1, 2)
        for j, i in enumerate(order):
            assert np.array_equal(p2[cu2[j]:cu2[j + 1]], packed[cu[i]:cu[i + 1]])


# ----- second, independent scalar evaluation of the whole path on tiny dims ------------------

def _scalar_encode(x, F, hush, W, n_layer, n_head, hush_audio=None):
    """Pure-Python scalar evaluation in a different loop order (output-element outer loops,
    math.fsum reductions, Python complex exponentials).  ``hush`` is the log-mel-level hush
    segment (rows appended after the normalisation); ``hush_audio`` the raw-audio-level one:
    its samples follow the buffer's, read through index arithmetic (no concatenated copy), and
    the framing, the maximum and the clamp then run over the whole of x (+) h."""
    Lx = len(x)
    L = Lx + (len(hush_audio) if hush_audio is not None else 0)
    T = L // 160

    def xs(i):                       # reflected sample of x (+) h
        if i < 0:
            i = -i
        if i >= L:
            i = 2 * L - 2 - i
        return float(x[i]) if i < Lx else float(hush_audio[i - Lx])

    n_mel = len(F)
    lg = [[0.0] * n_mel for _ in range(T)]
    for t in range(T):
        power = []
        for k in range(201):
            acc = 0j
            for n in range(400):
                wn = 0.5 * (1.0 - math.cos(2 * math.pi * n / 400))
                acc += wn * xs(160 * t + n - 200) * complex(math.cos(2 * math.pi * k * n / 400),
                                                            -math.sin(2 * math.pi * k * n / 400))
            power.append(acc.real ** 2 + acc.imag ** 2)
        for m in range(n_mel):
            lg[t][m] = math.log10(max(math.fsum(float(F[m][k]) * power[k] for k in range(201)), 1e-10))
    mx = max(max(r) for r in lg)
    Z = [[(max(v, mx - 8.0) + 4.0) / 4.0 for v in r] for r in lg]
    if hush is not None:
        Z = Z + [[float(v) for v in r] for r in hush]

    def gelu(u):
        return 0.5 * u * (1.0 + math.erf(u / math.sqrt(2.0)))

    def conv(inp, w, b, stride):
        rows, cin, cout = len(inp), len(inp[0]), len(b)
        n_out = (rows + stride - 1) // stride
        out = []
        for p in range(n_out):
            row = []
            for o in range(cout):
                terms = [float(b[o])]
                for c in range(cin):
                    for j in range(3):
                        r = stride * p + j - 1
                        if 0 <= r < rows:
                            terms.append(float(w[o][c][j]) * inp[r][c])
                row.append(gelu(math.fsum(terms)))
            out.append(row)
        return out

    c2 = conv(conv(Z, W["conv1_w"], W["conv1_b"], 1), W["conv2_w"], W["conv2_b"], 2)
    n, d = len(c2), len(c2[0])
    half = d // 2
    xr = [[c2[p][c] + (math.sin(p * 10000.0 ** (-(c) / (half - 1))) if c < half
                       else math.cos(p * 10000.0 ** (-(c - half) / (half - 1))))
           for c in range(d)] for p in range(n)]

    def ln(rows, g, b):
        out = []
        for r in rows:
            mu = math.fsum(r) / len(r)
            var = math.fsum((v - mu) ** 2 for v in r) / len(r)
            out.append([float(g[i]) * (r[i] - mu) / math.sqrt(var + 1e-5) + float(b[i]) for i in range(len(r))])
        return out

    def lin(rows, w, b=None):
        return [[math.fsum(float(w[o][i]) * r[i] for i in range(len(r))) + (float(b[o]) if b is not None else 0.0)
                 for o in range(len(w))] for r in rows]

    dh = d // n_head
    for l in range(n_layer):
        hN = ln(xr, W[f"ln1_g.{l}"], W[f"ln1_b.{l}"])
        q, k, v = lin(hN, W[f"wq.{l}"], W[f"bq.{l}"]), lin(hN, W[f"wk.{l}"]), lin(hN, W[f"wv.{l}"], W[f"bv.{l}"])
        att = [[0.0] * d for _ in range(n)]
        for a in range(n):
            for h in range(n_head):
                logit = [math.fsum(q[a][h * dh + e] * k[b_][h * dh + e] for e in range(dh)) / math.sqrt(dh)
                         for b_ in range(n)]
                z = math.fsum(math.exp(s) for s in logit)       # no max subtraction: tiny logits
                for e in range(dh):
                    att[a][h * dh + e] = math.fsum(math.exp(logit[b_]) / z * v[b_][h * dh + e] for b_ in range(n))
        proj = lin(att, W[f"wo.{l}"], W[f"bo.{l}"])
        xr = [[xr[p][c] + proj[p][c] for c in range(d)] for p in range(n)]
        h2 = ln(xr, W[f"ln2_g.{l}"], W[f"ln2_b.{l}"])
        m = [[gelu(u) for u in r] for r in lin(h2, W[f"w1.{l}"], W[f"b1.{l}"])]
        m2 = lin(m, W[f"w2.{l}"], W[f"b2.{l}"])
        xr = [[xr[p][c] + m2[p][c] for c in range(d)] for p in range(n)]
    return np.array(ln(xr, W["lnp_g"], W["lnp_b"]))


@pytest.mark.parametrize("n_samples", [480, 640])          # T' = 6 (even) and 7 (odd)
def test_whole_path_against_scalar_evaluation(n_samples):
    shape = _tiny_shape()
    W = {k: v.astype(np.float64) * 15 for k, v in I.encoder_weights(8, shape, bf16=False).items()}
    F = I.mel_filterbank(4)
    hush = I.hush_mel(8, 4, 3)
    x = I.synth_audio(8, 0, n_samples)
    got = O.encode_sequence(x, F, hush, W, 1, 2)
    ref = _scalar_encode(x, F, hush, W, 1, 2)
    assert got.shape == ref.shape == ((n_samples // 160 + 3 + 1) // 2, 8)
    assert np.max(np.abs(got - ref)) < 1e-10


@pytest.mark.parametrize("n_samples,n_hush", [(480, 480), (640, 410)])      # T = 6 and 6 (1050 // 160): junction mid-frame
def test_whole_path_raw_audio_hush_against_scalar_evaluation(n_samples, n_hush):
    """The raw-audio-level variant (Sec. 4.1.2): hush samples behind the buffer's, everything
    downstream over x (+) h.  A hush word put in front, framed separately, or left out of the
    maximum would each move the result."""
    shape = _tiny_shape()
    W = {k: v.astype(np.float64) * 15 for k, v in I.encoder_weights(8, shape, bf16=False).items()}
    F = I.mel_filterbank(4)
    x = I.synth_audio(8, 0, n_samples)
    h = 3.0 * I.hush_audio(8, n_hush)                   # louder than the buffer: the maximum sits in the hush part
    got = O.encode_sequence(x, F, h, W, 1, 2, hush_level="audio")
    ref = _scalar_encode(x, F, None, W, 1, 2, hush_audio=h)
    assert got.shape == ref.shape == (((n_samples + n_hush) // 160 + 1) // 2, 8)
    assert np.max(np.abs(got - ref)) < 1e-10
    swapped = O.encode_sequence(h, F, x, W, 1, 2, hush_level="audio")
    assert np.max(np.abs(swapped - ref)) > 1e-3


# ----- planted mistakes: each pin set must catch a plausible slip ----------------------------

def test_pins_catch_planted_mistakes(monkeypatch):
    x = 0.7 * np.sin(2 * math.pi * 40.0 * 37 * np.arange(16000) / 16000)
    good = O.dft_power(x)[20, 37]
    # symmetric (non-periodic) Hann would move the line amplitude
    monkeypatch.setattr(O, "hann_window", lambda n=400: np.hanning(n))
    assert not np.isclose(O.dft_power(x)[20, 37], good, rtol=1e-6)
    monkeypatch.undo()
    # transposed conv taps fail the impulse pin
    W = _rng(1).normal(size=(4, 5, 3))
    Z = np.zeros((8, 5)); Z[3, 2] = 1.0
    out = O.conv1d_k3(Z, W[:, :, ::-1], np.zeros(4), 1)
    assert not np.allclose(out[2], W[:, 2, 2])


# ----- measurement sanity: hush vs 30 s padding (Sec. 2.2 and Sec. 6.3 quote 3-3.7x) ---------

def test_cross_kv_hand_worked_and_linear():
    """cross_kv against values worked by hand (a transposed weight, a bias on the keys or a
    missing bias on the values would each change them) and against linearity."""
    h = np.array([[1.0, 2.0], [0.0, -1.0], [3.0, 0.5]])
    wk = np.array([[[1.0, 0.0], [2.0, -1.0]], [[0.0, 1.0], [1.0, 1.0]]])          # [L=2, out, in]
    wv = np.array([[[0.5, 0.5], [0.0, 2.0]], [[-1.0, 0.0], [0.0, 0.0]]])
    bv = np.array([[10.0, 20.0], [0.0, -5.0]])
    K, V = O.cross_kv(h, wk, wv, bv)
    assert K.shape == V.shape == (2, 3, 2)
    # K_0[t] = (h0, 2 h0 - h1);  K_1[t] = (h1, h0 + h1)
    assert np.array_equal(K[0], [[1.0, 0.0], [0.0, 1.0], [3.0, 5.5]])
    assert np.array_equal(K[1], [[2.0, 3.0], [-1.0, -1.0], [0.5, 3.5]])
    # V_0[t] = ((h0 + h1)/2 + 10, 2 h1 + 20);  V_1[t] = (-h0, -5)
    assert np.array_equal(V[0], [[11.5, 24.0], [9.5, 18.0], [11.75, 21.0]])
    assert np.array_equal(V[1], [[-1.0, -5.0], [0.0, -5.0], [-3.0, -5.0]])
    K0, V0 = O.cross_kv(np.zeros_like(h), wk, wv, bv)                              # keys carry no bias
    assert np.all(K0 == 0.0) and np.array_equal(V0[0], np.tile(bv[0], (3, 1)))
    K2, V2 = O.cross_kv(2.0 * h, wk, wv, bv)
    assert np.allclose(K2, 2.0 * K) and np.allclose(V2 - V0, 2.0 * (V - V0))


def test_padding_vs_hush_flop_ratio():
    shape = I.SHAPES["medium"]
    clips = I.uniform_lengths(3, 256, 5, 25)                # the paper's clip lengths, 5-25 s
    padded = I.algorithmic_flops(shape, np.full(256, 30 * 16000), hush_frames=0)["encoder"]
    hushed = I.algorithmic_flops(shape, clips)["encoder"]
    assert 1.8 < padded / hushed < 3.7
    n = I.tokens_of(clips)
    assert padded / hushed > 1500.0 * 256 / n.sum()         # attention makes it super-linear

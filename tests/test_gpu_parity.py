"""GPU parity: the CUDA library, called through its C ABI, against the fp64 oracle on the same
seeded inputs.  Tolerances: float32 path max-abs <= 1e-3 on final hidden states; bf16 path
max|err| / max|ref| <= 3e-2 per sequence and per-token cosine >= 0.999."""
import math

import numpy as np
import pytest

from oracle import wf_oracle as O
from paper_2412_11272_b200 import inputs as I
from tests._util import elementwise_excess, make_encoder, min_token_cosine, oracle_hidden, peak_rel_err, to_np

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

F32_TOL = 1e-3
BF16_REL, BF16_COS = 3e-2, 0.999
MEL_TOL = 2e-4   # normalised log-mel units; float32 DFT of 400 terms under a log10


def _dev(a, dtype=torch.float32):
    return torch.as_tensor(np.ascontiguousarray(a)).to("cuda:0", dtype)


def _small(dtype, **kw):
    base = dict(name="s", n_mel=80, d_model=128, n_layer=2, n_head=2, d_mlp=256, dtype=dtype, n_ctx=1536)
    base.update(kw)
    return I.EncoderShape(**base)


# ------------------------------------------------------------------------------ front end

def test_logmel_matches_oracle_ragged():
    shape = _small("f32", n_layer=0)
    W = I.encoder_weights(0, shape)
    lengths = [32000, 401, 160 * 64, 160 * 65 + 37, 160 * 129 + 159, 5000]
    batch = I.batch_from_lengths(11, lengths)
    enc = make_encoder(shape, W, 8, 4096, int(sum(lengths)))
    mel, frames = enc.wf_logmel(_dev(batch.audio), batch.lengths)
    torch.cuda.synchronize()
    assert list(frames) == [n // 160 for n in lengths]
    got = to_np(mel)
    F = I.mel_filterbank(80)
    off = 0
    for s in batch.sequences():
        ref = O.log_mel(s, F)
        g = got[off:off + ref.shape[0]]
        off += ref.shape[0]
        assert np.max(np.abs(g - ref)) < MEL_TOL
    assert off == got.shape[0]
    enc.close()


def test_logmel_pure_sine_and_silence():
    shape = _small("f32", n_layer=0)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 2, 1024, 40000)
    t = np.arange(16000)
    sine = (0.5 * np.sin(2 * math.pi * 1000.0 * t / 16000)).astype(np.float32)
    silence = np.zeros(8000, np.float32)
    mel, _ = enc.wf_logmel(_dev(np.concatenate([sine, silence])), [16000, 8000])
    got = to_np(mel)
    F = I.mel_filterbank(80)
    centre = np.argmax(F, axis=1) * 40.0
    assert np.argmax(got[50]) == np.argmin(np.abs(centre - 1000.0))
    assert np.allclose(got[100:], -1.5, atol=1e-6)          # (log10(1e-10) + 4) / 4
    enc.close()


# ------------------------------------------------------------------------------ float32 path

def test_f32_tiny_config_matches_oracle():
    """The smallest configuration: tiny-shaped float32 encoder, one 2.0 s buffer + 50 hush frames."""
    shape = I.SHAPES["tiny"]
    W = I.encoder_weights(0, shape)
    batch = I.config_batch("tiny")
    hush = I.hush_mel(0, shape.n_mel)
    enc = make_encoder(shape, W, 1, 125, 32000)
    out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    assert list(cu) == [0, 125] and out.shape == (125, 384) and out.dtype == torch.float32
    ref = oracle_hidden(batch, shape, W, hush)[0]
    assert np.max(np.abs(to_np(out) - ref)) <= F32_TOL
    enc.close()


def test_f32_ragged_batch_odd_even_and_invariance():
    shape = _small("f32")
    W = I.encoder_weights(3, shape, logit_gain=12.0)
    lengths = [160 * 7, 160 * 10, 401, 160 * 131, 160 * 64 + 5]      # T' odd and even, tiny, multi-tile
    batch = I.batch_from_lengths(5, lengths)
    hush = I.hush_mel(5, shape.n_mel, 3)
    enc = make_encoder(shape, W, 8, 512, int(sum(lengths)), hush_frames=3)
    out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    got = to_np(out)
    F = I.mel_filterbank(shape.n_mel)
    refs = [O.encode_sequence(s, F, hush, W, shape.n_layer, shape.n_head) for s in batch.sequences()]
    assert list(cu) == list(np.concatenate([[0], np.cumsum([r.shape[0] for r in refs])]))
    for i, r in enumerate(refs):
        assert np.max(np.abs(got[cu[i]:cu[i + 1]] - r)) <= F32_TOL, i
    # batch invariance: a sequence alone, or in another order, gives the same rows
    order = [3, 0, 4]
    b2 = I.Batch(np.concatenate([batch.sequences()[i] for i in order]), batch.lengths[order])
    out2, cu2 = enc.wf_encode(_dev(b2.audio), b2.lengths, _dev(hush))
    g2 = to_np(out2)
    for j, i in enumerate(order):
        assert np.max(np.abs(g2[cu2[j]:cu2[j + 1]] - got[cu[i]:cu[i + 1]])) <= 1e-5
    enc.close()


def test_encode_mel_entry_and_raw_audio_level_hush():
    """The paper attaches the hush word at raw-audio level: the caller concatenates samples and
    runs with hush_frames = 0; wf_encode_mel consumes rows made by wf_logmel."""
    shape = _small("f32")
    W = I.encoder_weights(4, shape)
    x = I.synth_audio(6, 0, 160 * 40)
    h = I.hush_audio(6)
    xa = np.concatenate([x, h]).astype(np.float32)
    enc = make_encoder(shape, W, 2, 256, len(xa), hush_frames=0)
    out, cu = enc.wf_encode(_dev(xa), [len(xa)], None)
    ref = O.encode_sequence(x, I.mel_filterbank(80), h, W, shape.n_layer, shape.n_head, hush_level="audio")
    assert list(cu) == [0, 45] and np.max(np.abs(to_np(out) - ref)) <= F32_TOL
    mel, frames = enc.wf_logmel(_dev(xa), [len(xa)])
    out2, _ = enc.wf_encode_mel(mel, frames, None)
    assert np.max(np.abs(to_np(out2) - to_np(out))) <= 1e-6
    enc.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_raw_audio_level_hush_fused_in_front_end(dtype):
    """wf_encode_raw_hush reads the hush samples in place (no concatenated copy) and must equal the
    oracle's raw-audio-level variant, including frames that straddle the junction."""
    shape = _small(dtype, d_model=256, n_head=4, d_mlp=512)
    W = I.encoder_weights(12, shape)
    lengths = [160 * 40, 160 * 7 + 93, 401, 160 * 130 + 159]        # junctions on and off the frame grid
    batch = I.batch_from_lengths(13, lengths)
    h = I.hush_audio(13)                                             # 8000 samples
    enc = make_encoder(shape, W, 4, 512, int(sum(lengths)), hush_frames=0)
    out, cu = enc.wf_encode_raw_hush(_dev(batch.audio), batch.lengths, _dev(h))
    enc.wf_check()
    got = to_np(out)
    F = I.mel_filterbank(80)
    assert list(np.diff(cu)) == [((n + 8000) // 160 + 1) // 2 for n in lengths]
    for i, x in enumerate(batch.sequences()):
        ref = O.encode_sequence(x, F, h, W, shape.n_layer, shape.n_head, hush_level="audio")
        g = got[cu[i]:cu[i + 1]]
        if dtype == "f32":
            assert np.max(np.abs(g - ref)) <= F32_TOL, i
        else:
            _check_bf16(g, ref)
    # the fused path equals running on caller-concatenated samples
    cat = np.concatenate([np.concatenate([x, h]) for x in batch.sequences()]).astype(np.float32)
    out2, cu2 = enc2_encode(shape, W, cat, [n + 8000 for n in lengths])
    assert list(cu2) == list(cu) and np.max(np.abs(to_np(out2) - got)) <= (1e-5 if dtype == "f32" else 2e-2)
    enc.close()


def enc2_encode(shape, W, audio, lengths):
    enc = make_encoder(shape, W, len(lengths), 1024, int(sum(lengths)), hush_frames=0)
    out, cu = enc.wf_encode(_dev(audio), lengths, None)
    enc.wf_check()
    res = (out.clone(), cu)
    enc.close()
    return res


# ------------------------------------------------------------------------------ bf16 components

@pytest.mark.parametrize("M,N,K", [(300, 384, 240), (1000, 1536, 512), (129, 256, 64), (4097, 1280, 1280),
                                   (77, 8, 8), (75, 5120, 1280), (200, 1000, 1024)])   # the last two: K split over a cluster
@pytest.mark.parametrize("mode", [0, 1])
def test_tcgen05_gemm_matches_fp64(M, N, K, mode):
    shape = _small("bf16", n_layer=0)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 1, 64, 1000)
    rng = np.random.default_rng(M + N + K + mode)
    A = I.round_to_bf16(rng.normal(size=(M, K)).astype(np.float32))
    Wm = I.round_to_bf16((rng.normal(size=(N, K)) / math.sqrt(K)).astype(np.float32))
    bias = rng.normal(size=N).astype(np.float32)
    ref = A.astype(np.float64) @ Wm.astype(np.float64).T + bias
    dA, dW, db = _dev(A, torch.bfloat16), _dev(Wm, torch.bfloat16), _dev(bias)
    if mode == 1:
        ref = O.gelu(ref)
    C = enc.wf_gemm_bf16(dA, dW, db, mode)
    enc.wf_check()
    got = to_np(C)
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1.0)) < 2.0 ** -8     # bf16 output rounding
    enc.close()


def _split_planes(x):
    """x float32 -> (hi, lo) bf16 CUDA tensors with hi = bf16(x), lo = bf16(x - hi), and hi + lo in float64."""
    xt = _dev(x)
    hi = xt.to(torch.bfloat16)
    lo = (xt - hi.float()).to(torch.bfloat16)
    return hi, lo, hi.double().cpu().numpy() + lo.double().cpu().numpy()


@pytest.fixture(autouse=True)
def _split_every_small_gemm(monkeypatch):
    """Encoders created by the tests of this file split the K range of small GEMMs from 8 K blocks on
    (the library's default is 64), so that the cluster split is exercised on all three kinds of epilogue."""
    monkeypatch.setenv("WF_GEMM_SPLIT_K", "8")


def _row_stats(x64):
    """[K / 128, M, 2] float32 partial (sum, sum of squares) of every 128 columns."""
    M, K = x64.shape
    parts = x64.reshape(M, K // 128, 128)
    return _dev(np.stack([parts.sum(-1).T, (parts ** 2).sum(-1).T], axis=-1).astype(np.float32))


@pytest.mark.parametrize("M,N,K", [(300, 384, 240), (1000, 1536, 512), (129, 256, 64), (4097, 1280, 1280),
                                   (77, 128, 8), (60, 1280, 5120), (775, 1280, 5120), (775, 1280, 1280)])   # the last three: K split over a cluster of 4 / 2 / 2
def test_tcgen05_residual_gemm_on_split_stream(M, N, K):
    """x <- x + A W^T + bias with x held as two bf16 planes (16 significant bits), and the row
    statistics the epilogue leaves for the LayerNorm that follows."""
    shape = _small("bf16", n_layer=0)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 1, 64, 1000)
    rng = np.random.default_rng(M + N + K)
    A = I.round_to_bf16(rng.normal(size=(M, K)).astype(np.float32))
    Wm = I.round_to_bf16((rng.normal(size=(N, K)) / math.sqrt(K)).astype(np.float32))
    bias = rng.normal(size=N).astype(np.float32)
    hi, lo, x0 = _split_planes((3.0 * rng.normal(size=(M, N)) + 0.5).astype(np.float32))
    ref = x0 + A.astype(np.float64) @ Wm.astype(np.float64).T + bias
    stats = enc.wf_gemm_resid_bf16(_dev(A, torch.bfloat16), _dev(Wm, torch.bfloat16), _dev(bias), hi, lo)
    enc.wf_check()
    got = hi.double().cpu().numpy() + lo.double().cpu().numpy()
    assert float(np.max(np.abs(got - ref) - 2.0 ** -16 * np.abs(ref))) <= 2e-5 * math.sqrt(K) + 1e-5
    hi64, lo64 = hi.double().cpu().numpy(), lo.double().cpu().numpy()
    assert float(np.max(np.abs(lo64) - 2.0 ** -8 * np.abs(hi64))) <= 0.0       # lo is the rounding remainder of hi
    st = stats.cpu().numpy().astype(np.float64)
    parts = got.reshape(M, N // 128, 128)
    assert np.max(np.abs(st[..., 0] - parts.sum(-1).T)) < 1e-5 * np.abs(parts).sum(-1).max()
    assert np.max(np.abs(st[..., 1] / (parts ** 2).sum(-1).T - 1.0)) < 1e-5
    enc.close()


@pytest.mark.parametrize("M,N,K", [(300, 384, 256), (1000, 1536, 512), (129, 256, 128), (4097, 3840, 1280), (77, 8, 128),
                                   (100, 3840, 1280), (275, 1280, 1024)])   # the last two: K split over a cluster
@pytest.mark.parametrize("gelu", [False, True])
def test_tcgen05_gemm_with_folded_layernorm(M, N, K, gelu):
    """(gelu of) LN(x) W^T + bias computed as rstd (x_hi W'^T - mean s) + c from the bf16 upper plane
    of x, the row statistics and the folded weights: tightly against the same formula evaluated in
    float64 with the library's folded weights, and against the definition on the unrounded x."""
    shape = _small("bf16", n_layer=0)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 1, 64, 1000)
    rng = np.random.default_rng(M + N + K + 7)
    # rows of different scale, each with a common mode of the order of its spread (the bf16 rounding of x
    # is relative to |x|, so a common mode far above the spread would cost accuracy in proportion)
    x = ((rng.normal(size=(M, K)) + 0.5 * rng.normal(size=(M, 1))) * rng.uniform(0.5, 4.0, size=(M, 1))).astype(np.float32)
    hi, lo, x64 = _split_planes(x)
    Wm = I.round_to_bf16((rng.normal(size=(N, K)) / math.sqrt(K)).astype(np.float32))
    g = (1.0 + 0.2 * rng.normal(size=K)).astype(np.float32)
    b = (0.2 * rng.normal(size=K)).astype(np.float32)
    bias = rng.normal(size=N).astype(np.float32)
    Wg, colsum, cbias = enc.wf_ln_fold(_dev(Wm), _dev(g), _dev(b), _dev(bias))
    Wg64 = Wg.double().cpu().numpy()
    assert np.array_equal(Wg.float().cpu().numpy(), I.round_to_bf16((Wm * g[None, :]).astype(np.float32)))
    assert np.max(np.abs(colsum.cpu().numpy() - Wg64.sum(1))) < 1e-5 * np.abs(Wg64).sum(1).max()
    assert np.max(np.abs(cbias.cpu().numpy() - (bias + Wm.astype(np.float64) @ b))) < 1e-5
    out = to_np(enc.wf_gemm_ln_bf16(hi, _row_stats(x64), Wg, colsum, cbias, gelu))
    enc.wf_check()
    mu = x64.mean(1, keepdims=True)
    rstd = 1.0 / np.sqrt(x64.var(1, keepdims=True) + 1e-5)
    same = rstd * (hi.double().cpu().numpy() @ Wg64.T - mu * Wg64.sum(1)[None, :]) + (bias + Wm.astype(np.float64) @ b)[None, :]
    ref = O.layer_norm(x64, g, b) @ Wm.astype(np.float64).T + bias
    if gelu:
        same, ref = O.gelu(same), O.gelu(ref)
    assert np.max(np.abs(out - same) / (np.abs(same) + 1.0)) < 2.0 ** -8 + 1e-3      # bf16 output rounding (+ GELU form)
    assert np.max(np.abs(out - ref) / (np.abs(ref) + 1.0)) < 2.5e-2                   # + bf16 rounding of x and of W gamma
    enc.close()


def test_gelu_epilogue_pointwise():
    """The GELU of the bf16 GEMM epilogue on a grid of arguments (fed through a one-hot GEMM so that
    the accumulator is the argument itself) against the oracle's erf form: within bf16 rounding of
    the result plus 1e-3 over [-12, 12], the negative tail included."""
    shape = _small("bf16", n_layer=0)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 1, 64, 1000)
    x = I.round_to_bf16(np.concatenate([np.linspace(-12.0, 12.0, 4001), np.linspace(-1.0, 1.0, 2001)]).astype(np.float32))
    A = np.zeros((len(x), 8), np.float32)
    A[:, 0] = x
    Wm = np.zeros((8, 8), np.float32)
    Wm[:, 0] = 1.0
    out = to_np(enc.wf_gemm_bf16(_dev(A, torch.bfloat16), _dev(Wm, torch.bfloat16), _dev(np.zeros(8, np.float32)), 1))
    enc.wf_check()
    ref = O.gelu(x.astype(np.float64))
    err = np.abs(out[:, 3] - ref)
    assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 1e-3), float(np.max(err - 2.0 ** -8 * np.abs(ref)))
    enc.close()


@pytest.mark.parametrize("mode", [0, 2])
def test_tcgen05_gemm_ragged_last_tile_repeated(mode):
    """M leaves whole 32-row groups of the last tile outside the matrix and N leaves 64-column
    pieces outside: the epilogue warps that own them store nothing there, and must still not
    reuse a staging buffer that the previous tile's last copy is reading (mode 0: plain bf16
    output; mode 2: the residual update on the split stream, which also fetches through those
    buffers).  That is a race, so the launch is repeated; every repetition is compared in full
    (on the device)."""
    shape = _small("bf16", n_layer=0)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 1, 64, 1000)
    M, N, K = 20000, (1184 if mode == 0 else 1152), 640
    rng = np.random.default_rng(5)
    A = I.round_to_bf16(rng.normal(size=(M, K)).astype(np.float32))
    Wm = I.round_to_bf16((rng.normal(size=(N, K)) / math.sqrt(K)).astype(np.float32))
    bias = rng.normal(size=N).astype(np.float32)
    hi0, lo0, x0 = _split_planes(rng.normal(size=(M, N)).astype(np.float32))
    ref = A.astype(np.float64) @ Wm.astype(np.float64).T + bias + (x0 if mode == 2 else 0.0)
    d_ref = _dev(ref.astype(np.float32))
    dA, dW, db = _dev(A, torch.bfloat16), _dev(Wm, torch.bfloat16), _dev(bias)
    worst, first = 0.0, None
    for _ in range(25):
        if mode == 2:
            hi, lo = hi0.clone(), lo0.clone()
            stats = enc.wf_gemm_resid_bf16(dA, dW, db, hi, lo)
            err = (hi.float() + lo.float() - d_ref).abs()
            if first is None:
                first = (hi, lo, stats)
            else:   # no atomics anywhere: every repetition reproduces every bit
                assert torch.equal(hi, first[0]) and torch.equal(lo, first[1]) and torch.equal(stats, first[2])
        else:
            err = (enc.wf_gemm_bf16(dA, dW, db, 0).float() - d_ref).abs()
        worst = max(worst, float((err / (d_ref.abs() + 1.0)).max()) if mode == 0 else float(err.max()))
    enc.wf_check()
    assert worst < (2.0 ** -8 if mode == 0 else 2e-5 * math.sqrt(K) + 1e-5 + 2.0 ** -14), worst
    enc.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_cross_kv_projection_matches_oracle(dtype):
    """Encoder output -> cross-attention keys/values of every decoder layer (one GEMM)."""
    bf16 = dtype == "bf16"
    shape = _small(dtype, n_layer=0, d_model=256 if bf16 else 128, n_head=4 if bf16 else 2, d_mlp=256)
    d, L, M = shape.d_model, 3, 333                                   # ragged against the 128/256-row tiles
    enc = make_encoder(shape, I.encoder_weights(0, shape), 1, 64, 1000)
    Wc = I.cross_kv_weights(11, d, L, bf16)
    hidden = I.normal01(11, 6_100_000, M * d).astype(np.float32).reshape(M, d)
    if bf16:
        hidden = I.round_to_bf16(hidden)
    K, V = O.cross_kv(hidden, Wc["wk"], Wc["wv"], Wc["bv"])
    W_kv = np.concatenate([np.concatenate([Wc["wk"][l], Wc["wv"][l]]) for l in range(L)])      # [L * 2d, d]
    b_kv = np.concatenate([np.concatenate([np.zeros(d, np.float32), Wc["bv"][l]]) for l in range(L)])
    tdt = torch.bfloat16 if bf16 else torch.float32
    kv = to_np(enc.wf_cross_kv(_dev(hidden, tdt), _dev(W_kv, tdt), _dev(b_kv)))
    enc.wf_check()
    assert kv.shape == (M, L * 2 * d)
    for l in range(L):
        for got, ref in ((kv[:, 2 * l * d:2 * l * d + d], K[l]), (kv[:, 2 * l * d + d:2 * (l + 1) * d], V[l])):
            err = np.max(np.abs(got - ref))
            assert err < (2.0 ** -8 * (np.max(np.abs(ref)) + 1e-3) if bf16 else 1e-5), (l, err)
    assert enc.wf_cross_kv(_dev(hidden[:0], tdt), _dev(W_kv, tdt), _dev(b_kv)).shape[0] == 0   # empty
    enc.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_varlen_attention_matches_oracle(dtype):
    shape = _small(dtype, n_layer=0, d_model=256, n_head=4, d_mlp=256)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 8, 4096, 1000)
    lens = [1, 63, 64, 65, 200, 1525, 17]
    cu = np.concatenate([[0], np.cumsum(lens)])
    rng = np.random.default_rng(9)
    qkv = rng.normal(size=(cu[-1], 3 * 256)).astype(np.float32)
    qkv[:, :256] *= 3.0                                     # logits with std ~ 3: softmax far from uniform
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    if dtype == "bf16":
        qkv = I.round_to_bf16(qkv)
    out = to_np(enc.wf_attention(_dev(qkv, tdt), cu))
    enc.wf_check()
    q64 = qkv.astype(np.float64)
    tol = 2e-2 if dtype == "bf16" else 1e-5
    for i in range(len(lens)):
        s = slice(cu[i], cu[i + 1])
        ref = O.attention(q64[s, :256], q64[s, 256:512], q64[s, 512:], 4)
        assert np.max(np.abs(out[s] - ref)) < tol, (i, lens[i])
    # logits that grow along the sequence: the running reference maximum has to be raised again
    # and again (the tensor-core kernel then rescales its accumulator in tensor memory)
    q3 = qkv.copy()
    ramp = np.concatenate([1.0 + 6.0 * np.arange(n) / max(n - 1, 1) for n in lens])
    q3[:, 256:512] *= ramp[:, None]
    if dtype == "bf16":
        q3 = I.round_to_bf16(q3)
    out3 = to_np(enc.wf_attention(_dev(q3, tdt), cu))
    enc.wf_check()
    q3_64 = q3.astype(np.float64)
    for i in range(len(lens)):
        s = slice(cu[i], cu[i + 1])
        ref = O.attention(q3_64[s, :256], q3_64[s, 256:512], q3_64[s, 512:], 4)
        assert np.max(np.abs(out3[s] - ref)) < (4e-2 if dtype == "bf16" else 1e-4), (i, lens[i])   # logits up to ~60
    # one key far above everything seen before it, sitting where the tensor-core kernel evaluates 2^a on
    # the FMA pipe (in-step key indices 6, 7, 14, 15, ... of a 96-key step) in a step after the first:
    # the reference maximum must be raised there too.  Every query of the sequence carries a constant
    # in channel 0 of each head, the chosen keys a large value in the same channel.
    q4 = qkv.copy()
    def spike(seq, key, nats):
        rows = slice(cu[seq], cu[seq + 1])
        for h in range(4):
            q4[rows, 64 * h] = 8.0
            q4[cu[seq] + key, 256 + 64 * h] = nats
    spike(4, 96 + 6, 150.0)                 # 200 keys: second step, FMA-pipe lane
    spike(5, 3 * 96 + 7, 130.0)             # 1525 keys: two such keys in two different steps,
    spike(5, 9 * 96 + 31, 280.0)            # the later one higher again
    if dtype == "bf16":
        q4 = I.round_to_bf16(q4)
    out4 = to_np(enc.wf_attention(_dev(q4, tdt), cu))
    enc.wf_check()
    q4_64 = q4.astype(np.float64)
    for i in (4, 5):
        s = slice(cu[i], cu[i + 1])
        ref = O.attention(q4_64[s, :256], q4_64[s, 256:512], q4_64[s, 512:], 4)
        assert np.max(np.abs(out4[s] - ref)) < tol, (i, lens[i])
    key = cu[5] + 9 * 96 + 31                # the dominant key's value row comes back for every query
    assert np.max(np.abs(out4[cu[5]:cu[6]] - q4_64[key, 512:])) < tol
    # identical keys -> mean of values
    q2 = qkv.copy()
    q2[:, 256:512] = q2[0, 256:512]
    out2 = to_np(enc.wf_attention(_dev(q2, tdt), cu))
    s = slice(cu[4], cu[5])
    assert np.max(np.abs(out2[s] - q2[s, 512:].astype(np.float64).mean(axis=0))) < tol
    enc.close()


# ------------------------------------------------------------------------------ bf16 path

def _check_bf16(got, ref):
    """The stated bf16 tolerance read as max|err| / max|ref| per sequence and per-token cosine, plus
    an element-wise bound that also covers channels far below the sequence's peak."""
    assert peak_rel_err(got, ref) <= BF16_REL
    assert min_token_cosine(got, ref) >= BF16_COS
    assert elementwise_excess(got, ref, BF16_REL) <= 1.0


def test_bf16_small_ragged_matches_oracle():
    shape = _small("bf16", d_model=256, n_head=4, d_mlp=1024, n_layer=3)
    W = I.encoder_weights(7, shape)
    lengths = [160 * 7, 160 * 300, 401, 160 * 131, 160 * 64 + 5, 160 * 10]
    batch = I.batch_from_lengths(8, lengths)
    hush = I.round_to_bf16(I.hush_mel(8, shape.n_mel))
    enc = make_encoder(shape, W, 8, 2048, int(sum(lengths)))
    out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    assert out.dtype == torch.bfloat16
    got = to_np(out)
    refs = oracle_hidden(batch, shape, W, hush)
    for i, r in refs.items():
        _check_bf16(got[cu[i]:cu[i + 1]], r)
    enc.close()


def test_bf16_deep_encoder_with_spare_capacity():
    """Many layers on an encoder sized far beyond the batch: the rows between the batch's last token and
    the end of the last stored tile exist in memory and pass through every layer.  They must stay
    finite (they are written as zeros): the attention kernel multiplies the rows behind a sequence's
    end by zero probabilities, and anything non-finite there would spoil the last sequence."""
    shape = _small("bf16", d_model=256, n_head=4, d_mlp=1024, n_layer=24)
    W = I.encoder_weights(13, shape)
    batch = I.batch_from_lengths(13, [160 * 150, 160 * 611])          # 100 + 331 tokens: 431 = 3 x 128 + 47
    hush = I.round_to_bf16(I.hush_mel(13, shape.n_mel))
    enc = make_encoder(shape, W, 16, 8192, 16 * 160 * 1500)
    for _ in range(2):                                                   # the second call finds the first call's rows
        out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
        enc.wf_check()
        got = to_np(out)
        assert np.isfinite(got).all()
        refs = oracle_hidden(batch, shape, W, hush)
        for i, ref in refs.items():
            _check_bf16(got[cu[i]:cu[i + 1]], ref)
    enc.close()


def test_bf16_many_minimal_buffers():
    """400 buffers, most of them the shortest the front end accepts (401 samples: 2 frames + hush =
    26 tokens), some a little longer: work lists, tile maps and metadata at a high sequence count."""
    shape = _small("bf16", d_model=256, n_head=4, d_mlp=512, n_layer=2)
    W = I.encoder_weights(12, shape)
    rng = np.random.default_rng(12)
    lengths = [401 if rng.random() < 0.7 else int(rng.integers(402, 160 * 12)) for _ in range(400)]
    batch = I.batch_from_lengths(13, lengths)
    hush = I.round_to_bf16(I.hush_mel(13, shape.n_mel))
    tokens = int(I.tokens_of(batch.lengths).sum())
    enc = make_encoder(shape, W, 400, tokens, int(batch.lengths.sum()))
    out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    again, _ = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    assert cu[-1] == tokens and torch.equal(out, again)
    got = to_np(out)
    picks = [0, 1, 199, 398, 399, int(np.argmax(lengths))]
    for i, r in oracle_hidden(batch, shape, W, hush, only=set(picks)).items():
        _check_bf16(got[cu[i]:cu[i + 1]], r)
    enc.close()


def test_bf16_attention_stress_weights():
    """Query/key weights scaled so that logits have a standard deviation of a few units."""
    shape = _small("bf16", d_model=256, n_head=4, d_mlp=512, n_layer=2)
    W = I.encoder_weights(9, shape, logit_gain=6.0)
    batch = I.batch_from_lengths(10, [160 * 250, 160 * 33])
    hush = I.round_to_bf16(I.hush_mel(10, shape.n_mel))
    enc = make_encoder(shape, W, 2, 1024, int(batch.lengths.sum()))
    out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    got = to_np(out)
    for i, r in oracle_hidden(batch, shape, W, hush).items():
        _check_bf16(got[cu[i]:cu[i + 1]], r)
    enc.close()


def test_bf16_base_config_matches_oracle():
    """Base-shaped encoder, 16 buffers of 1-10 s + hush, ragged (the second configuration)."""
    shape = I.SHAPES["base"]
    W = I.encoder_weights(1, shape)
    batch = I.config_batch("base")
    hush = I.round_to_bf16(I.hush_mel(1, shape.n_mel))
    M = int(I.tokens_of(batch.lengths).sum())
    enc = make_encoder(shape, W, 16, M, int(batch.lengths.sum()))
    out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    got = to_np(out)
    assert cu[-1] == M
    for i, r in oracle_hidden(batch, shape, W, hush).items():
        _check_bf16(got[cu[i]:cu[i + 1]], r)
    # host-buffer entry point gives the same result, bit for bit
    a_host = torch.as_tensor(batch.audio).pin_memory()
    o_host = torch.empty((M, shape.d_model), dtype=torch.bfloat16).pin_memory()
    enc.wf_encode_host(a_host, batch.lengths, _dev(hush), o_host)
    assert torch.equal(o_host, out.cpu())
    # and so does the pipelined form: seven calls on sub-batches of different sizes, in flight two at a
    # time, each compared (after its own ticket) with the synchronous call on the same sub-batch
    subs = [(0, 16), (3, 9), (0, 1), (5, 16), (15, 16), (2, 4), (0, 16)]
    offs = np.concatenate([[0], np.cumsum(batch.lengths)])
    audio_h = [torch.as_tensor(batch.audio[offs[lo]:offs[hi]].copy()).pin_memory() for lo, hi in subs]
    want = []
    for (lo, hi), a_h in zip(subs, audio_h):
        w = torch.empty((int(cu[hi] - cu[lo]), shape.d_model), dtype=torch.bfloat16).pin_memory()
        enc.wf_encode_host(a_h, batch.lengths[lo:hi], _dev(hush), w)
        want.append(w.clone())
    assert torch.equal(want[0], out.cpu())
    pending = []
    for j, (lo, hi) in enumerate(subs):
        o_h = torch.full((int(cu[hi] - cu[lo]), shape.d_model), float("nan"), dtype=torch.bfloat16).pin_memory()
        ticket, cu_sub = enc.wf_encode_host_async(audio_h[j], batch.lengths[lo:hi], _dev(hush), o_h)
        assert list(cu_sub) == list(cu[lo:hi + 1] - cu[lo])
        pending.append((ticket, j, o_h))
        if len(pending) > 2:
            t, i, o = pending.pop(0)
            enc.wf_encode_host_wait(t)
            assert torch.equal(o, want[i]), subs[i]
    for t, i, o in pending:
        enc.wf_encode_host_wait(t)
        assert torch.equal(o, want[i]), subs[i]
    enc.wf_check()
    enc.close()


def test_dtw_matches_oracle_bit_for_bit():
    from oracle import dtw_oracle
    shape = _small("f32", n_layer=0)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 8, 64, 1000)
    # first batch: ragged, degenerate, wide, tall, all small enough for the arg-min bytes to stay in
    # shared memory; second batch: a problem too large for that (bytes go to the workspace) and one
    # with more tokens than threads (several cells per thread and anti-diagonal)
    for batch in ([(40, 300), (1, 17), (23, 1), (150, 775), (300, 97), (7, 7)], [(300, 900), (5, 9), (600, 300)]):
        costs = [I.dtw_cost(4, b, n, m) for b, (n, m) in enumerate(batch)]
        packed = np.concatenate([c.reshape(-1) for c in costs])
        start, total = enc.wf_dtw(_dev(packed), [n for n, _ in batch], [m for _, m in batch])
        enc.wf_check()
        start, total = start.cpu().numpy(), total.cpu().numpy()
        off = 0
        for b, c in enumerate(costs):
            t_ref, _, s_ref = dtw_oracle.dtw(c)
            assert total[b] == t_ref                               # same float32 additions, same order
            assert np.array_equal(start[off:off + len(s_ref)], s_ref), (batch, b)
            off += len(s_ref)
    # ties: matrices whose cells tie by construction (constant, small integers), where the stated order
    # (diagonal, then the token step, then the frame step) decides the path
    rng = np.random.default_rng(8)
    ties = [np.ones((2, 3), np.float32), np.array([[5, -1], [-1, 0]], np.float32), np.zeros((3, 3), np.float32),
            np.zeros((37, 150), np.float32), rng.integers(0, 3, size=(60, 200)).astype(np.float32)]
    start, total = enc.wf_dtw(_dev(np.concatenate([c.reshape(-1) for c in ties])), [c.shape[0] for c in ties],
                              [c.shape[1] for c in ties])
    enc.wf_check()
    start, total = start.cpu().numpy(), total.cpu().numpy()
    off = 0
    for b, c in enumerate(ties):
        t_ref, _, s_ref = dtw_oracle.dtw(c)
        assert total[b] == t_ref and np.array_equal(start[off:off + len(s_ref)], s_ref), b
        off += len(s_ref)
    enc.close()


# ------------------------------------------------------------------------------ resident stream windows

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_stream_windows_match_encoding_from_scratch(dtype):
    """Windows that grow at the end every round and are cut at the front now and then (Sec. 3.2):
    only the changed frames are recomputed, and the encoding of the resident windows equals,
    bit for bit, wf_encode of the same windows, and the oracle's from-scratch result."""
    from paper_2412_11272_b200.binding import Streams, WfError
    bf16 = dtype == "bf16"
    shape = _small(dtype, n_layer=1, **({"d_model": 256, "n_head": 4, "d_mlp": 512} if bf16 else {}))
    W = I.encoder_weights(21, shape)
    hush_np = I.hush_mel(21, 80)
    if bf16:
        hush_np = I.round_to_bf16(hush_np)
    hush = _dev(hush_np)
    n_streams, cap = 4, 160 * 700
    enc = make_encoder(shape, W, n_streams, 4 * 400, n_streams * cap)
    st = Streams(enc, n_streams, cap)
    feed = [I.synth_audio(21, 40 + i, 16000 * 12) for i in range(n_streams)]      # each stream's endless input
    pos = [0] * n_streams                    # samples consumed from the feed
    start = [0] * n_streams                  # first sample of the window within the feed
    rng = np.random.default_rng(3)
    for rnd in range(9):
        ids = [i for i in range(n_streams) if rnd == 0 or rng.random() < 0.8] or [0]
        ids = [int(i) for i in rng.permutation(ids)]
        n_new, trim = [], []
        for i in ids:
            add = int(rng.choice([16000, 8000, 16000 + 37, 3 * 160 + 1, 700]))
            win = pos[i] - start[i]
            cut = 0
            if rnd == 0:
                add = max(add, 1000)
            elif rnd == 7 and i == ids[0]:
                cut, add = (win // 160) * 160, 16000                    # all but a ragged remainder goes
            elif rnd in (3, 6) and win > 1200:
                cut = 160 * int(rng.integers(1, (win - 800) // 160 + 1))
            if win - cut + add > cap:
                cut += -(-(win - cut + add - cap) // 160) * 160
            n_new.append(add)
            trim.append(cut)
        new_audio = np.concatenate([feed[i][pos[i]:pos[i] + a] for i, a in zip(ids, n_new)])
        st.wf_streams_push(ids, _dev(new_audio), n_new, trim)
        for i, a, c in zip(ids, n_new, trim):
            pos[i] += a
            start[i] += c
            assert st.wf_streams_length(i) == pos[i] - start[i]
        live = [i for i in range(n_streams) if pos[i] - start[i] >= 401]
        out, cu = st.wf_encode_streams(live, hush)
        windows = [feed[i][start[i]:pos[i]] for i in live]
        lengths = [len(w) for w in windows]
        ref, cu_ref = enc.wf_encode(_dev(np.concatenate(windows)), lengths, hush)
        enc.wf_check()
        assert list(cu) == list(cu_ref)
        assert torch.equal(out, ref), rnd
        if rnd in (4, 8):
            got = to_np(out)
            for k, w in enumerate(windows[:2]):
                r = O.encode_sequence(w, I.mel_filterbank(80), hush_np, W, shape.n_layer, shape.n_head)
                if bf16:
                    _check_bf16(got[cu[k]:cu[k + 1]], r)
                else:
                    assert np.max(np.abs(got[cu[k]:cu[k + 1]] - r)) <= F32_TOL
    # errors leave the windows untouched
    before = [st.wf_streams_length(i) for i in range(n_streams)]
    for ids, n_new, trim, status in (([0, 0], [160, 160], None, "WF_ERR_INVALID_ARG"),
                                     ([1], [160], [100], "WF_ERR_INVALID_ARG"),
                                     ([1], [cap], None, "WF_ERR_CAPACITY"),
                                     ([2], [0], [(before[2] // 160) * 160], "WF_ERR_TOO_SHORT"),
                                     ([9], [160], None, "WF_ERR_INVALID_ARG")):
        with pytest.raises(WfError) as ei:
            st.wf_streams_push(ids, _dev(np.zeros(max(sum(n_new), 1), np.float32)), n_new, trim)
        assert ei.value.status == status, (ids, n_new, trim)
    assert [st.wf_streams_length(i) for i in range(n_streams)] == before
    st.close()
    enc.close()


# ------------------------------------------------------------------------------ errors and edges

def test_bounded_wait_runs_out_and_is_reported():
    """The failure path of every bounded device-side wait, exercised without a fault: a one-warp
    kernel waits with the library's wait routine on a barrier nobody signals; the wait gives up
    after the requested number of polls, the kernel ends normally, wf_check reports
    WF_ERR_DEVICE_TIMEOUT once, and the handle then encodes as before."""
    from paper_2412_11272_b200.binding import WfError
    shape = _small("bf16", d_model=256, n_head=4, d_mlp=512, n_layer=2)
    W = I.encoder_weights(11, shape)
    batch = I.batch_from_lengths(11, [160 * 40, 160 * 121])
    hush = I.round_to_bf16(I.hush_mel(11, shape.n_mel))
    enc = make_encoder(shape, W, 2, 200, int(batch.lengths.sum()))
    before, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    enc.wf_selftest_wait_timeout(2000)
    with pytest.raises(WfError) as ei:
        enc.wf_check()
    assert ei.value.status == "WF_ERR_DEVICE_TIMEOUT"
    enc.wf_check()                                   # the record was cleared by the failing check
    after, _ = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush))
    enc.wf_check()
    assert torch.equal(before, after)
    refs = oracle_hidden(batch, shape, W, hush)
    for i, ref in refs.items():
        _check_bf16(to_np(after)[cu[i]:cu[i + 1]], ref)
    enc.close()


def test_errors_and_edge_cases():
    from paper_2412_11272_b200.binding import WfError
    shape = _small("f32", n_layer=1, n_ctx=40)
    W = I.encoder_weights(2, shape)
    enc = make_encoder(shape, W, 2, 64, 20000, hush_frames=3)
    hush = _dev(I.hush_mel(2, 80, 3))
    audio = _dev(I.synth_audio(2, 0, 20000))
    out, cu = enc.wf_encode(audio, [], hush)                          # empty batch
    assert list(cu) == [0] and out.shape[0] == 0
    for lengths, status in (([400], "WF_ERR_TOO_SHORT"), ([160 * 80], "WF_ERR_TOO_LONG"),
                            ([1000, 1000, 1000], "WF_ERR_CAPACITY"), ([10000, 10001], "WF_ERR_CAPACITY")):
        with pytest.raises(WfError) as ei:
            enc.wf_encode(audio, lengths, hush)
        assert ei.value.status == status, lengths
    with pytest.raises(WfError) as ei:
        enc.wf_encode(audio, [1600], None)                            # hush required
    assert ei.value.status == "WF_ERR_INVALID_ARG"
    out, cu = enc.wf_encode(audio, [160 * 77], hush)                  # exactly n_ctx tokens is fine
    assert cu[-1] == 40
    enc.wf_check()
    enc.close()
    bad = I.EncoderShape("bad", 80, 96, 1, 2, 256, "f32")
    with pytest.raises(WfError):
        make_encoder(bad, I.encoder_weights(0, bad), 1, 8, 1000)

"""Parity at the full sizes of the named configurations, in the launch configuration the
benchmark times: the whole ragged batch runs on the GPU, the fp64 oracle re-computes a few
whole sequences (legal because sequences are independent) and those rows are compared."""
import numpy as np
import pytest

from paper_2412_11272_b200 import inputs as I
from tests._util import elementwise_excess, make_encoder, min_token_cosine, oracle_hidden, peak_rel_err, to_np

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _dev(a):
    return torch.as_tensor(np.ascontiguousarray(a)).to("cuda:0", torch.float32)


_weights = {}


def _run(name, batch, hush_frames, picks, n_ctx=None):
    shape = I.SHAPES[name]
    seed = I.CONFIG_SEED[name]
    if name not in _weights:
        _weights.clear()                      # one model's weights at a time
        _weights[name] = I.encoder_weights(seed, shape)
    W = _weights[name]
    hush = I.round_to_bf16(I.hush_mel(seed, shape.n_mel)) if hush_frames else None
    tokens = int(I.tokens_of(batch.lengths, hush_frames).sum())
    enc = make_encoder(shape, W, len(batch.lengths), tokens, int(batch.lengths.sum()), hush_frames=hush_frames,
                       n_ctx=n_ctx)
    out, cu = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush) if hush_frames else None)
    enc.wf_check()
    assert cu[-1] == tokens
    assert list(np.diff(cu)) == list(I.tokens_of(batch.lengths, hush_frames))
    got = to_np(out)
    assert np.isfinite(got).all()
    # a property that holds at any size: the path has a fixed order of operations, so repeating the
    # call reproduces every bit (a data race anywhere in the launch sequence shows up here)
    first = out.clone()
    for _ in range(3):
        again, _ = enc.wf_encode(_dev(batch.audio), batch.lengths, _dev(hush) if hush_frames else None)
        assert torch.equal(again, first), name
    refs = oracle_hidden(batch, shape, W, hush, only=set(picks))
    for i, ref in refs.items():
        g = got[cu[i]:cu[i + 1]]
        assert peak_rel_err(g, ref) <= 3e-2, (name, i)
        assert min_token_cosine(g, ref) >= 0.999, (name, i)
        assert elementwise_excess(g, ref) <= 1.0, (name, i)
    enc.close()
    return got, cu


def _extremes(lengths, extra=1):
    order = np.argsort(lengths)
    picks = [int(order[0]), int(order[-1])] + [int(order[len(order) // 2])][:extra]
    return sorted(set(picks))


def test_small_config_64_ragged_buffers_up_to_30s():
    batch = I.config_batch("small")
    assert len(batch.lengths) == 64 and I.tokens_of(batch.lengths).max() <= 1525
    _run("small", batch, 50, _extremes(batch.lengths), n_ctx=1536)


def test_medium_config_padded_30s_and_hush_truncated():
    padded = I.config_batch("medium", variant="padded")
    hushed = I.config_batch("medium", variant="hush")
    assert np.all(padded.lengths == 480000)
    _run("medium", padded, 0, [0])                      # 1500 tokens each, no hush
    _run("medium", hushed, 50, _extremes(hushed.lengths, extra=0))
    # the hush-terminated run costs a fraction of the padded run (Sec. 2.2 / Sec. 6.3: ~3-3.7x on 5-25 s clips;
    # these 1-8 s buffers save more)
    shape = I.SHAPES["medium"]
    ratio = (I.algorithmic_flops(shape, padded.lengths, 0)["encoder"] /
             I.algorithmic_flops(shape, hushed.lengths)["encoder"])
    assert 4.0 < ratio < 12.0


def test_large_config_round_15_and_staggered_round():
    full = I.config_batch("large", round_s=15)
    _run("large", full, 50, [0, 63])
    ragged = I.config_batch("large", round_s=7, staggered=True)     # windows of 1..15 s in one batch
    assert len(set(ragged.lengths.tolist())) == 15
    _run("large", ragged, 50, _extremes(ragged.lengths, extra=0))

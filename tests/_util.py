"""Shared helpers for the GPU parity tests (inputs, oracle runs, error metrics)."""
import numpy as np

from oracle import wf_oracle as O
from paper_2412_11272_b200 import inputs as I


def has_gpu():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def make_encoder(shape, weights, max_batch, max_tokens, max_samples, **kw):
    from paper_2412_11272_b200.binding import Encoder
    return Encoder(shape, weights, I.mel_filterbank(shape.n_mel), max_batch, max_tokens, max_samples, **kw)


def oracle_hidden(batch, shape, weights, hush, only=None):
    """Oracle output per sequence (dict index -> [n_i, d]); `only` restricts to some sequences."""
    F = I.mel_filterbank(shape.n_mel)
    out = {}
    for i, s in enumerate(batch.sequences()):
        if only is not None and i not in only:
            continue
        out[i] = O.encode_sequence(s, F, hush, weights, shape.n_layer, shape.n_head)
    return out


def peak_rel_err(got, ref):
    """max|got - ref| / max|ref| over one sequence (the 'max-rel' of the bf16 tolerance)."""
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


def elementwise_excess(got, ref, rel=3e-2):
    """max over elements of |got - ref| / (rel |ref| + rel rms(ref row)): at most 1 when every element is
    within `rel` of its own magnitude plus `rel` of its token's root mean square (covers the channels
    far below the sequence's peak, which the peak-normalised measure cannot see)."""
    rms = np.sqrt((ref ** 2).mean(axis=1, keepdims=True))
    return float((np.abs(got - ref) / (rel * np.abs(ref) + rel * rms)).max())


def min_token_cosine(got, ref):
    num = (got * ref).sum(axis=1)
    den = np.linalg.norm(got, axis=1) * np.linalg.norm(ref, axis=1)
    return float(np.min(num / den))


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)

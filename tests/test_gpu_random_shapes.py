"""Randomised robustness sweep of the bf16 kernels: GEMM, variable-length attention and the whole
encoder on shapes drawn around the tile and step boundaries.  Every launch is repeated and must
reproduce its first result bit for bit (the default path has a fixed order of operations, so any
difference is a data race), and is compared with a float32 evaluation on the device.  This is a
race and edge-case detector; the parity claims are the oracle comparisons in the other files."""
import math

import numpy as np
import pytest

from paper_2412_11272_b200 import inputs as I
from tests._util import make_encoder

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

D_MODEL, N_HEAD = 256, 4


@pytest.fixture(scope="module")
def enc():
    shape = I.EncoderShape("sweep", 80, D_MODEL, 2, N_HEAD, 512, "bf16", n_ctx=1600)
    e = make_encoder(shape, I.encoder_weights(3, shape), 24, 40000, 24 * 160 * 1500 + 1000)
    yield e
    e.close()


def test_gemm_random_shapes(enc):
    """mode 0 / 1: plain and GELU epilogue; 2: residual update on the split stream (N a multiple of
    128); 3: LayerNorm folded into the GEMM (K a multiple of 128)."""
    rng = np.random.default_rng(100)
    for _ in range(160):
        M = max(1, int(rng.choice([1, 7, 31, 127, 128, 129, 255, 257, 300, 1000, 4097, 9000, 20000])) + int(rng.integers(-3, 4)))
        N, K, mode = 8 * int(rng.integers(1, 200)), 8 * int(rng.integers(1, 200)), int(rng.integers(0, 4))
        if mode == 2:
            N = 128 * int(rng.integers(1, 13))
        if mode == 3:
            K = 128 * int(rng.integers(1, 11))
        A = torch.randn(M, K, device="cuda").to(torch.bfloat16)
        W = (torch.randn(N, K, device="cuda") / math.sqrt(K)).to(torch.bfloat16)
        b = torch.randn(N, device="cuda")
        ref = A.float() @ W.float().T + b
        outs = []
        if mode == 3:
            stats = torch.stack([A.float().view(M, K // 128, 128).sum(-1).T, (A.float() ** 2).view(M, K // 128, 128).sum(-1).T],
                                dim=-1).contiguous()
            ones, zeros = torch.ones(K, device="cuda"), torch.zeros(K, device="cuda")
            Wg, colsum, cbias = enc.wf_ln_fold(W.float(), ones, zeros, b)
            assert torch.equal(Wg, W)
            mu = A.float().mean(1, keepdim=True)
            ref = (A.float() - mu) / torch.sqrt(A.float().var(1, unbiased=False, keepdim=True) + 1e-5) @ W.float().T + b
        for _ in range(3):
            if mode == 2:
                hi, lo = torch.ones(M, N, device="cuda").to(torch.bfloat16), torch.full((M, N), 2.0 ** -10, device="cuda").to(torch.bfloat16)
                st = enc.wf_gemm_resid_bf16(A, W, b, hi, lo)
                outs.append(torch.cat([hi.float() + lo.float(), st[..., 0].T, st[..., 1].T], dim=1))
            elif mode == 3:
                outs.append(enc.wf_gemm_ln_bf16(A, stats, Wg, colsum, cbias, False))
            else:
                outs.append(enc.wf_gemm_bf16(A, W, b, mode))
        got = outs[0]
        if mode == 2:
            ref = ref + 1.0 + 2.0 ** -10
            sums = got[:, N:N + N // 128].sum(1)
            assert float(((sums - got[:, :N].sum(1)).abs() / (got[:, :N].abs().sum(1) + 1.0)).max()) < 1e-5, (M, N, K)
            got = got[:, :N]
        elif mode == 1:
            ref = torch.nn.functional.gelu(ref)
        err = float(((got.float() - ref).abs() / (ref.abs() + 1.0)).max())
        assert all(torch.equal(outs[0], o) for o in outs[1:]), (M, N, K, mode)
        assert err < (2e-4 * math.sqrt(K) if mode == 2 else 2.0 ** -7), (M, N, K, mode, err)
    enc.wf_check()


def test_attention_random_batches(enc):
    rng = np.random.default_rng(101)
    edges = [1, 2, 5, 31, 95, 96, 97, 127, 128, 129, 191, 192, 193, 255, 256, 257, 300, 513, 775, 1000, 1525]
    for _ in range(120):
        B = int(rng.integers(1, 20))
        lens = [max(1, int(rng.choice(edges)) + int(rng.integers(-2, 3))) for _ in range(B)]
        cu = np.concatenate([[0], np.cumsum(lens)])
        qkv = (torch.randn(int(cu[-1]), 3 * D_MODEL, device="cuda") * float(rng.choice([0.5, 1.0, 3.0]))).to(torch.bfloat16)
        outs = [enc.wf_attention(qkv, cu) for _ in range(3)]
        assert all(torch.equal(outs[0], o) for o in outs[1:]), lens
        q, k, v = qkv.float().split(D_MODEL, dim=1)
        ref = torch.empty(int(cu[-1]), D_MODEL, device="cuda")
        for i in range(B):
            s, e = int(cu[i]), int(cu[i + 1])
            qq, kk, vv = (t[s:e].view(-1, N_HEAD, 64).transpose(0, 1) for t in (q, k, v))
            p = torch.softmax(qq @ kk.transpose(1, 2) / 8.0, dim=-1)
            ref[s:e] = (p @ vv).transpose(0, 1).reshape(-1, D_MODEL)
        assert float((outs[0].float() - ref).abs().max() / ref.abs().max()) < 4e-2, lens
    enc.wf_check()


def test_encode_random_batches_repeat_and_are_batch_invariant(enc):
    rng = np.random.default_rng(102)
    hush = torch.as_tensor(I.round_to_bf16(I.hush_mel(3, 80))).cuda()
    for _ in range(60):
        B = int(rng.integers(1, 24))
        lens = np.array([int(rng.integers(401, 160 * 1500)) if rng.random() < 0.3
                         else 160 * int(rng.integers(3, 400)) + int(rng.integers(0, 160)) for _ in range(B)])
        batch = I.batch_from_lengths(int(rng.integers(0, 1000)), lens)
        audio = torch.as_tensor(batch.audio).cuda()
        outs = [enc.wf_encode(audio, batch.lengths, hush)[0] for _ in range(3)]
        assert all(torch.equal(outs[0], o) for o in outs[1:]), list(lens)
        assert bool(torch.isfinite(outs[0].float()).all())
        solo = enc.wf_encode(audio[:int(lens[0])].contiguous(), lens[:1], hush)[0]     # sequence 0 alone
        assert float((solo.float() - outs[0][:solo.shape[0]].float()).abs().max()) < 0.1, list(lens)
    enc.wf_check()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_spare_capacity_gives_the_same_bits_as_an_exact_fit(dtype):
    """One deep encoder sized far beyond its batches, fed batches of very different sizes one after
    the other, against encoders created to fit each batch exactly: kernel choices depend on the
    batch, not on the capacity, so every bit must agree -- whatever earlier calls left in the
    workspace rows behind the batch's last token."""
    n_layer = 16 if dtype == "bf16" else 3
    shape = I.EncoderShape("cap", 80, 128, n_layer, 2, 256, dtype, n_ctx=1600)
    W = I.encoder_weights(5, shape)
    hush_np = I.hush_mel(5, 80)
    hush = torch.as_tensor(I.round_to_bf16(hush_np) if dtype == "bf16" else hush_np).cuda()
    big = make_encoder(shape, W, 32, 20000, 32 * 160 * 1500)
    rng = np.random.default_rng(103)
    for case in range(8):
        B = int(rng.choice([1, 2, 17, 32]))
        lens = np.array([160 * int(rng.integers(3, 1200 if case % 2 else 60)) + int(rng.integers(0, 160)) for _ in range(B)])
        lens = lens[: max(1, min(B, int(19000 // max(1, int(I.tokens_of(lens).max())))))]      # stay inside the big encoder's tokens
        batch = I.batch_from_lengths(200 + case, lens)
        audio = torch.as_tensor(batch.audio).cuda()
        got, cu = big.wf_encode(audio, batch.lengths, hush)
        big.wf_check()
        fit = make_encoder(shape, W, len(lens), int(cu[-1]), int(batch.lengths.sum()))
        want, cu2 = fit.wf_encode(audio, batch.lengths, hush)
        fit.wf_check()
        assert list(cu) == list(cu2) and bool(torch.isfinite(got.float()).all())
        assert torch.equal(got, want), (case, list(lens))
        fit.close()
    big.close()

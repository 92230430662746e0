"""Runs one component of the library alone, for timing and for profiler captures: the commands
quoted in the profiler summaries that ship with the library are invocations of this module.

    python -m paper_2412_11272_b200.probe gemm --M 16384 --N 3840 --K 1280 --mode 0    (modes: 0 bias, 1 + GELU,
                                         2 residual update on the split stream, 3 / 4 LayerNorm folded in)
    python -m paper_2412_11272_b200.probe attention --n 775 --batch 64
    python -m paper_2412_11272_b200.probe encode --shape large --seconds 3 --batch 16
    python -m paper_2412_11272_b200.probe logmel --seconds 15 --batch 64
    python -m paper_2412_11272_b200.probe dtw --batch 64 --n 150
    python -m paper_2412_11272_b200.probe crosskv --M 49600 --layers 32
    python -m paper_2412_11272_b200.probe streams --shape large --batch 64      (resident windows: push 1 s, encode, 15 rounds)
    python -m paper_2412_11272_b200.probe config --name small        (tiny, base, small, medium-padded, medium-hush, large)

Each command warms up, times ``--iters`` launches with CUDA events on the launching stream and
prints one JSON line (milliseconds per launch and the algorithmic rate).  Inputs are synthetic.
"""
from __future__ import annotations

import argparse
import json
import math

import numpy as np
import torch

from . import inputs as I
from .binding import Encoder, Streams


def _time(fn, iters, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _component_encoder(d_model=128, n_head=2, max_batch=1, max_tokens=64):
    shape = I.EncoderShape("probe", 80, d_model, 0, n_head, 256, "bf16", n_ctx=4096)
    return Encoder(shape, I.encoder_weights(0, shape), I.mel_filterbank(80), max_batch, max_tokens, 1000)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["gemm", "attention", "encode", "logmel", "config", "dtw", "crosskv", "streams"])
    ap.add_argument("--name", default="base")
    ap.add_argument("--M", type=int, default=16384)
    ap.add_argument("--N", type=int, default=3840)
    ap.add_argument("--K", type=int, default=1280)
    ap.add_argument("--mode", type=int, default=0)
    ap.add_argument("--n", type=int, default=775)
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--d_model", type=int, default=1280)
    ap.add_argument("--shape", default="large")
    ap.add_argument("--seconds", type=float, default=3.0)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--iters", type=int, default=10)
    a = ap.parse_args()
    out = {"what": a.what}
    if a.what == "gemm":
        enc = _component_encoder()
        A = torch.randn(a.M, a.K, device="cuda").to(torch.bfloat16)
        W = (torch.randn(a.N, a.K, device="cuda") / math.sqrt(a.K)).to(torch.bfloat16)
        b = torch.randn(a.N, device="cuda")
        # --mode 0 bias, 1 bias + GELU, 2 residual update on the split stream, 3 / 4 LayerNorm folded in (4: + GELU)
        if a.mode == 2:
            hi = torch.randn(a.M, a.N, device="cuda").to(torch.bfloat16)
            lo = torch.zeros_like(hi)
            ms = _time(lambda: enc.wf_gemm_resid_bf16(A, W, b, hi, lo), a.iters)
        elif a.mode >= 3:
            stats = torch.stack([A.float().view(a.M, a.K // 128, 128).sum(-1).T,
                                 (A.float() ** 2).view(a.M, a.K // 128, 128).sum(-1).T], dim=-1).contiguous()
            cs = W.float().sum(1)
            ms = _time(lambda: enc.wf_gemm_ln_bf16(A, stats, W, cs, b, a.mode == 4), a.iters)
        else:
            C = torch.zeros(a.M, a.N, device="cuda", dtype=torch.bfloat16)
            ms = _time(lambda: enc.wf_gemm_bf16(A, W, b, a.mode, C), a.iters)
        enc.wf_check()
        out.update(M=a.M, N=a.N, K=a.K, mode=a.mode, ms=ms, tflops=2.0 * a.M * a.N * a.K / ms / 1e9)
    elif a.what == "attention":
        d = a.d_model
        enc = _component_encoder(d, d // 64, a.batch, a.batch * a.n)
        cu = np.arange(a.batch + 1) * a.n
        qkv = torch.randn(int(cu[-1]), 3 * d, device="cuda").to(torch.bfloat16)
        ms = _time(lambda: enc.wf_attention(qkv, cu), a.iters)
        enc.wf_check()
        out.update(n=a.n, batch=a.batch, d_model=d, ms=ms, tflops=4.0 * a.batch * a.n * a.n * d / ms / 1e9)
    elif a.what == "crosskv":
        # --M encoder tokens of width --d_model projected to the keys and values of --layers decoder layers
        d, N = a.d_model, a.layers * 2 * a.d_model
        enc = _component_encoder(d, d // 64)
        hidden = torch.randn(a.M, d, device="cuda").to(torch.bfloat16)
        W = (torch.randn(N, d, device="cuda") * 0.02).to(torch.bfloat16)
        b = torch.zeros(N, device="cuda")
        kv = torch.empty(a.M, N, device="cuda", dtype=torch.bfloat16)
        ms = _time(lambda: enc.wf_cross_kv(hidden, W, b, kv), a.iters)
        enc.wf_check()
        out.update(M=a.M, d_model=d, layers=a.layers, ms=ms, tflops=2.0 * a.M * N * d / ms / 1e9,
                   write_gbs=2.0 * a.M * N / ms / 1e6)
    elif a.what == "streams":
        # --batch streams, 15 rounds: every round each window grows by 1 s, then all windows are encoded;
        # "push" times wf_streams_push (framing of the new second only), "front_end_full" times the
        # front end over the whole windows (wf_logmel) for comparison
        shape = I.SHAPES[a.shape]
        B, rounds = a.batch, 15
        tokens = int(I.tokens_of(np.full(B, rounds * 16000)).sum())
        enc = Encoder(shape, I.encoder_weights(0, shape), I.mel_filterbank(shape.n_mel), B, tokens, B * rounds * 16000)
        st = Streams(enc, B, rounds * 16000)
        feed = torch.as_tensor(np.stack([I.synth_audio(0, b, rounds * 16000) for b in range(B)])).cuda()
        hush = torch.as_tensor(I.round_to_bf16(I.hush_mel(0, shape.n_mel))).cuda()
        outb = torch.empty((tokens, shape.d_model), dtype=enc.out_dtype, device="cuda")
        ids = list(range(B))
        ev = lambda: torch.cuda.Event(enable_timing=True)
        push_ms = enc_ms = full_ms = 0.0
        for k in range(1, rounds + 1):
            new = feed[:, (k - 1) * 16000:k * 16000].contiguous().reshape(-1)
            win = feed[:, :k * 16000].contiguous().reshape(-1)
            e = [ev() for _ in range(4)]
            e[0].record()
            st.wf_streams_push(ids, new, [16000] * B)
            e[1].record()
            st.wf_encode_streams(ids, hush, out=outb)
            e[2].record()
            enc.wf_logmel(win, [k * 16000] * B)
            e[3].record()
            torch.cuda.synchronize()
            push_ms += e[0].elapsed_time(e[1]); enc_ms += e[1].elapsed_time(e[2]); full_ms += e[2].elapsed_time(e[3])
        enc.wf_check()
        out.update(shape=a.shape, streams=B, rounds=rounds, push_ms_total=push_ms, encode_ms_total=enc_ms,
                   front_end_full_ms_total=full_ms, audio_s_per_s=B * sum(range(1, rounds + 1)) / (push_ms + enc_ms) * 1e3)
        st.close()
    elif a.what == "dtw":
        # --batch problems of --n tokens x (5 * --n) frames (150 tokens x 750 frames by default)
        n_tok, n_frm = (a.n if a.n != 775 else 150), 5 * (a.n if a.n != 775 else 150)
        enc = _component_encoder(128, 2, max(a.batch, 1), 64)
        cost = torch.as_tensor(np.concatenate([I.dtw_cost(0, b, n_tok, n_frm).reshape(-1) for b in range(a.batch)])).cuda()
        nt, nf = [n_tok] * a.batch, [n_frm] * a.batch
        ms = _time(lambda: enc.wf_dtw(cost, nt, nf), a.iters)
        enc.wf_check()
        cells = a.batch * n_tok * n_frm
        out.update(batch=a.batch, n_tok=n_tok, n_frm=n_frm, ms=ms, gcells_per_s=cells / ms / 1e6,
                   gbs=cells * 5.0 / ms / 1e6, sequential_steps=n_tok + n_frm - 1)
    elif a.what == "config":
        # one named configuration end to end (device-resident inputs), per-call times with CUDA events
        base = a.name.split("-")[0]
        shape = I.SHAPES[base]
        seed = I.CONFIG_SEED[base]
        kw = {"variant": a.name.split("-")[1]} if base == "medium" else {}
        hush_frames = 0 if a.name == "medium-padded" else 50
        batch = I.config_batch(base, **kw)
        tokens = int(I.tokens_of(batch.lengths, hush_frames).sum())
        enc = Encoder(shape, I.encoder_weights(seed, shape), I.mel_filterbank(shape.n_mel), len(batch.lengths),
                      tokens, int(batch.lengths.sum()), hush_frames=hush_frames)
        audio = torch.as_tensor(batch.audio).cuda()
        hush = torch.as_tensor(I.round_to_bf16(I.hush_mel(seed, shape.n_mel))).cuda() if hush_frames else None
        outb = torch.empty((tokens, shape.d_model), dtype=enc.out_dtype, device="cuda")
        for _ in range(10):
            enc.wf_encode(audio, batch.lengths, hush, out=outb)
        torch.cuda.synchronize()
        evs = []
        for _ in range(max(a.iters, 50)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            enc.wf_encode(audio, batch.lengths, hush, out=outb)
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        enc.wf_check()
        times = sorted(x.elapsed_time(y) for x, y in evs)
        ms = times[len(times) // 2]
        fl = I.algorithmic_flops(shape, batch.lengths, hush_frames)
        real_s = batch.meta.get("real_samples", int(batch.lengths.sum())) / I.SAMPLE_RATE
        out.update(name=a.name, dtype=shape.dtype, batch=len(batch.lengths), tokens=tokens, p50_ms_per_call=ms,
                   p50_ms_per_buffer=ms / len(batch.lengths), p90_ms_per_call=times[int(len(times) * 0.9)],
                   audio_s_per_s=real_s / ms * 1e3, tokens_per_s=tokens / ms * 1e3,
                   tflops=fl["encoder"] / ms / 1e9, gflop_per_call=fl["encoder"] / 1e9)
    else:
        shape = I.SHAPES[a.shape]
        n_layer = shape.n_layer if a.what == "encode" else 0
        shape = I.EncoderShape(shape.name, shape.n_mel, shape.d_model, n_layer, shape.n_head, shape.d_mlp,
                               shape.dtype, shape.n_ctx)
        L = int(a.seconds * 100) * 160
        lengths = np.full(a.batch, L, dtype=np.int64)
        batch = I.batch_from_lengths(0, lengths)
        audio = torch.as_tensor(batch.audio).cuda()
        hush = torch.as_tensor(I.round_to_bf16(I.hush_mel(0, shape.n_mel))).cuda()
        tokens = int(I.tokens_of(lengths).sum())
        enc = Encoder(shape, I.encoder_weights(0, shape), I.mel_filterbank(shape.n_mel), a.batch, tokens,
                      int(lengths.sum()))
        if a.what == "encode":
            ms = _time(lambda: enc.wf_encode(audio, lengths, hush), a.iters)
            fl = I.algorithmic_flops(shape, lengths)
            out.update(shape=a.shape, tokens=tokens, ms=ms, tflops=fl["encoder"] / ms / 1e9)
        else:
            ms = _time(lambda: enc.wf_logmel(audio, lengths), a.iters)
            frames = int((lengths // 160).sum())
            out.update(frames=frames, ms=ms, gbs=(4.0 * lengths.sum() + 4.0 * frames * shape.n_mel) / ms / 1e6,
                       fp32_tflops=frames * (2 * 201 * 399 + 2 * 201 * shape.n_mel) / ms / 1e9)
        enc.wf_check()
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()

"""Host-side helpers for running the encoder on several GPUs, one process per GPU.

Sequences are independent (no operation of the path crosses a sequence boundary), so the path
shards without any exchange of activations: weights are replicated, every rank encodes its own
sequences, and the only collectives are the barrier and the max-reduction of the timing.
"""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist


def rank_stream_ids(rank: int, streams_per_rank: int) -> list[int]:
    """Weak scaling: rank r owns streams r*S .. r*S + S - 1 (ids are global, never shared)."""
    return list(range(rank * streams_per_rank, (rank + 1) * streams_per_rank))


def sequence_cost(n_tokens, d_model: int, d_mlp: int, n_layer: int) -> np.ndarray:
    """Algorithmic FLOPs of encoding sequences of n_tokens tokens (GEMMs + attention)."""
    n = np.asarray(n_tokens, dtype=np.float64)
    return n_layer * (n * (8.0 * d_model * d_model + 4.0 * d_model * d_mlp) + 4.0 * n * n * d_model)


def lpt_partition(costs, world: int) -> list[list[int]]:
    """Strong scaling of one ragged batch: longest-processing-time-first assignment of sequences
    to ranks.  Returns, for every rank, the indices of its sequences in their original order."""
    costs = np.asarray(costs, dtype=np.float64)
    load = np.zeros(world)
    parts: list[list[int]] = [[] for _ in range(world)]
    for i in np.argsort(-costs, kind="stable"):
        r = int(np.argmin(load))
        parts[r].append(int(i))
        load[r] += costs[i]
    return [sorted(p) for p in parts]


def rank_cu_seqlens(tokens, part) -> np.ndarray:
    """Token prefix sums of the sub-batch a rank encodes: its sequences `part` (indices into the
    whole batch, ascending) keep their relative order."""
    t = np.asarray(tokens, dtype=np.int64)[list(part)]
    return np.concatenate([[0], np.cumsum(t)]).astype(np.int64)


def reassemble_packed(shards, parts, tokens) -> np.ndarray:
    """Packed hidden states of the whole batch, rows in the original sequence order, from every
    rank's packed output (`shards[r]` is rank r's [sum of its tokens, d] array, `parts[r]` its
    sequence indices).  This is the optional gather behind a strong-scaling split: the sequences
    themselves never exchange anything."""
    tokens = np.asarray(tokens, dtype=np.int64)
    cu = np.concatenate([[0], np.cumsum(tokens)])
    d = shards[0].shape[1]
    out = np.empty((int(cu[-1]), d), dtype=shards[0].dtype)
    for shard, part in zip(shards, parts):
        local = rank_cu_seqlens(tokens, part)
        assert shard.shape[0] == local[-1], "a rank's output does not match its sequences"
        for j, i in enumerate(part):
            out[cu[i]:cu[i + 1]] = shard[local[j]:local[j + 1]]
    return out


def gather_packed(local: torch.Tensor, tokens, parts) -> torch.Tensor:
    """The collective behind a strong-scaling split: every rank contributes the packed hidden
    states of its own sequences (`local`, [sum of its tokens, d], on the device of the process
    group's backend) and receives the whole batch's packed rows in the original sequence order.
    One all-gather of shards padded to the largest shard (NCCL over NVLink on GPUs, gloo on CPU);
    nothing else crosses ranks.  `parts[r]` lists rank r's sequences, `tokens` every sequence's
    token count.  Without a process group (or with one rank) it returns `local` reordered."""
    tokens = np.asarray(tokens, dtype=np.int64)
    cu = np.concatenate([[0], np.cumsum(tokens)])
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    rows = [int(tokens[list(p)].sum()) for p in parts]
    if world == 1:
        shards = [local]
    else:
        pad = max(rows)
        mine = torch.zeros((pad, local.shape[1]), dtype=local.dtype, device=local.device)
        mine[: local.shape[0]] = local
        bufs = [torch.empty_like(mine) for _ in range(world)]
        dist.all_gather(bufs, mine)
        shards = [b[:n] for b, n in zip(bufs, rows)]
    out = torch.empty((int(cu[-1]), local.shape[1]), dtype=local.dtype, device=local.device)
    for shard, part in zip(shards, parts):
        lc = rank_cu_seqlens(tokens, part)
        for j, i in enumerate(part):
            out[cu[i]:cu[i + 1]] = shard[lc[j]:lc[j + 1]]
    return out


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what a multi-GPU throughput has to be computed from."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()

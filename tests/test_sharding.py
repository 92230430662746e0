"""Multi-rank host logic on CPU (gloo, world size 2): stream ownership, the max-over-ranks
timing reduction, and the cost-balanced partition of one ragged batch with the per-rank
cu_seqlens and the reassembly of the packed rows."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_11272_b200 import inputs as I
from paper_2412_11272_b200 import sharding


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ids = sharding.rank_stream_ids(rank, 4)
        gathered = [None] * world
        dist.all_gather_object(gathered, ids)
        slowest = sharding.max_over_ranks(10.0 + 5.0 * rank)
        sharding.barrier()
        lengths = I.uniform_lengths(2, 64, 1, 30)
        shape = I.SHAPES["small"]
        cost = sharding.sequence_cost(I.tokens_of(lengths), shape.d_model, shape.d_mlp, shape.n_layer)
        mine = sharding.lpt_partition(cost, world)[rank]
        all_parts = [None] * world
        dist.all_gather_object(all_parts, mine)
        loads = [float(cost[p].sum()) for p in all_parts]
        # strong scaling of ONE ragged batch: every rank "encodes" its sequences (a stand-in that
        # marks each row with its sequence and position), the packed outputs are gathered and put
        # back into the order a single-rank call would have produced
        tokens = I.tokens_of(lengths)
        cu_mine = sharding.rank_cu_seqlens(tokens, mine)
        rows = np.concatenate([np.stack([np.full(tokens[i], i), np.arange(tokens[i])], axis=1) for i in mine])
        assert rows.shape[0] == cu_mine[-1] and list(np.diff(cu_mine)) == [int(tokens[i]) for i in mine]
        shards = [None] * world
        dist.all_gather_object(shards, rows)
        whole = sharding.reassemble_packed(shards, all_parts, tokens)
        expect = np.concatenate([np.stack([np.full(t, i), np.arange(t)], axis=1) for i, t in enumerate(tokens)])
        reassembled = float(np.array_equal(whole, expect))
        # the same through the collective (one all-gather of padded shards)
        gathered_rows = sharding.gather_packed(torch.as_tensor(rows), tokens, all_parts)
        reassembled *= float(np.array_equal(gathered_rows.numpy(), expect))
        np.save(os.path.join(out_dir, f"r{rank}.npy"),
                np.array([slowest, float(sorted(sum(gathered, [])) == list(range(4 * world))),
                          float(sorted(sum(all_parts, [])) == list(range(64))), max(loads) / (sum(loads) / world),
                          reassembled]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_on_gloo(tmp_path):
    world = 2
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        slowest, disjoint, covered, imbalance, reassembled = np.load(tmp_path / f"r{rank}.npy")
        assert reassembled == 1.0              # per-rank cu_seqlens and the gather restore the single-rank row order
        assert slowest == 15.0                 # the max, on every rank
        assert disjoint == 1.0 and covered == 1.0
        assert imbalance < 1.05                # LPT balances 64 ragged sequences within 5 %


def test_lpt_partition_properties():
    cost = np.array([9.0, 1.0, 8.0, 2.0, 7.0, 3.0])
    parts = sharding.lpt_partition(cost, 3)
    assert sorted(sum(parts, [])) == list(range(6))
    assert all(p == sorted(p) for p in parts)
    assert max(cost[p].sum() for p in parts) == 10.0
    assert sharding.lpt_partition(cost, 1) == [list(range(6))]
    assert sharding.max_over_ranks(3.5) == 3.5          # no process group: identity

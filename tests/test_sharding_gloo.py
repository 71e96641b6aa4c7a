"""World-size-2 CPU test (gloo) of the multi-rank plumbing: head sharding and the max-over-ranks timing."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2609_34272_b200.sharding import max_over_ranks, shard_heads
from paper_2609_34272_b200.workloads import Workload, bits, make_inputs


def test_shard_heads_partitions_exactly():
    for total in (1, 7, 16, 128):
        for world in (1, 2, 3, 8):
            parts = [list(shard_heads(total, world, r)) for r in range(world)]
            assert sorted(sum(parts, [])) == list(range(total))
            assert max(map(len, parts)) - min(map(len, parts)) <= 1


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # each rank scores its own heads with no exchange; results must tile the full problem
        w = Workload("shard", 2, 3, 64, 8, True, seed=3)      # six (batch, head) pairs: the split cuts through a batch
        inp = {k: bits(v) for k, v in make_inputs(w).items()}
        mine = list(shard_heads(w.B * w.H, world, rank))
        part = oracle.attn_fwd_bwd_f64(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True, heads=mine)
        for name in ("O", "dQ", "dK", "dV"):
            np.save(os.path.join(out_dir, f"{name}_{rank}.npy"), part[name])
        slowest = max_over_ranks(10.0 + rank, world)
        assert slowest == 10.0 + (world - 1)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    w = Workload("shard", 2, 3, 64, 8, True, seed=3)
    inp = {k: bits(v) for k, v in make_inputs(w).items()}
    full = oracle.attn_fwd_bwd_f64(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
    for name in ("O", "dQ", "dK", "dV"):
        got = np.concatenate([np.load(tmp_path / f"{name}_{r}.npy") for r in range(2)])
        assert np.array_equal(got, full[name].reshape(got.shape)), name     # the shards tile the one-rank result exactly


def test_share_of_a_rank_is_a_dense_problem_of_its_own():
    # what `bench.py --shard heads` hands to rank r: the flat (batch, head) axis cut at shard_heads(), batch 1
    w = Workload("shard", 2, 3, 64, 8, False, seed=5)
    inp = make_inputs(w)
    full = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, False)
    for world in (2, 4):
        parts = []
        for r in range(world):
            mine = shard_heads(w.B * w.H, world, r)
            sub = {k: v.reshape(1, w.B * w.H, w.N, w.d)[:, mine.start:mine.stop].contiguous() for k, v in inp.items()}
            if len(mine):
                parts.append(oracle.attn_fwd_bwd_f64(*(bits(sub[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, False)["dK"][0])
        assert np.array_equal(np.concatenate(parts), full["dK"].reshape(w.B * w.H, w.N, w.d))

"""The multi-GPU path on CPU: two gloo ranks shard a layer over token rows (weights replicated, no
collective on the data path), and the shards together equal the unsharded result bit for bit."""
import os
import tempfile

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2411_09909_b200 import inputs, sharding


def test_shard_rows_cover_everything_once():
    for total, world in [(2048, 2), (2048, 8), (300, 4), (128, 8), (1000, 3)]:
        got = [sharding.shard_rows(total, world, r) for r in range(world)]
        pos = 0
        for start, count in got:
            assert start == pos and count >= 0
            pos += count
        assert pos == total
        assert all(c % 128 == 0 for _, c in got[:-1] if c and _ + c < total)
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.aggregate_rate(10.0, 4, 2000.0) == 20.0


def _worker(rank, world, init_file, out_dir):
    dist.init_process_group("gloo", init_method=f"file://{init_file}", rank=rank, world_size=world)
    try:
        M = 384
        a = inputs.activation(1, 0, M=M)
        w = inputs.weight(1, 0, N=256)
        start, count = sharding.shard_rows(M, world, rank)
        qa = oracle.quantize(a[start:start + count], 32)
        qw = oracle.quantize(w, 32)                           # replicated weight
        c = oracle.gemm(*qa, *qw, 32)
        np.save(os.path.join(out_dir, f"c{rank}.npy"), c)
        slowest = sharding.max_over_ranks(10.0 + rank)        # rank 1 is "slower"
        assert slowest == 10.0 + (world - 1)
        dist.barrier()
        if rank == 0:
            full = oracle.gemm(*oracle.quantize(a, 32), *qw, 32)
            parts = np.concatenate([np.load(os.path.join(out_dir, f"c{r}.npy")) for r in range(world)])
            assert np.array_equal(parts, full)
            assert sharding.aggregate_rate(count, world, slowest) == world * count / (slowest * 1e-3)
    finally:
        dist.destroy_process_group()


def test_two_rank_row_sharding_matches_unsharded():
    oracle.lib()                                              # build once before forking
    with tempfile.TemporaryDirectory() as d:
        mp.spawn(_worker, args=(2, os.path.join(d, "rendezvous"), d), nprocs=2, join=True)

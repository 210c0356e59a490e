"""Multi-rank host logic on CPU (gloo, world size 2): token shards are disjoint and cover the batch,
per-shard results of a token-wise function reassemble to the unsharded result, and the timing
reduction takes the slowest rank."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2501_10054_b200 import sharding as S
from oracle import tardis_oracle as O


def test_token_shard_partitions():
    for n in (0, 1, 7, 64, 65, 512):
        for world in (1, 2, 3, 8):
            spans = [S.token_shard(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == n
            for (f0, c0), (f1, _) in zip(spans, spans[1:]):
                assert f0 + c0 == f1
            counts = [c for _, c in spans]
            assert max(counts) - min(counts) <= 1 and counts == sorted(counts, reverse=True)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(0)                     # same data on every rank
        d, h = 8, 16
        W1, W2 = rng.normal(size=(h, d)), rng.normal(size=(d, h))
        x = rng.normal(size=(n, d))
        first, count = S.token_shard(n, world, rank)
        y = O.dense_ffn(x[first:first + count], W1, W2)    # any token-wise function will do
        np.save(os.path.join(out_dir, "y%d.npy" % rank), y)
        slowest = S.max_over_ranks(10.0 + rank)
        total = S.sum_over_ranks(count)
        assert slowest == 10.0 + world - 1 and total == n
        dist.barrier()
        if rank == 0:
            parts = [np.load(os.path.join(out_dir, "y%d.npy" % r)) for r in range(world)]
            np.testing.assert_allclose(np.concatenate(parts, 0), O.dense_ffn(x, W1, W2), rtol=0, atol=1e-12)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce(tmp_path):
    mp.spawn(_worker, args=(2, _free_port(), 13, str(tmp_path)), nprocs=2, join=True)

"""The N > 1 path on CPU: two gloo ranks shard the batch, each estimates dW from its own samples with
the same probes (computed here by the oracle), and the all-reduced sum equals the full-batch estimate."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2106_06998_b200 import dp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import xconv_oracle as O
    g = np.random.Generator(np.random.PCG64(5))
    B, Cin, Cout, H, W, r = 7, 3, 4, 5, 6, 9                     # odd batch: shards of 4 and 3
    X = g.standard_normal((B, Cin, H, W)); dY = g.standard_normal((B, Cout, H, W))
    Z = g.standard_normal((r, Cin, H, W))                        # same probes on every rank
    lo, hi = dp.batch_shard(B, rank, world)
    S_local = O.sketch(X[lo:hi], Z)
    dW = torch.from_numpy(O.wgrad_estimate(S_local, dY[lo:hi], Z))
    dp.allreduce_dw(dW)
    full = O.wgrad_estimate(O.sketch(X, Z), dY, Z)
    out[rank] = float(np.abs(dW.numpy() - full).max() / np.abs(full).max())
    dist.destroy_process_group()


def test_two_rank_batch_sharding_sums_to_the_full_batch_estimate():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        assert len(out) == world and all(v < 1e-12 for v in out.values()), dict(out)


def test_batch_shards_partition_the_batch():
    for B in (1, 7, 512):
        for world in (1, 2, 3, 8):
            edges = [dp.batch_shard(B, k, world) for k in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == B
            assert all(edges[k][1] == edges[k + 1][0] for k in range(world - 1))
            sizes = [b - a for a, b in edges]
            assert max(sizes) - min(sizes) <= 1


def test_allreduce_is_a_noop_without_a_process_group():
    t = torch.ones(3)
    assert dp.allreduce_dw(t) is t and float(t.sum()) == 3.0

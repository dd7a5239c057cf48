"""Host logic of the multi-GPU path on CPU: two gloo ranks each verify their slice of a batch
(the oracle stands in for the device step), gather, and must reproduce the unsharded result."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2512_13194_b200.shard import shard_range
from paper_2512_13194_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, K, V, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    _, t, d, x = synth.tiny_inputs(B, K, V, "fp32", seed=3)
    lo, n = shard_range(B, rank, world)
    r = oracle.verify(t[lo:lo + n], d[lo:lo + n], x[lo:lo + n], 1.0, 0.1, seed=4, offset=9, b_first=lo)
    mine = torch.full((B, K + 2), -7, dtype=torch.int32)
    mine[lo:lo + n, 0] = torch.from_numpy(r.accept_len)
    mine[lo:lo + n, 1:] = torch.from_numpy(r.tokens)
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    ms = torch.tensor([float(rank + 1)])
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)      # the bench's max-over-ranks timing
    if rank == 0:
        full = torch.full((B, K + 2), -7, dtype=torch.int32)
        for rr, p in enumerate(parts):
            a, c = shard_range(B, rr, world)
            full[a:a + c] = p[a:a + c]
        np.save(out_path, np.concatenate([full.numpy().ravel(), [int(ms.item())]]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_full_batch(tmp_path):
    B, K, V, world = 7, 3, 500, 2
    out = str(tmp_path / "gathered.npy")
    mp.spawn(_worker, args=(world, _free_port(), B, K, V, out), nprocs=world, join=True)
    got = np.load(out)
    assert got[-1] == world
    got = got[:-1].reshape(B, K + 2)
    _, t, d, x = synth.tiny_inputs(B, K, V, "fp32", seed=3)
    ref = oracle.verify(t, d, x, 1.0, 0.1, seed=4, offset=9)
    assert np.array_equal(got[:, 0], ref.accept_len)
    assert np.array_equal(got[:, 1:], ref.tokens)

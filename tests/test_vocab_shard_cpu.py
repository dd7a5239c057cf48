"""The vocabulary-sharded form on CPU: its numpy oracle must reproduce the unsharded C oracle for
any split (shard invariance: the pin of oracle/sharded.py), and two gloo ranks driving
``verify_vocab_sharded`` with the real communicator must do the same."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from oracle.sharded import OracleShardStep
from paper_2512_13194_b200 import synth
from paper_2512_13194_b200.shard import TorchDistComm, verify_vocab_sharded, vocab_range


class LocalComm:
    """All shards in one process, run in lockstep."""
    def __init__(self, size):
        self.size = size


def run_lockstep(steps):
    all_stats = torch.stack([s.stats() for s in steps])
    all_mass = torch.stack([s.decide(all_stats) for s in steps])
    outs = [s.pick(r, all_stats, all_mass) for r, s in enumerate(steps)]
    acc = outs[0][0]
    for a, _ in outs[1:]:
        assert torch.equal(a, acc)
    tok = torch.stack([t for _, t in outs]).max(0).values
    return acc, tok, outs


def split_points(V, cuts):
    edges = [0] + sorted(cuts) + [V]
    return [(a, b - a) for a, b in zip(edges[:-1], edges[1:])]


@pytest.mark.parametrize("cuts", [[], [37], [1, 150], [64, 65, 190]])
@pytest.mark.parametrize("beta,noise", [(0.0, 2.0), (0.5, 1.0)])
def test_sharded_oracle_reproduces_the_unsharded_one(cuts, beta, noise):
    B, K, V, T = 40, 3, 200, 0.9
    _, t, d, x = synth.tiny_inputs(B, K, V, "fp32", seed=31, noise=noise, temperature=T)
    t = t.clone(); d = d.clone(); x = x.clone()
    t[0, 0, 10:90] = float("-inf"); d[0, 0, 10:90] = float("-inf"); x[0, 0] = 5   # masked columns, one shard nearly empty
    t[1, 1, :] = float("-inf")         # invalid sequence
    x[2, 0] = V                        # invalid token
    t[3, 2, 7] = float("nan")
    ref = oracle.verify(t, d, x, T, beta, seed=5, offset=2, b_first=11)
    steps = [OracleShardStep(t[:, :, a:a + n], d[:, :, a:a + n], x, a, V, T, beta, seed=5, offset=2, b_first=11)
             for a, n in split_points(V, cuts)]
    acc, tok, outs = run_lockstep(steps)
    assert np.array_equal(acc.numpy(), ref.accept_len)
    assert np.array_equal(tok.numpy(), ref.tokens)
    assert (ref.accept_len[1:4] == -1).all() and (ref.accept_len >= 0).sum() >= B - 3
    # exactly one shard owns each final token
    final = torch.stack([t_[torch.arange(B), acc.clamp(min=0).long()] for _, t_ in outs])
    owners = (final >= 0).sum(0)
    assert torch.equal(owners[acc >= 0], torch.ones_like(owners[acc >= 0]))
    if beta == 0.0:
        assert (ref.accept_len[4:] < K).mean() > 0.3      # the residual draw is exercised
    else:
        assert (ref.accept_len[4:] == K).any()            # and the bonus draw


def test_vocab_range_covers_the_vocabulary():
    for V, n in ((32000, 2), (32001, 3), (128256, 8), (64, 4), (152064, 5)):
        parts = [vocab_range(V, r, n) for r in range(n)]
        assert parts[0][0] == 0 and sum(c for _, c in parts) == V
        for (a, c), (a2, _) in zip(parts[:-1], parts[1:]):
            assert a + c == a2 and c % 8 == 0
    with pytest.raises(ValueError):
        vocab_range(3, 0, 4)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, K, V, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    _, t, d, x = synth.tiny_inputs(B, K, V, "fp32", seed=8, noise=1.5)
    a, n = vocab_range(V, rank, world)
    step = OracleShardStep(t[:, :, a:a + n], d[:, :, a:a + n], x, a, V, 1.1, 0.2, seed=4, offset=9)
    acc, tok = verify_vocab_sharded(step, TorchDistComm())
    np.save(f"{out_path}.{rank}.npy", np.concatenate([acc.numpy().ravel(), tok.numpy().ravel()]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_step(tmp_path):
    B, K, V, world = 9, 3, 500, 2
    out = str(tmp_path / "sharded")
    mp.spawn(_worker, args=(world, _free_port(), B, K, V, out), nprocs=world, join=True)
    _, t, d, x = synth.tiny_inputs(B, K, V, "fp32", seed=8, noise=1.5)
    ref = oracle.verify(t, d, x, 1.1, 0.2, seed=4, offset=9)
    want = np.concatenate([ref.accept_len.ravel(), ref.tokens.ravel()])
    for rank in range(world):
        assert np.array_equal(np.load(f"{out}.{rank}.npy"), want)   # every rank holds the full result

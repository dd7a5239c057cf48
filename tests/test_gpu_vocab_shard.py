"""The vocabulary-sharded step (ears_shard_stats / _decide / _pick) through the C ABI against the
UNSHARDED oracle on the concatenated rows.  The shards of a step run one after another on one
device, phase by phase, and the test performs the exchanges (a stack of the small results): the
kernels of different shards never wait for one another, so this is the multi-device data path
itself, minus the transport."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from paper_2512_13194_b200 import synth
from paper_2512_13194_b200.shard import vocab_range
from oracle.parity import Tally, assert_parity, compare

pytestmark = pytest.mark.gpu


def split_points(V, cuts):
    edges = [0] + sorted(cuts) + [V]
    return [(a, b - a) for a, b in zip(edges[:-1], edges[1:])]


def run_sharded(ears, t, d, x, parts, V, T, beta, seed, offset, b_first=0):
    dev = "cuda:0"
    xg = x.to(dev)
    steps = [ears.ShardStep(t[:, :, a:a + n].contiguous().to(dev), d[:, :, a:a + n].contiguous().to(dev), xg, a, V,
                            T, beta, seed, offset, b_first) for a, n in parts]
    all_stats = torch.stack([s.stats() for s in steps])
    all_mass = torch.stack([s.decide(all_stats) for s in steps])
    outs = [s.pick(r, all_stats, all_mass) for r, s in enumerate(steps)]
    torch.cuda.synchronize()
    acc = outs[0][0].cpu()
    for a, _ in outs[1:]:
        assert torch.equal(a.cpu(), acc), "accept lengths differ between shards"
    toks = torch.stack([tk.cpu() for _, tk in outs])
    return acc, toks.max(0).values, toks, all_mass.cpu()


CASES = [
    # B, K, V, dtype, cuts
    (3, 2, 9, "fp32", [4]), (4, 3, 1025, "bf16", [512]), (2, 2, 4097, "fp32", [1000, 1001, 3000]),
    (5, 4, 32000, "bf16", [16000]), (6, 3, 32001, "fp16", [8000, 16000, 24000]), (40, 3, 70001, "fp32", [35000]),
    (300, 2, 700, "bf16", [350]), (3, 64, 2051, "fp32", [1024]), (2, 1, 300000, "bf16", [100000, 200000]),
    # enough rows for the warp-per-row statistics kernel, aligned and unaligned columns
    (3000, 2, 704, "bf16", [352]), (3000, 2, 523, "fp32", [260]),
]


@pytest.mark.parametrize("B,K,V,dtype,cuts", CASES)
def test_sharded_parity_shapes(ears, B, K, V, dtype, cuts):
    tally = Tally()
    for i, (T, beta, noise) in enumerate([(1.0, 0.0, 2.0), (0.8, 0.3, 1.0), (1.3, 1.0, 0.5)]):
        w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=500 + i, temperature=T, noise=noise)
        acc, tok, toks, _ = run_sharded(ears, t, d, x, split_points(V, cuts), V, T, beta, seed=i, offset=3 * i)
        ora = oracle.verify(t, d, x, T, beta, seed=i, offset=3 * i)
        tally.merge(compare(acc.numpy(), tok.numpy(), ora, K, inputs=(t, d, T)))
        # one shard at most writes a sequence's final token
        n = acc.clamp(min=0).long()
        owners = (toks[:, torch.arange(B), n] >= 0).sum(0)
        assert (owners[acc >= 0] == 1).all()
    assert_parity(tally, max_explained=max(1, int(np.ceil(1e-4 * tally.rows))))


def test_sharded_agrees_with_the_single_device_step(ears):
    """Same inputs through ears.verify and through 1, 2 and 4 shards: the same lengths and tokens
    except where the oracle flags a near-tie; and one shard alone is the whole step."""
    w = replace(synth.workload(2), B=64)
    t, d, x = synth.make_inputs(w, "cpu")
    ora = oracle.verify(t, d, x, w.temperature, 0.25, seed=2, offset=5, nthreads=oracle.max_threads())
    acc0, tok0 = ears.verify(t.cuda(), d.cuda(), x.cuda(), w.temperature, 0.25, 2, 5)
    tl = compare(acc0.cpu().numpy(), tok0.cpu().numpy(), ora, w.K, inputs=(t, d, w.temperature))
    for n in (1, 2, 4):
        parts = [vocab_range(w.V, r, n) for r in range(n)]
        acc, tok, _, mass = run_sharded(ears, t, d, x, parts, w.V, w.temperature, 0.25, seed=2, offset=5)
        tl.merge(compare(acc.numpy(), tok.numpy(), ora, w.K, inputs=(t, d, w.temperature)))
        assert (mass.sum(0)[acc >= 0] > 0).all()
    assert_parity(tl)


@pytest.mark.parametrize("dtype", ["fp32", "bf16", "fp16"])
def test_sharded_invalid_sequences_and_masked_columns(ears, dtype):
    B, K, V = 10, 3, 5000
    w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=9)
    t = t.clone(); d = d.clone(); x = x.clone()
    x[1, 0] = V
    x[2, 2] = -3
    t[3, 1, 77] = float("nan")         # odd lane of a packed pair (2-byte types)
    d[4, 0, 4999] = float("inf")
    t[5, 3, :] = float("-inf")
    t[7, 2, 2578] = float("nan")       # even lane, second shard
    t[0, 0, 0:2500] = float("-inf")    # a whole shard of a row masked: legal
    d[0, 0, 0:2500] = float("-inf")
    x[0, 0] = 2600
    t[6, 1, 2500:] = float("-inf")     # the other shard of another row
    d[6, 1, 2500:] = float("-inf")
    x[6, 1] = 17
    ora = oracle.verify(t, d, x, 1.0, 0.1, seed=1, offset=2)
    assert ora.accept_len[[1, 2, 3, 4, 5, 7]].tolist() == [-1] * 6 and (ora.accept_len[[0, 6, 8, 9]] >= 0).all()
    acc, tok, _, _ = run_sharded(ears, t, d, x, [(0, 2500), (2500, 2500)], V, 1.0, 0.1, seed=1, offset=2)
    assert_parity(compare(acc.numpy(), tok.numpy(), ora, K, inputs=(t, d, 1.0)), max_explained=0)


@pytest.mark.parametrize("idx,B,n", [(3, 32, 2), (4, 48, 4), (5, 24, 8)])
def test_sharded_parity_workload_rows(ears, idx, B, n):
    """Rows of workloads 3-5 split over 2, 4 and 8 shards with vocab_range."""
    w = replace(synth.workload(idx), B=B)
    t, d, x = synth.make_inputs(w, "cpu")
    parts = [vocab_range(w.V, r, n) for r in range(n)]
    tally = Tally()
    for offset, beta in enumerate([w.beta, 0.0]):
        acc, tok, _, _ = run_sharded(ears, t, d, x, parts, w.V, w.temperature, beta, seed=w.verify_seed, offset=offset,
                                     b_first=100)
        ora = oracle.verify(t, d, x, w.temperature, beta, seed=w.verify_seed, offset=offset, b_first=100,
                            nthreads=oracle.max_threads())
        tally.merge(compare(acc.numpy(), tok.numpy(), ora, w.K, inputs=(t, d, w.temperature)))
    assert_parity(tally)


def test_shard_argument_errors(ears):
    w, t, d, x = synth.tiny_inputs(2, 2, 64, "fp32", seed=1)
    dev = "cuda:0"
    with pytest.raises(ears.EarsError) as e:
        ears.ShardStep(t.to(dev), d.to(dev), x.to(dev), 10, 70, 1.0, 0.1).stats()     # columns run past V
    assert e.value.status == -2
    with pytest.raises(ears.EarsError) as e:
        ears.ShardStep(t.to(dev), d.to(dev), x.to(dev), 0, 64, 0.0, 0.1).stats()      # temperature 0
    assert e.value.status == -3

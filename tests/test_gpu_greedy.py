"""The temperature -> 0 form (ears_verify_greedy) through the C ABI against the oracle: bit-exact
(integers only: top tokens, lengths)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_13194_b200 import synth

pytestmark = pytest.mark.gpu


def make(B, K, V, dtype, seed, miss=0.25):
    """Target rows with ties sprinkled in, draft tokens that mostly hit the top token."""
    w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=seed)
    g = torch.Generator().manual_seed(seed)
    if V > 4:
        rows = torch.randint(0, B * (K + 1), (max(1, B // 2),), generator=g)
        flat = t.view(-1, V)
        for r in rows.tolist():                       # exact ties for the top place: the first index must win
            top = flat[r].float().max()
            idx = torch.randint(0, V, (3,), generator=g)
            flat[r, idx] = (top + 1).to(flat.dtype)
    am = t.float().argmax(-1)                         # torch returns some maximal index; the oracle decides
    x = am[:, :K].to(torch.int32).clone()
    flip = torch.rand((B, K), generator=g) < miss
    x[flip] = torch.randint(0, V, (int(flip.sum()),), generator=g, dtype=torch.int32)
    return t, x


@pytest.mark.parametrize("B,K,V,dtype", [
    (1, 1, 1, "fp32"), (2, 3, 7, "bf16"), (3, 2, 1023, "fp32"), (2, 2, 4097, "bf16"), (4, 5, 32000, "fp32"),
    (3, 4, 32001, "bf16"), (6, 7, 128256, "bf16"), (1, 64, 515, "fp32"), (700, 2, 130, "fp32"), (2, 1, 1000003, "fp32"),
    (2, 3, 7, "fp16"), (2, 2, 4097, "fp16"), (6, 7, 128256, "fp16"), (300, 2, 1400, "fp16"),
])
def test_greedy_parity_shapes(ears, B, K, V, dtype):
    t, x = make(B, K, V, dtype, seed=B + K + V)
    acc, tok = ears.verify_greedy(t.cuda(), x.cuda())
    torch.cuda.synchronize()
    assert ears.last_device_status() == 0
    o_acc, o_tok, _ = oracle.verify_greedy(t, x)
    assert np.array_equal(acc.cpu().numpy(), o_acc)
    assert np.array_equal(tok.cpu().numpy(), o_tok)
    if B * K >= 64:
        assert (o_acc < K).any()


@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_greedy_parity_workloads(ears, idx):
    w = synth.workload(idx)
    t, d, x = synth.make_inputs(w, "cpu")
    am = t.float().argmax(-1)[:, :w.K].to(torch.int32)
    g = torch.Generator().manual_seed(idx)
    keep = torch.rand(am.shape, generator=g) < 0.8
    xx = torch.where(keep, am, x)
    acc, tok = ears.verify_greedy(t.cuda(), xx.cuda())
    o_acc, o_tok, _ = oracle.verify_greedy(t, xx)
    assert np.array_equal(acc.cpu().numpy(), o_acc) and np.array_equal(tok.cpu().numpy(), o_tok)


@pytest.mark.parametrize("dtype", ["fp32", "bf16", "fp16"])
def test_greedy_invalid_sequences_are_marked(ears, dtype):
    """NaN in an odd and an even lane of a packed pair (2-byte types), +inf, a fully masked row,
    tokens out of range: each marks its own sequence only."""
    t, x = make(10, 3, 5000, dtype, seed=5)
    t[1, 2, 77] = float("nan")                        # odd lane
    t[2, 0, 4999] = float("inf")
    t[3, 3, :] = float("-inf")
    x[4, 1] = 5000
    x[5, 0] = -1
    t[6, 1, 78] = float("nan")                        # even lane
    top = int(t[7, 0].float().argmax())
    t[7, 0, top ^ 1] = float("nan")                   # beside the row's top entry
    t[0, 0, 10:500] = float("-inf")                   # masked entries are legal
    dev = "cuda:0"
    acc, tok = ears.verify_greedy(t.to(dev), x.to(dev))
    torch.cuda.synchronize()
    assert ears.last_device_status() & ears.DEV_INVALID_INPUT
    o_acc, o_tok, _ = oracle.verify_greedy(t, x)
    assert o_acc[1:8].tolist() == [-1] * 7 and (o_acc[[0, 8, 9]] >= 0).all()
    assert np.array_equal(acc.cpu().numpy(), o_acc) and np.array_equal(tok.cpu().numpy(), o_tok)


def test_greedy_workspace_and_repeats(ears):
    dev = "cuda:0"
    # caller workspace, repeated calls, clean status afterwards
    t2, x2 = make(8, 3, 5000, "bf16", seed=6)
    ws = torch.empty(ears.workspace_bytes(8, 3, 5000) + 256, dtype=torch.uint8, device=dev)
    ws = ws[(-ws.data_ptr()) % 256:]
    ref = oracle.verify_greedy(t2, x2)
    for rep in range(3):
        a, k = ears.verify_greedy(t2.to(dev), x2.to(dev), workspace=ws if rep % 2 else None)
        torch.cuda.synchronize()
        assert np.array_equal(a.cpu().numpy(), ref[0]) and np.array_equal(k.cpu().numpy(), ref[1])
    assert ears.last_device_status() == 0
    with pytest.raises(ears.EarsError):
        ears.verify_greedy(t2.to(dev), x2.to(dev), workspace=ws[:256])

"""The sampler object (the plug-in form of Sec. 3.3 item 4) driven for several steps against the
oracle at the matching offsets."""
import numpy as np
import pytest
import torch

import oracle
from oracle.parity import Tally, assert_parity, compare
from paper_2512_13194_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("uncertainty", ["maxprob", "entropy"])
def test_sampler_steps_match_the_oracle(ears, uncertainty):
    dev = "cuda:0"
    B, K, V = 12, 4, 20000
    s = ears.EarsSampler(temperature=0.9, beta=0.2, seed=41, first_offset=100, uncertainty=uncertainty,
                         report_entropy=uncertainty == "entropy")
    tally = Tally()
    total = 0
    for step in range(4):
        w, t, d, x = synth.tiny_inputs(B, K, V, "bf16", seed=900 + step, noise=1.0, temperature=0.9)
        res = s(t.to(dev), d.to(dev), x.to(dev))
        assert res.offset == 100 + step and s.offset == 101 + step
        ora = oracle.verify(t, d, x, 0.9, 0.2, seed=41, offset=100 + step, nthreads=8, uncertainty=uncertainty)
        tally.merge(compare(res.accept_len.cpu().numpy(), res.tokens.cpu().numpy(), ora, K, inputs=(t, d, 0.9)))
        if uncertainty == "entropy":
            np.testing.assert_allclose(res.entropy.cpu().numpy(), ora.entropy, rtol=1e-5, atol=5e-7)
        for n, row, em in zip(res.accept_len.tolist(), res.tokens.tolist(), res.emitted()):
            assert em == row[:n + 1] and len(em) == n + 1
        total += int(ora.accept_len.sum())
    assert_parity(tally, max_explained=1)
    if not tally.explained:
        assert abs(s.mean_accept_len() - total / (4 * B)) < 1e-12
    assert s.state() == {"seed": 41, "offset": 104, "steps": 4}


def test_sampler_with_per_sequence_parameters_and_replay(ears):
    dev = "cuda:0"
    B, K, V = 9, 3, 9000
    Ts = torch.linspace(0.6, 1.4, B)
    betas = torch.tensor([0.0, 0.1, 0.5] * 3)
    s = ears.EarsSampler(temperature=Ts.to(dev), beta=betas.to(dev), seed=7, first_offset=3, b_first=20)
    w, t, d, x = synth.tiny_inputs(B, K, V, "fp32", seed=950, noise=1.0)
    first = s(t.to(dev), d.to(dev), x.to(dev))
    ora = oracle.verify(t, d, x, 1.0, 0.0, seed=7, offset=3, b_first=20, seq_temperature=Ts.numpy(), seq_beta=betas.numpy())
    assert_parity(compare(first.accept_len.cpu().numpy(), first.tokens.cpu().numpy(), ora, K, inputs=(t, d, Ts.numpy())),
                  max_explained=1)
    # a second sampler started from the recorded state reproduces the step
    again = ears.EarsSampler(temperature=Ts.to(dev), beta=betas.to(dev), seed=7, first_offset=first.offset, b_first=20)
    rep = again(t.to(dev), d.to(dev), x.to(dev))
    assert torch.equal(rep.accept_len, first.accept_len) and torch.equal(rep.tokens, first.tokens)

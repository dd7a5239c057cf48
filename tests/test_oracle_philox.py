"""Pins for the oracle's random stream: published Philox4x32-10 known answers
(tests/golden/philox4x32_10_kat.txt) and the layout of the uniforms drawn from it."""
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], tuple(w[6:10])))
    return rows


def test_published_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert oracle.philox4x32_10(ctr, key) == want


def test_accept_uniform_is_top_24_bits_of_word0():
    for seed, offset, b, k in [(0, 0, 0, 0), (42, 7, 1, 4), (2**63 + 5, 2**40 + 3, 511, 2)]:
        w = oracle.philox4x32_10((offset & 0xFFFFFFFF, offset >> 32, b, k), (seed & 0xFFFFFFFF, seed >> 32))
        u = oracle.uniform_accept(seed, offset, b, k)
        assert u == (w[0] >> 8) / 2.0**24
        assert 0.0 <= u < 1.0
        assert np.float32(u) == u  # exactly representable in fp32: both sides hold the same number


def test_final_uniform_is_top_53_bits_of_words01():
    for seed, offset, b, K in [(0, 0, 0, 4), (9, 1, 3, 5), (2**64 - 1, 2**64 - 1, 127, 7)]:
        w = oracle.philox4x32_10((offset & 0xFFFFFFFF, offset >> 32, b, K), (seed & 0xFFFFFFFF, seed >> 32))
        u = oracle.uniform_final(seed, offset, b, K)
        assert u == (((w[0] << 32) | w[1]) >> 11) / 2.0**53
        assert 0.0 <= u < 1.0


def test_streams_are_distinct_and_uniform():
    n = 20000
    u = np.array([oracle.uniform_accept(3, 11, b, 0) for b in range(n)])
    v = np.array([oracle.uniform_accept(3, 11, b, 1) for b in range(n)])
    w = np.array([oracle.uniform_accept(3, 12, b, 0) for b in range(n)])
    f = np.array([oracle.uniform_final(3, 11, b, 2) for b in range(n)])
    for a in (u, v, w, f):
        assert abs(a.mean() - 0.5) < 5 * np.sqrt(1 / 12 / n)
        assert abs(a.var() - 1 / 12) < 0.005
        hist = np.histogram(a, bins=16, range=(0, 1))[0]
        assert ((hist - n / 16) ** 2 / (n / 16)).sum() < 45  # chi2, 15 dof, p ~ 1e-4
    assert abs(np.corrcoef(u, v)[0, 1]) < 0.04
    assert abs(np.corrcoef(u, w)[0, 1]) < 0.04
    assert len(set(u.tolist())) > 0.99 * n

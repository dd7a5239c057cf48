"""Pins for the fp64 oracle against what the paper and the mathematics fix.

Each test names the passage it rests on.  Expected values are computed here with
library routines (scipy softmax, numpy cumsum/searchsorted) or closed forms, never
by calling the oracle on itself.
"""
import numpy as np
import pytest
from scipy import stats
from scipy.special import softmax as sp_softmax

import oracle

EPS = 1e-10


def tile(rows_t, rows_d, toks, B):
    """Same (target, draft, tokens) for B sequences; only the random counters differ."""
    t = np.broadcast_to(np.asarray(rows_t, np.float32), (B,) + np.shape(rows_t)).copy()
    d = np.broadcast_to(np.asarray(rows_d, np.float32), (B,) + np.shape(rows_d)).copy()
    x = np.broadcast_to(np.asarray(toks, np.int32), (B, len(toks))).copy()
    return t, d, x


def closed_form_accept(t_rows, d_rows, toks, T, beta):
    """a_k = min(1, R_k + beta (1 - max P_t)): the acceptance region [0, R + Tol] of Sec. 3.2."""
    a = []
    for k, tok in enumerate(toks):
        pt = sp_softmax(np.asarray(t_rows[k], np.float64) / T)
        pd = sp_softmax(np.asarray(d_rows[k], np.float64) / T)
        R = pt[tok] / max(pd[tok], EPS)
        a.append(min(1.0, R + beta * (1.0 - pt.max())))
    return np.array(a)


# --------------------------------------------------------------------------- softmax
def test_softmax_matches_library_routine():
    rng = np.random.default_rng(1)
    for V, T in [(7, 1.0), (1000, 0.7), (32000, 1.3)]:
        l = rng.normal(0, 3, V)
        p, m, Z = oracle.softmax(l, T)
        np.testing.assert_allclose(p, sp_softmax(l / T), rtol=1e-12, atol=0)
        assert m == l.max()
        assert abs(p.sum() - 1) < 1e-12
        assert abs(p.max() - 1.0 / Z) < 1e-15  # max P = exp(0)/Z: what the GPU path relies on
        p2, _, _ = oracle.softmax(l + 123.25, T)  # shift invariance
        np.testing.assert_allclose(p2, p, rtol=1e-9)


def test_softmax_masked_and_bad_rows():
    p, _, _ = oracle.softmax([0.0, -np.inf, 1.0], 1.0)
    assert p[1] == 0.0 and abs(p.sum() - 1) < 1e-15
    for bad in ([0.0, np.nan], [np.inf, 0.0], [-np.inf, -np.inf]):
        with pytest.raises(ValueError):
            oracle.softmax(bad, 1.0)


# ----------------------------------------------------------------------- inverse CDF
def test_inverse_cdf_matches_searchsorted():
    rng = np.random.default_rng(2)
    for V in (1, 2, 8, 1000):
        r = rng.random(V)
        r[rng.random(V) < 0.3] = 0.0
        if r.sum() == 0:
            r[0] = 1.0
        C = np.cumsum(r)
        for u in rng.random(200):
            got = oracle.inverse_cdf(r, u)
            want = int(np.searchsorted(C, u * C[-1], side="right"))
            assert got["token"] == want
            assert r[want] > 0
            assert got["lo"] <= u < got["hi"] + 1e-15


def test_inverse_cdf_hand_cases():
    r = [0.0, 0.25, 0.0, 0.5, 0.25, 0.0]
    assert oracle.inverse_cdf(r, 0.0)["token"] == 1          # u = 0 -> first positive mass
    assert oracle.inverse_cdf(r, 0.2499999)["token"] == 1
    assert oracle.inverse_cdf(r, 0.25)["token"] == 3         # boundary belongs to the next token (strict <)
    assert oracle.inverse_cdf(r, 0.75)["token"] == 4
    assert oracle.inverse_cdf(r, 1.0 - 2.0**-53)["token"] == 4
    assert oracle.inverse_cdf([0, 0, 0], 0.5)["token"] == -1
    near = oracle.inverse_cdf(r, 0.25 + 1e-9, band=1e-6)
    assert (near["token"], near["band_lo"], near["band_hi"]) == (3, 1, 3)


def test_inverse_cdf_band_width_is_the_stated_one():
    """The band lists the tokens whose CDF interval comes within `band` of u: a neighbour whose
    interval ends 5e-6 from u is outside at band 1e-6 and inside at band 1e-5, on either side of u;
    a band ten times too wide (or too narrow) fails one of these."""
    r = [0.25, 0.25, 0.5]                                   # boundaries at 0.25 and 0.5
    below = oracle.inverse_cdf(r, 0.25 + 5e-6, band=1e-6)   # token 0 ends 5e-6 below u
    assert (below["token"], below["band_lo"], below["band_hi"]) == (1, 1, 1)
    below = oracle.inverse_cdf(r, 0.25 + 5e-6, band=1e-5)
    assert (below["token"], below["band_lo"], below["band_hi"]) == (1, 0, 1)
    above = oracle.inverse_cdf(r, 0.5 - 5e-6, band=1e-6)    # token 2 starts 5e-6 above u
    assert (above["token"], above["band_lo"], above["band_hi"]) == (1, 1, 1)
    above = oracle.inverse_cdf(r, 0.5 - 5e-6, band=1e-5)
    assert (above["token"], above["band_lo"], above["band_hi"]) == (1, 1, 2)
    # just inside and just outside the stated width, both sides
    assert oracle.inverse_cdf(r, 0.25 + 0.9e-6, band=1e-6)["band_lo"] == 0
    assert oracle.inverse_cdf(r, 0.25 + 1.1e-6, band=1e-6)["band_lo"] == 1
    assert oracle.inverse_cdf(r, 0.5 - 0.9e-6, band=1e-6)["band_hi"] == 2
    assert oracle.inverse_cdf(r, 0.5 - 1.1e-6, band=1e-6)["band_hi"] == 1
    # the band is in probability units, not in units of mass: scaling the masses changes nothing
    scaled = oracle.inverse_cdf([250.0, 250.0, 500.0], 0.25 + 5e-6, band=1e-5)
    assert (scaled["token"], scaled["band_lo"], scaled["band_hi"]) == (1, 0, 1)
    # zero-mass tokens may sit between the ends of a band but are never its ends
    gap = oracle.inverse_cdf([0.25, 0.0, 0.0, 0.25, 0.5], 0.25 + 1e-9, band=1e-6)
    assert (gap["token"], gap["band_lo"], gap["band_hi"]) == (3, 0, 3)


def test_cdf_margin_is_the_distance_to_the_nearer_interval_end():
    """verify() reports min(u - lo, hi - u) of the drawn token's interval.  Bonus draw from
    P_t = (1/4, 1/4, 1/2) (identical rows: everything accepted); u comes from the pinned Philox
    stream, the interval ends are known by hand."""
    K, V = 2, 3
    row = np.log(np.array([1.0, 1.0, 2.0])).astype(np.float32)
    t = np.broadcast_to(row, (64, K + 1, V)).copy()
    d = np.broadcast_to(row, (64, K, V)).copy()
    x = np.zeros((64, K), np.int32)
    res = oracle.verify(t, d, x, 1.0, 0.0, seed=12, offset=34)
    assert (res.accept_len == K).all()
    edges = np.array([0.0, 0.25, 0.5, 1.0])
    seen = set()
    for b in range(64):
        u = oracle.uniform_final(12, 34, b, K)
        j = int(np.searchsorted(edges, u, side="right")) - 1
        assert res.tokens[b, K] == j
        want = min(u - edges[j], edges[j + 1] - u)
        assert abs(res.cdf_margin[b] - want) < 1e-7, (b, u, res.cdf_margin[b], want)
        assert res.band_lo[b] == res.band_hi[b] == j or want < 1e-6
        seen.add(j)
    assert seen == {0, 1, 2}


def test_compare_refuses_a_zero_mass_token_inside_the_band():
    """The parity helper accepts a token disagreement only when the other token lies in the oracle's
    band AND has mass in the oracle's row.  Planted here: a 'GPU' answer that differs from the
    oracle's by a zero-mass token inside the band (refused), by the positive-mass neighbour (accepted)
    and by a token outside the band (refused)."""
    from oracle.parity import compare
    K, V = 1, 6
    # P_t = (1/4, 0, 0, 1/4, 1/2, 0) on the extra row; tokens 1, 2, 5 are masked out
    row = np.array([0.0, -np.inf, -np.inf, 0.0, np.log(2.0), -np.inf], np.float32)
    t = np.broadcast_to(row, (1, K + 1, V)).copy()
    d = np.broadcast_to(row, (1, K, V)).copy()
    x = np.zeros((1, K), np.int32)
    # find a (seed, offset) whose final uniform falls just above the boundary at 0.25
    hit = None
    for off in range(200000):
        u = oracle.uniform_final(3, off, 0, K)
        if 0.25 < u < 0.25 + 1e-6:
            hit = off
            break
    if hit is None:      # no such draw among these offsets: plant the band through a wide one instead
        hit, band = 0, 1.0
    else:
        band = 1e-6
    ora = oracle.verify(t, d, x, 1.0, 0.0, seed=3, offset=hit, band=band)
    n = int(ora.accept_len[0])
    assert n == K
    o = int(ora.tokens[0, n])
    lo, hi = int(ora.band_lo[0]), int(ora.band_hi[0])
    assert lo <= 0 and hi >= 3                  # the band spans tokens 0..3, of which 1 and 2 have no mass
    inputs = (t, d, 1.0)

    def gpu_answer(g):
        tok = ora.tokens.copy()
        tok[0, n] = g
        return compare(ora.accept_len.copy(), tok, ora, K, inputs=inputs)

    other = 0 if o == 3 else 3
    ok = gpu_answer(other)
    assert ok.explained_tokens == 1 and not ok.unexplained
    for zero in (1, 2):
        bad = gpu_answer(zero)
        assert bad.explained_tokens == 0 and bad.unexplained and bad.unexplained[0][1] == "token-zero-mass"
    out = gpu_answer(5)
    assert out.unexplained and out.unexplained[0][1] in ("token", "token-zero-mass")
    # without the inputs nothing can be explained
    tok = ora.tokens.copy()
    tok[0, n] = other
    assert compare(ora.accept_len.copy(), tok, ora, K).unexplained[0][1] == "token-unchecked"
    # and an exact match is clean
    clean = compare(ora.accept_len.copy(), ora.tokens.copy(), ora, K, inputs=inputs)
    assert not clean.unexplained and clean.explained == 0


# -------------------------------------------------- closed-form acceptance probability
@pytest.mark.parametrize("beta,T", [(0.0, 1.0), (0.1, 0.9), (0.5, 1.3), (1.0, 1.0)])
def test_acceptance_probability_closed_form(beta, T):
    """P(accept position k) = min(1, R_k + Tol_k) for U uniform (Sec. 3.2, acceptance region)."""
    rng = np.random.default_rng(3)
    K, V, B = 3, 6, 200_000
    t_rows = rng.normal(0, 1.5, (K + 1, V))
    d_rows = t_rows[:K] + rng.normal(0, 1.0, (K, V))
    toks = [1, 4, 2]
    t, d, x = tile(t_rows, d_rows, toks, B)
    res = oracle.verify(t, d, x, T, beta, seed=5, offset=9, nthreads=4)
    # float32 storage of the rows: recompute the closed form from what the oracle saw
    a = closed_form_accept(t[0], d[0], toks, np.float32(T), np.float32(beta))
    emp = (res.cls != 0).mean(axis=0)
    sigma = np.sqrt(np.maximum(a * (1 - a), 1e-12) / B)
    assert np.all(np.abs(emp - a) < 5 * sigma + 1e-9), (emp, a)
    # first-rejection logic (Sec. 3.1): P(n = j) = prod_{i<j} a_i * (1 - a_j)
    pn = np.array([np.prod(a[:j]) * (1 - a[j]) for j in range(K)] + [np.prod(a)])
    counts = np.bincount(res.accept_len, minlength=K + 1)
    keep = pn * B > 5
    chi = ((counts[keep] - pn[keep] * B) ** 2 / (pn[keep] * B)).sum()
    assert chi < stats.chi2.ppf(1 - 1e-5, max(keep.sum() - 1, 1)), (counts, pn * B)
    assert counts[~keep].sum() <= 5 * (pn[~keep].sum() * B + 2)


# ------------------------------------------------------------- output law, tiny vocab
def _law(pt, pd, beta):
    """Law of the token emitted at position 0 when x ~ P_d (refs [1],[2] with the EARS region)."""
    a = np.minimum(1.0, pt / np.maximum(pd, EPS) + beta * (1 - pt.max()))
    res = np.maximum(pt - pd, 0.0)
    rej = (pd * (1 - a)).sum()
    return pd * a + (rej * res / res.sum() if res.sum() > 0 else 0.0)


@pytest.mark.parametrize("V,beta", [(4, 0.0), (8, 0.0), (8, 0.3)])
def test_emitted_token_law_brute_force(V, beta):
    """beta = 0 is standard speculative sampling, whose output law is exactly P_t
    (Sec. 3.2 step 5 'identical to traditional'; refs [1],[2]); beta > 0 follows the
    same enumeration with the widened acceptance region."""
    rng = np.random.default_rng(40 + V)
    B, T = 1_000_000, 1.0
    t_rows = rng.normal(0, 1.2, (2, V)).astype(np.float32)
    d_rows = (t_rows[:1] + rng.normal(0, 1.0, (1, V))).astype(np.float32)
    pt = sp_softmax(t_rows[0].astype(np.float64))
    pd = sp_softmax(d_rows[0].astype(np.float64))
    law = _law(pt, pd, beta)
    assert abs(law.sum() - 1) < 1e-12
    if beta == 0.0:
        np.testing.assert_allclose(law, pt, atol=1e-12)  # algebraic identity
    x = rng.choice(V, size=(B, 1), p=pd).astype(np.int32)  # the draft model's own sampling
    t = np.broadcast_to(t_rows, (B, 2, V)).copy()
    d = np.broadcast_to(d_rows, (B, 1, V)).copy()
    res = oracle.verify(t, d, x, T, beta, seed=77, offset=1, nthreads=4)
    counts = np.bincount(res.tokens[:, 0], minlength=V)
    chi, p = stats.chisquare(counts, law * B)
    assert p > 1e-4, (chi, p, counts / B, law)
    # prefix property: an accepted sequence repeats the draft token
    acc = res.accept_len == 1
    assert np.array_equal(res.tokens[acc, 0], x[acc, 0])
    # a resampled token differs from the rejected one and has P_t > P_d there
    rej = ~acc
    assert np.all(res.tokens[rej, 0] != x[rej, 0])
    assert np.all(pt[res.tokens[rej, 0]] > pd[res.tokens[rej, 0]])
    assert np.all(res.tokens[rej, 1] == -1)


def test_bonus_token_law():
    """All drafts accepted (identical rows give R = 1): the extra token follows P_t of row K."""
    rng = np.random.default_rng(6)
    B, K, V, T = 400_000, 2, 8, 0.8
    t_rows = rng.normal(0, 1.5, (K + 1, V)).astype(np.float32)
    t, d, x = tile(t_rows, t_rows[:K], [3, 5], B)
    res = oracle.verify(t, d, x, T, 0.0, seed=1, offset=2, nthreads=4)
    assert np.all(res.accept_len == K)
    assert np.all(res.tokens[:, :K] == x)
    law = sp_softmax(t_rows[K].astype(np.float64) / np.float32(T))
    chi, p = stats.chisquare(np.bincount(res.tokens[:, K], minlength=V), law * B)
    assert p > 1e-4, (chi, p)
    np.testing.assert_allclose(res.resid_mass, 1.0, atol=1e-12)


# ------------------------------------------------------------------- tolerance term
def test_one_hot_target_gives_zero_tolerance():
    """max P_t = 1 makes Uncertainty = 0, so every beta decides like beta = 0 (Sec. 3.2)."""
    rng = np.random.default_rng(7)
    B, K, V = 2000, 3, 50
    t = rng.normal(0, 1, (B, K + 1, V)).astype(np.float32)
    hot = rng.integers(0, V, (B, K + 1))
    np.put_along_axis(t, hot[..., None], 800.0, axis=2)
    d = rng.normal(0, 1, (B, K, V)).astype(np.float32)
    x = np.where(rng.random((B, K)) < 0.5, hot[:, :K], rng.integers(0, V, (B, K))).astype(np.int32)
    base = oracle.verify(t, d, x, 1.0, 0.0, seed=3)
    assert np.all(base.max_pt == 1.0)
    for beta in (0.2, 1.0, 50.0):
        r = oracle.verify(t, d, x, 1.0, beta, seed=3)
        assert np.array_equal(r.cls != 0, base.cls != 0)
        assert np.array_equal(r.margin, base.margin)
        assert np.array_equal(r.tokens, base.tokens)
        assert not np.any(r.cls == 2)  # no pardon without tolerance


def test_accept_sets_nested_in_beta():
    """Tolerance is proportional to beta, so with the same uniforms the accepted set only grows."""
    rng = np.random.default_rng(8)
    B, K, V = 500, 5, 300
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = (t[:, :K] + rng.normal(0, 1.5, (B, K, V))).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    prev = None
    for beta in (0.0, 0.05, 0.1, 0.2, 0.5, 1.0, 2.0):
        r = oracle.verify(t, d, x, 1.0, beta, seed=11, offset=4)
        if prev is not None:
            assert np.all((prev.cls != 0) <= (r.cls != 0))
            assert np.all(prev.accept_len <= r.accept_len)
            assert np.array_equal(prev.cls == 1, r.cls == 1)  # the direct path ignores beta
        prev = r
    assert np.any(prev.cls == 2)


def test_tolerance_grows_with_temperature():
    """Higher temperature flattens P_t, lowers max P_t and so raises the tolerance (Sec. 4.3)."""
    rng = np.random.default_rng(9)
    B, K, V = 20, 2, 500
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = rng.normal(0, 2, (B, K, V)).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    prev = None
    for T in (0.5, 0.9, 1.0, 1.5, 3.0):
        r = oracle.verify(t, d, x, T, 0.1)
        if prev is not None:
            assert np.all(r.max_pt < prev.max_pt)
        prev = r


def test_clamp_is_inert_and_eps_guard_applies():
    """Sec. 3.3 item 2: threshold max(U - Tol, 0) and P_d^safe = max(P_d, 1e-10)."""
    rng = np.random.default_rng(10)
    B, K, V, beta = 5000, 1, 16, 1.0
    t = rng.normal(0, 0.3, (B, K + 1, V)).astype(np.float32)   # flat target: Tol close to beta
    d = rng.normal(0, 0.3, (B, K, V)).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    r = oracle.verify(t, d, x, 1.0, beta, seed=2)
    U = np.array([oracle.uniform_accept(2, 0, b, 0) for b in range(B)])
    tol = beta * (1 - r.max_pt[:, 0])
    clamped = U - tol < 0
    assert clamped.sum() > 100
    assert np.all(r.cls[clamped, 0] != 0)                       # R >= 0 always clears a zero threshold
    R = r.pt_tok[:, 0] / np.maximum(r.pd_tok[:, 0], EPS)
    np.testing.assert_allclose(r.margin[clamped, 0], R[clamped], rtol=1e-12)
    np.testing.assert_allclose(r.margin[~clamped, 0], (R - (U - tol))[~clamped], rtol=1e-9, atol=1e-12)
    # a draft token whose draft probability is below eps: R uses eps, not P_d
    t1 = np.zeros((1, 2, 4), np.float32)
    t1[0, 0] = [0.0, 0.0, 0.0, -30.0]                           # P_t(tok 3) ~ 3e-14
    d1 = np.zeros((1, 1, 4), np.float32)
    d1[0, 0, 3] = -60.0                                         # P_d(tok 3) ~ 3e-27 < eps
    r1 = oracle.verify(t1, d1, np.array([[3]], np.int32), 1.0, 0.0, seed=0)
    assert r1.pd_tok[0, 0] < 1e-20
    U0 = oracle.uniform_accept(0, 0, 0, 0)
    assert abs((r1.margin[0, 0] + U0) - r1.pt_tok[0, 0] / EPS) < 1e-12
    assert r1.accept_len[0] == 0                                # unguarded R = 1e13 would have accepted


# ----------------------------------------------------------------------- invariants
def test_invariants_on_random_batch():
    rng = np.random.default_rng(12)
    B, K, V, T, beta = 300, 4, 777, 1.1, 0.1
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = (t[:, :K] + rng.normal(0, 1.0, (B, K, V))).astype(np.float32)
    x = np.stack([[rng.choice(V, p=sp_softmax(d[b, k].astype(np.float64) / T)) for k in range(K)]
                  for b in range(B)]).astype(np.int32)
    r = oracle.verify(t, d, x, T, beta, seed=21, offset=3)
    assert r.accept_len.min() >= 0 and r.accept_len.max() <= K
    assert 0 < (r.accept_len < K).sum() < B
    for b in range(B):
        n = r.accept_len[b]
        assert np.array_equal(r.tokens[b, :n], x[b, :n])
        assert np.all(r.tokens[b, n + 1:] == -1)
        assert 0 <= r.tokens[b, n] < V
        # decisions recomputed from library softmax and the published uniform layout
        for k in range(K):
            pt = sp_softmax(t[b, k].astype(np.float64) / np.float32(T))
            pd = sp_softmax(d[b, k].astype(np.float64) / np.float32(T))
            np.testing.assert_allclose(r.pt_tok[b, k], pt[x[b, k]], rtol=1e-11)
            np.testing.assert_allclose(r.pd_tok[b, k], pd[x[b, k]], rtol=1e-11)
            np.testing.assert_allclose(r.max_pt[b, k], pt.max(), rtol=1e-12)
        u = oracle.uniform_final(21, 3, b, K)
        if n < K:
            pt = sp_softmax(t[b, n].astype(np.float64) / np.float32(T))
            pd = sp_softmax(d[b, n].astype(np.float64) / np.float32(T))
            S = 0.5 * np.abs(pt - pd).sum()                      # total-variation identity
            np.testing.assert_allclose(r.resid_mass[b], S, rtol=1e-10)
            R = pt[x[b, n]] / pd[x[b, n]]
            assert r.resid_mass[b] >= pd[x[b, n]] * (1 - R) - 1e-15
            assert r.tokens[b, n] != x[b, n] and pt[r.tokens[b, n]] > pd[r.tokens[b, n]]
            mass = np.maximum(pt - pd, 0)
        else:
            mass = sp_softmax(t[b, K].astype(np.float64) / np.float32(T))
        C = np.cumsum(mass)
        want = int(np.searchsorted(C, u * C[-1], side="right"))
        if r.cdf_margin[b] > 1e-9:                               # away from a boundary the pick is unique
            assert r.tokens[b, n] == want
        else:
            assert r.band_lo[b] <= want <= r.band_hi[b]
    # first rejection = first position whose class is 0
    first = np.array([np.argmax(np.append(r.cls[b] == 0, True)) for b in range(B)])
    assert np.array_equal(first, r.accept_len)
    # shifting every row by a constant changes nothing
    r2 = oracle.verify(t + np.float32(8.0), d - np.float32(4.0), x, T, beta, seed=21, offset=3)
    assert np.array_equal(r2.accept_len, r.accept_len)
    assert (r2.tokens != r.tokens).mean() < 0.01   # +8 in fp32 re-rounds the logits slightly
    # threads do not change results
    r3 = oracle.verify(t, d, x, T, beta, seed=21, offset=3, nthreads=4)
    assert np.array_equal(r3.tokens, r.tokens) and np.array_equal(r3.margin, r.margin)


def test_identical_rows_accept_everything():
    rng = np.random.default_rng(13)
    B, K, V = 50, 6, 100
    t = rng.normal(0, 3, (B, K + 1, V)).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    r = oracle.verify(t, t[:, :K].copy(), x, 0.9, 0.0, seed=5)
    assert np.all(r.accept_len == K) and np.all(r.cls == 1)
    np.testing.assert_allclose(r.pt_tok, r.pd_tok, rtol=0, atol=0)


def test_batch_shards_reproduce_the_full_batch():
    """The random counter carries the global sequence index, so shards agree with the whole."""
    rng = np.random.default_rng(14)
    B, K, V = 12, 3, 64
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = (t[:, :K] + rng.normal(0, 1.5, (B, K, V))).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    full = oracle.verify(t, d, x, 1.0, 0.1, seed=9, offset=100)
    for lo, hi in [(0, 5), (5, 12)]:
        part = oracle.verify(t[lo:hi], d[lo:hi], x[lo:hi], 1.0, 0.1, seed=9, offset=100, b_first=lo)
        assert np.array_equal(part.tokens, full.tokens[lo:hi])
        assert np.array_equal(part.accept_len, full.accept_len[lo:hi])
    other = oracle.verify(t, d, x, 1.0, 0.1, seed=9, offset=101)
    assert not np.array_equal(other.margin, full.margin)


def test_bf16_rows_widen_exactly():
    import torch
    g = torch.Generator().manual_seed(0)
    B, K, V = 4, 2, 200
    t = torch.randn(B, K + 1, V, generator=g).to(torch.bfloat16)
    d = torch.randn(B, K, V, generator=g).to(torch.bfloat16)
    x = torch.randint(0, V, (B, K), generator=g).to(torch.int32)
    a = oracle.verify(t, d, x, 1.0, 0.2, seed=1)
    b = oracle.verify(t.float(), d.float(), x, 1.0, 0.2, seed=1)
    assert np.array_equal(a.tokens, b.tokens) and np.array_equal(a.pt_tok, b.pt_tok)


def test_fp16_bits_widen_like_the_library_conversion():
    """All 65536 binary16 patterns against numpy's float16 -> float64 conversion; fp16 rows give the
    same step as the same values held in fp32."""
    import torch
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.half_to_double(int(b)) for b in bits])
    assert np.array_equal(np.isnan(want), np.isnan(got))
    ok = ~np.isnan(want)
    assert np.array_equal(want[ok], got[ok]) and np.array_equal(np.signbit(want[ok]), np.signbit(got[ok]))
    g = torch.Generator().manual_seed(3)
    B, K, V = 4, 2, 200
    t = (3 * torch.randn(B, K + 1, V, generator=g)).to(torch.float16)
    d = (3 * torch.randn(B, K, V, generator=g)).to(torch.float16)
    t[0, 1, 5] = float("-inf")
    t[1, 0, 7] = 6e-8   # subnormal in binary16
    x = torch.randint(0, V, (B, K), generator=g).to(torch.int32)
    a = oracle.verify(t, d, x, 0.9, 0.2, seed=1)
    b = oracle.verify(t.float(), d.float(), x, 0.9, 0.2, seed=1)
    c = oracle.verify(t.numpy(), d.numpy(), x, 0.9, 0.2, seed=1)
    assert np.array_equal(a.tokens, b.tokens) and np.array_equal(a.pt_tok, b.pt_tok) and np.array_equal(a.margin, b.margin)
    assert np.array_equal(a.tokens, c.tokens) and np.array_equal(a.pt_tok, c.pt_tok)


def test_invalid_sequences_are_marked_not_fatal():
    rng = np.random.default_rng(15)
    B, K, V = 6, 2, 32
    t = rng.normal(0, 1, (B, K + 1, V)).astype(np.float32)
    d = rng.normal(0, 1, (B, K, V)).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    good = oracle.verify(t, d, x, 1.0, 0.1)
    x[1, 0] = V
    x[2, 1] = -1
    t[3, 1, 5] = np.nan
    d[4, 0, 7] = np.inf
    t[5, K, :] = -np.inf
    t[0, 0, 3] = -np.inf  # a masked vocabulary entry is legal
    r = oracle.verify(t, d, x, 1.0, 0.1)
    assert np.all(r.accept_len[1:] == -1) and np.all(r.tokens[1:] == -1)
    assert r.accept_len[0] >= 0 and good.accept_len[0] >= 0
    with pytest.raises(ValueError):
        oracle.verify(t, d, x, 0.0, 0.1)
    with pytest.raises(ValueError):
        oracle.verify(t, d, x, 1.0, -0.1)


# --------------------------------------------------------------------------- per-sequence temperature and beta
def test_per_sequence_parameters_match_closed_forms_and_scalar_calls():
    """Sec. 3.3 item 3 treats sequences independently, so each may carry its own temperature
    (Sec. 4.3) and base tolerance (Sec. 3.2).  Pins: (i) probabilities of sequence b against a
    library softmax at T_b; (ii) the whole result of sequence b against a scalar call on that
    sequence alone with (T_b, beta_b) and the same global index; (iii) equal entries reproduce
    the scalar call; (iv) a value the scalar form refuses invalidates only its own sequence."""
    rng = np.random.default_rng(77)
    B, K, V = 6, 3, 50
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = (t[:, :K] + rng.normal(0, 0.8, (B, K, V))).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    Ts = np.array([0.5, 0.8, 1.0, 1.3, 2.0, 0.9], np.float32)
    betas = np.array([0.0, 0.1, 0.3, 0.05, 1.0, 0.2], np.float32)
    res = oracle.verify(t, d, x, 1.0, 0.1, seed=3, offset=9, b_first=4, seq_temperature=Ts, seq_beta=betas)
    for b in range(B):
        for k in range(K):
            pt = sp_softmax(t[b, k].astype(np.float64) / float(Ts[b]))
            pd = sp_softmax(d[b, k].astype(np.float64) / float(Ts[b]))
            assert res.pt_tok[b, k] == pytest.approx(pt[x[b, k]], rel=1e-12)
            assert res.pd_tok[b, k] == pytest.approx(pd[x[b, k]], rel=1e-12)
            U = oracle.uniform_accept(3, 9, 4 + b, k)
            thr = max(U - float(betas[b]) * (1.0 - pt.max()), 0.0)
            assert res.margin[b, k] == pytest.approx(pt[x[b, k]] / max(pd[x[b, k]], EPS) - thr, abs=1e-12)
        one = oracle.verify(t[b:b + 1], d[b:b + 1], x[b:b + 1], float(Ts[b]), float(betas[b]), seed=3, offset=9,
                            b_first=4 + b)
        assert one.accept_len[0] == res.accept_len[b]
        assert np.array_equal(one.tokens[0], res.tokens[b])
        assert one.resid_mass[0] == res.resid_mass[b]
    same = oracle.verify(t, d, x, 7.0, 7.0, seed=3, offset=9, seq_temperature=np.full(B, 0.9, np.float32),
                         seq_beta=np.full(B, 0.25, np.float32))
    ref = oracle.verify(t, d, x, np.float32(0.9), 0.25, seed=3, offset=9)
    assert np.array_equal(same.tokens, ref.tokens) and np.array_equal(same.margin, ref.margin)
    bad_T = Ts.copy(); bad_T[2] = 0.0; bad_T[4] = np.nan
    bad_b = betas.copy(); bad_b[1] = -0.5
    bad = oracle.verify(t, d, x, 1.0, 0.1, seed=3, offset=9, b_first=4, seq_temperature=bad_T, seq_beta=bad_b)
    assert bad.accept_len[[1, 2, 4]].tolist() == [-1, -1, -1] and (bad.tokens[[1, 2, 4]] == -1).all()
    for b in (0, 3, 5):
        assert bad.accept_len[b] == res.accept_len[b] and np.array_equal(bad.tokens[b], res.tokens[b])


# --------------------------------------------------------------------------- stopping at the first rejection
def test_stop_at_first_reject_reads_nothing_beyond_it():
    """Sec. 3.1: rejecting x_i rejects every later draft token, so their rows cannot influence the
    result.  Pins: identical lengths, tokens and masses as the full evaluation on clean data; data
    planted after the first rejection (NaN rows, tokens out of range, a broken extra row) changes
    nothing in this mode but invalidates the sequence in the full one; data planted at or before
    the first rejection invalidates it in both."""
    rng = np.random.default_rng(5)
    B, K, V = 40, 4, 30
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = (t[:, :K] + rng.normal(0, 1.5, (B, K, V))).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    full = oracle.verify(t, d, x, 1.0, 0.05, seed=2, offset=1)
    stop = oracle.verify(t, d, x, 1.0, 0.05, seed=2, offset=1, stop_at_first_reject=True)
    assert np.array_equal(full.accept_len, stop.accept_len) and np.array_equal(full.tokens, stop.tokens)
    assert np.array_equal(full.resid_mass, stop.resid_mass)
    n = full.accept_len
    assert (n < K).sum() > 10 and (n == K).sum() > 2 and (n < K - 1).sum() > 5
    for b in range(B):       # diagnostics exist up to the first rejection only
        upto = min(n[b] + 1, K)
        assert np.array_equal(stop.pt_tok[b, :upto], full.pt_tok[b, :upto])
        assert (stop.pt_tok[b, upto:] == 0).all()
    t2, d2, x2 = t.copy(), d.copy(), x.copy()
    early = [b for b in range(B) if n[b] < K - 1]
    for i, b in enumerate(early):
        k = n[b] + 1                      # a position after the first rejection
        if i % 3 == 0:
            t2[b, k, 3] = np.nan
        elif i % 3 == 1:
            x2[b, k] = V + 7
        else:
            d2[b, k, :] = -np.inf
    rej = [b for b in range(B) if n[b] < K]
    for b in rej[::2]:
        t2[b, K, 0] = np.inf              # the extra row is not needed after a rejection
    stop2 = oracle.verify(t2, d2, x2, 1.0, 0.05, seed=2, offset=1, stop_at_first_reject=True)
    full2 = oracle.verify(t2, d2, x2, 1.0, 0.05, seed=2, offset=1)
    assert np.array_equal(stop2.accept_len, full.accept_len) and np.array_equal(stop2.tokens, full.tokens)
    assert (full2.accept_len[early] == -1).all() and (full2.accept_len[rej[::2]] == -1).all()
    t3 = t.copy()
    for b in rej:
        t3[b, n[b], 1] = np.nan           # at the rejected position itself
    stop3 = oracle.verify(t3, d, x, 1.0, 0.05, seed=2, offset=1, stop_at_first_reject=True)
    assert (stop3.accept_len[rej] == -1).all()
    ok = [b for b in range(B) if n[b] == K]
    assert np.array_equal(stop3.tokens[ok], full.tokens[ok])


# --------------------------------------------------------------------------- the deterministic limit
def test_greedy_limit_matches_argmax_and_the_low_temperature_step():
    """Sec. 1 names temperature = 0 as the regime where plain verification works.  Pins of the
    greedy form: (i) its per-row choice is numpy's argmax (first index on ties); (ii) lengths and
    tokens follow from it by the first-mismatch rule; (iii) it is the limit of the stochastic step:
    with one-hot drafts (the draft token's logit far above the rest) and a temperature far below
    the gap between the two best target logits, the ordinary oracle gives the same lengths and
    tokens for any beta and any seed."""
    rng = np.random.default_rng(11)
    B, K, V = 30, 4, 40
    t = rng.normal(0, 3, (B, K + 1, V)).astype(np.float32)
    top2 = np.sort(t, axis=-1)[..., -2:]
    t[np.arange(B)[:, None], np.arange(K + 1)[None, :], t.argmax(-1)] += (top2[..., 1] - top2[..., 0] < 1.0) * 1.5   # clear winners
    am = t.argmax(-1)
    x = am[:, :K].astype(np.int32).copy()
    flip = rng.random((B, K)) < 0.3
    x[flip] = (x[flip] + 1 + rng.integers(0, V - 1, flip.sum())) % V            # some drafts miss
    acc, tok, am_o = oracle.verify_greedy(t, x)
    assert np.array_equal(am_o, am)
    for b in range(B):
        miss = np.nonzero(x[b] != am[b, :K])[0]
        n = int(miss[0]) if miss.size else K
        assert acc[b] == n
        assert tok[b, :n].tolist() == x[b, :n].tolist() and tok[b, n] == am[b, n] and (tok[b, n + 1:] == -1).all()
    assert (acc < K).sum() > 5 and (acc == K).sum() > 2
    d = np.full((B, K, V), -50.0, np.float32)
    d[np.arange(B)[:, None], np.arange(K)[None, :], x] = 50.0                     # greedy drafts: P_d(x) = 1
    for beta, seed in ((0.0, 1), (0.3, 2), (1.0, 3)):
        res = oracle.verify(t, d, x, 0.02, beta, seed=seed, offset=5)
        assert np.array_equal(res.accept_len, acc) and np.array_equal(res.tokens, tok)
    # ties go to the smallest index; invalid rows and tokens mark the sequence
    t2 = t.copy()
    t2[0, 0, :] = 0.0
    t2[0, 0, [7, 3, 9]] = 5.0
    assert oracle.verify_greedy(t2, x)[2][0, 0] == 3
    t2[1, 2, 5] = np.nan
    t2[2, K, :] = -np.inf
    x2 = x.copy()
    x2[3, 1] = V
    acc2, tok2, _ = oracle.verify_greedy(t2, x2)
    assert acc2[1:4].tolist() == [-1, -1, -1] and (tok2[1:4] == -1).all() and np.array_equal(acc2[4:], acc[4:])


# -------------------------------------------------- entropy as the uncertainty measure (Sec. 5 item 1)
def test_entropy_matches_library_routine_and_closed_forms():
    rng = np.random.default_rng(11)
    for V in (1, 2, 7, 1000):
        p = rng.random(V)
        p[rng.random(V) < 0.2] = 0.0
        if p.sum() == 0:
            p[0] = 1.0
        p /= p.sum()
        assert abs(oracle.entropy(p) - stats.entropy(p)) < 1e-12
    for V in (2, 8, 4096):
        assert abs(oracle.entropy(np.full(V, 1.0 / V)) - np.log(V)) < 1e-12        # flat: ln V
        assert abs(oracle.entropy_uncertainty(np.log(V), V) - 1.0) < 1e-15
        one_hot = np.zeros(V)
        one_hot[V // 2] = 1.0
        assert oracle.entropy(one_hot) == 0.0                                       # one-hot: 0
    assert oracle.entropy_uncertainty(0.0, 1) == 0.0                                # a single entry leaves no doubt
    # two-point distribution: H = -q ln q - (1 - q) ln(1 - q)
    q = 0.2
    assert abs(oracle.entropy([q, 1 - q]) - (-q * np.log(q) - (1 - q) * np.log(1 - q))) < 1e-15


def test_entropy_output_matches_the_row_softmax():
    rng = np.random.default_rng(12)
    B, K, V = 5, 3, 300
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    t[0, 1, 10:200] = -np.inf                       # masked entries contribute nothing
    d = (t[:, :K] + rng.normal(0, 1, (B, K, V))).astype(np.float32)
    x = rng.integers(0, 10, (B, K)).astype(np.int32)
    for T in (0.7, 1.0, 1.6):
        res = oracle.verify(t, d, x, T, 0.3, seed=1, offset=2, want_entropy=True)
        for b in range(B):
            for k in range(K):
                p = sp_softmax(t[b, k].astype(np.float64) / np.float32(T))
                assert abs(res.entropy[b, k] - stats.entropy(p)) < 1e-10
    # the measure the paper prints is untouched by asking for the entropy
    a = oracle.verify(t, d, x, 1.0, 0.3, seed=1, offset=2)
    b_ = oracle.verify(t, d, x, 1.0, 0.3, seed=1, offset=2, want_entropy=True)
    assert np.array_equal(a.accept_len, b_.accept_len) and np.array_equal(a.tokens, b_.tokens)
    assert np.array_equal(a.margin, b_.margin)


@pytest.mark.parametrize("beta,T", [(0.1, 0.9), (0.5, 1.3), (1.0, 1.0)])
def test_acceptance_probability_closed_form_with_entropy(beta, T):
    """With the entropy measure the acceptance region is the printed one with the other uncertainty:
    P(accept position k) = min(1, R_k + beta H_k / ln V)."""
    rng = np.random.default_rng(13)
    K, V, B = 3, 6, 200_000
    t_rows = rng.normal(0, 1.5, (K + 1, V))
    d_rows = t_rows[:K] + rng.normal(0, 1.0, (K, V))
    toks = [1, 4, 2]
    t, d, x = tile(t_rows, d_rows, toks, B)
    res = oracle.verify(t, d, x, T, beta, seed=6, offset=1, nthreads=4, uncertainty="entropy")
    a = np.empty(K)
    for k in range(K):
        pt = sp_softmax(t[0, k].astype(np.float64) / np.float32(T))
        pd = sp_softmax(d[0, k].astype(np.float64) / np.float32(T))
        R = pt[toks[k]] / max(pd[toks[k]], 1e-10)
        a[k] = min(1.0, R + float(np.float32(beta)) * stats.entropy(pt) / np.log(V))
    emp = (res.cls != 0).mean(axis=0)
    sigma = np.sqrt(np.maximum(a * (1 - a), 1e-12) / B)
    assert np.all(np.abs(emp - a) < 5 * sigma + 1e-9), (emp, a)
    # and it differs from the printed measure on these rows (otherwise the test proves nothing)
    plain = closed_form_accept(t[0], d[0], toks, np.float32(T), np.float32(beta))
    assert np.abs(plain - a).max() > 0.01


def test_entropy_measure_one_hot_flat_and_monotone_in_beta():
    rng = np.random.default_rng(14)
    B, K, V = 40, 4, 50
    t = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = (t[:, :K] + rng.normal(0, 1.5, (B, K, V))).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    # accept sets are nested in beta
    prev = None
    for beta in (0.0, 0.05, 0.2, 0.5, 1.0):
        res = oracle.verify(t, d, x, 1.0, beta, seed=2, offset=3, uncertainty="entropy")
        acc = res.cls != 0
        if prev is not None:
            assert np.all(acc | ~prev)
            assert np.all(res.accept_len >= prev_len)
        prev, prev_len = acc, res.accept_len
    # beta = 0: the measure plays no role
    a = oracle.verify(t, d, x, 1.0, 0.0, seed=2, offset=3, uncertainty="entropy")
    b = oracle.verify(t, d, x, 1.0, 0.0, seed=2, offset=3)
    assert np.array_equal(a.accept_len, b.accept_len) and np.array_equal(a.tokens, b.tokens)
    # one-hot target rows: H = 0, zero tolerance whatever beta
    t1 = t.copy()
    t1[:, :, 7] += 400.0
    a = oracle.verify(t1, d, x, 1.0, 1.0, seed=2, offset=3, uncertainty="entropy")
    b = oracle.verify(t1, d, x, 1.0, 0.0, seed=2, offset=3, uncertainty="entropy")
    assert np.array_equal(a.accept_len, b.accept_len) and np.array_equal(a.cls, b.cls)
    assert np.all(a.entropy < 1e-100)
    # flat target rows: H = ln V, uncertainty 1, so beta = 1 accepts everything (R + 1 >= U)
    tf = np.zeros_like(t)
    a = oracle.verify(tf, d, x, 1.0, 1.0, seed=2, offset=3, uncertainty="entropy")
    assert np.all(a.accept_len == K) and np.allclose(a.entropy, np.log(V), atol=1e-12)

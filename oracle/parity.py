"""Comparison of the CUDA path's outputs with the oracle's, with the near-tie rules
(TEST INFRASTRUCTURE: the checker's side, like everything under oracle/).

accept lengths and tokens must be bit-exact except
  - a decision whose oracle margin |R - max(U - Tol, 0)| is below 1e-5, or
  - a final token that lies in the oracle's band of tokens whose CDF interval comes
    within 1e-6 (in probability) of the uniform AND carries mass in the oracle's own row
    (a token of zero mass is never a legitimate draw, wherever it sits in the band);
such explained disagreements are counted (one per sequence at most), anything else is
unexplained and fails.  Probabilities must agree to 1e-5 relative (or 1e-30 absolute:
fp32 cannot hold what fp64 underflows to).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import ears_oracle as _oracle

DECISION_BAND = 1e-5
CDF_BAND = 1e-6
PROB_RTOL = 1e-5
PROB_ATOL = 1e-30


@dataclass
class Tally:
    sequences: int = 0
    rows: int = 0
    explained_decisions: int = 0
    explained_tokens: int = 0
    unexplained: list = field(default_factory=list)
    flagged_decisions: int = 0     # oracle says near-tie, whether or not the GPU agreed
    flagged_tokens: int = 0
    max_rel_prob_err: float = 0.0

    @property
    def explained(self) -> int:
        return self.explained_decisions + self.explained_tokens

    def merge(self, o: "Tally") -> "Tally":
        self.sequences += o.sequences
        self.rows += o.rows
        self.explained_decisions += o.explained_decisions
        self.explained_tokens += o.explained_tokens
        self.unexplained += o.unexplained
        self.flagged_decisions += o.flagged_decisions
        self.flagged_tokens += o.flagged_tokens
        self.max_rel_prob_err = max(self.max_rel_prob_err, o.max_rel_prob_err)
        return self


def final_token_mass(inputs, b: int, n: int, K: int, token: int) -> float:
    """Mass the oracle's row gives `token` as the final token of sequence b after n acceptances:
    max(0, P_t - P_d) of position n after a rejection (P_t if that residual is empty, as in the
    oracle), P_t of the extra row when n = K.  inputs = (target_logits, draft_logits, temperature),
    temperature a scalar or a [B] array."""
    t, d, temperature = inputs
    V = t.shape[-1]
    if not 0 <= token < V:
        return 0.0
    T = float(np.asarray(temperature).reshape(-1)[b]) if np.ndim(temperature) else float(temperature)
    pt = _oracle.row_softmax(t, b * (K + 1) + n, V, T)
    if n >= K:
        return float(pt[token])
    pd = _oracle.row_softmax(d, b * K + n, V, T)
    r = np.maximum(pt - pd, 0.0)
    if r.sum() < 1e-300:
        return float(pt[token])
    return float(r[token])


def compare(gpu_len, gpu_tok, ora, K: int, stats=None, inputs=None) -> Tally:
    """gpu_len [B], gpu_tok [B,K+1] numpy int32; ora an oracle.OracleResult; stats the GPU's dict;
    inputs = (target_logits, draft_logits, temperature) as given to the oracle (CPU).  A token
    disagreement counts as explained only if the other token lies in the oracle's band and has
    positive mass in the oracle's row, which needs `inputs`; without them it stays unexplained."""
    gpu_len = np.asarray(gpu_len)
    gpu_tok = np.asarray(gpu_tok)
    B = gpu_len.shape[0]
    t = Tally(sequences=B, rows=B * (2 * K + 1))
    valid = ora.accept_len >= 0
    t.flagged_decisions = int((np.abs(ora.margin[valid]) < DECISION_BAND).sum())
    t.flagged_tokens = int((ora.cdf_margin[valid] < CDF_BAND).sum())
    for b in range(B):
        n_o, n_g = int(ora.accept_len[b]), int(gpu_len[b])
        if n_o < 0 or n_g < 0:
            if n_o != n_g or not np.all(gpu_tok[b] == -1):
                t.unexplained.append((b, "invalid-marking", n_o, n_g))
            continue
        if n_o != n_g:
            k0 = min(n_o, n_g)
            if abs(ora.margin[b, k0]) < DECISION_BAND:
                t.explained_decisions += 1
            else:
                t.unexplained.append((b, "decision", k0, float(ora.margin[b, k0]), n_o, n_g))
            continue
        n = n_o
        if not np.array_equal(gpu_tok[b, :n], ora.tokens[b, :n]) or not np.all(gpu_tok[b, n + 1:] == -1):
            t.unexplained.append((b, "prefix/padding", gpu_tok[b].tolist(), ora.tokens[b].tolist()))
            continue
        g, o = int(gpu_tok[b, n]), int(ora.tokens[b, n])
        if g != o:
            in_band = ora.band_lo[b] <= g <= ora.band_hi[b]
            if in_band and inputs is not None and final_token_mass(inputs, b, n, K, g) > 0.0:
                t.explained_tokens += 1
            else:
                why = "token" if not in_band else ("token-unchecked" if inputs is None else "token-zero-mass")
                t.unexplained.append((b, why, g, o, int(ora.band_lo[b]), int(ora.band_hi[b]),
                                      float(ora.cdf_margin[b])))
    if stats is not None:
        for key in ("pt_tok", "pd_tok", "max_pt"):
            got = np.asarray(stats[key], dtype=np.float64)[valid]
            want = getattr(ora, key)[valid]
            err = np.abs(got - want)
            rel = err / np.maximum(np.abs(want), 1e-300)
            bad = (rel > PROB_RTOL) & (err > PROB_ATOL)
            if bad.any():
                i = int(np.argmax(np.where(bad, rel, 0)))
                t.unexplained.append(("prob", key, float(got.flat[i]), float(want.flat[i])))
            ok = err > PROB_ATOL
            if ok.any():
                t.max_rel_prob_err = max(t.max_rel_prob_err, float(rel[ok].max()))
    return t


def assert_parity(t: Tally, max_explained=None):
    assert not t.unexplained, t.unexplained[:5]
    if max_explained is None:
        max_explained = max(1, int(np.ceil(1e-4 * t.rows)))
    assert t.explained <= max_explained, (t.explained, t.rows)

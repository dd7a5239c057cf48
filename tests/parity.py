"""Comparison of the CUDA path's outputs with the oracle's, with the near-tie rules.

accept lengths and tokens must be bit-exact except
  - a decision whose oracle margin |R - max(U - Tol, 0)| is below 1e-5, or
  - a final token that lies in the oracle's band of tokens whose CDF interval comes
    within 1e-6 (in probability) of the uniform;
such explained disagreements are counted (one per sequence at most), anything else is
unexplained and fails.  Probabilities must agree to 1e-5 relative (or 1e-30 absolute:
fp32 cannot hold what fp64 underflows to).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

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


def compare(gpu_len, gpu_tok, ora, K: int, stats=None) -> Tally:
    """gpu_len [B], gpu_tok [B,K+1] numpy int32; ora an oracle.OracleResult; stats the GPU's dict."""
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
            if ora.band_lo[b] <= g <= ora.band_hi[b]:
                t.explained_tokens += 1
            else:
                t.unexplained.append((b, "token", g, o, int(ora.band_lo[b]), int(ora.band_hi[b]),
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

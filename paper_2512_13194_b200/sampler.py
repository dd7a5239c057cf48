"""The verification step as the object a decoding loop holds (Sec. 3.3 item 4 describes EARS as a
pluggable sampler: it receives the target model's logits and the draft information of a step and
returns the accept / reject decisions).  No serving framework is needed or imported.

The object owns what must persist between steps -- the random stream's seed and offset (one offset
per verification step, see include/ears.h), the tolerance beta and the temperature, as scalars or
one value per sequence -- and leaves every computation to the C-ABI library: ``__call__`` marshals
one call of ``verify`` and advances the offset.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch

from . import binding


@dataclass
class StepResult:
    accept_len: torch.Tensor      # [B] int32: accepted draft tokens per sequence (-1: the sequence's data was unusable)
    tokens: torch.Tensor          # [B,K+1] int32: accepted prefix, then the resampled or bonus token, then -1
    offset: int                   # the random stream's offset this step used
    entropy: Optional[torch.Tensor] = None   # [B,K] float64 H(P_t) per position, when asked for

    def emitted(self):
        """Per sequence the tokens this step adds to its text (accepted drafts + the final token)."""
        out = []
        for n, row in zip(self.accept_len.tolist(), self.tokens.tolist()):
            out.append([] if n < 0 else row[:n + 1])
        return out


class EarsSampler:
    """EARS verification for a speculative-decoding loop.

    temperature, beta: floats, or float32 CUDA tensors [B] with one value per sequence (requests of
    a serving batch bring their own).  uncertainty: "maxprob" (1 - max P_t, Sec. 3.2) or "entropy"
    (H(P_t) / ln V, Sec. 5 item 1).  seed: the random stream of this sampler; the offset starts at
    ``first_offset`` and goes up by one per step, so that a run can be replayed from (seed, offset).
    b_first: global index of this rank's first sequence when a batch is sharded across GPUs.
    """

    def __init__(self, temperature=1.0, beta=0.1, *, seed: int = 0, first_offset: int = 0,
                 uncertainty: str = "maxprob", stop_at_first_reject: bool = False, b_first: int = 0,
                 report_entropy: bool = False):
        self.temperature, self.beta = temperature, beta
        self.seed, self.offset = int(seed), int(first_offset)
        self.uncertainty, self.stop_at_first_reject = uncertainty, bool(stop_at_first_reject)
        self.b_first, self.report_entropy = int(b_first), bool(report_entropy)
        self.steps = 0
        self.accepted = 0          # draft tokens accepted so far (read from the outputs on request only)
        self._pending = []         # accept_len tensors not yet folded into `accepted`

    @staticmethod
    def _split(value):
        """-> (scalar, per-sequence tensor or None)"""
        if isinstance(value, torch.Tensor):
            return 1.0, value
        return float(value), None

    def __call__(self, target_logits: torch.Tensor, draft_logits: torch.Tensor, draft_tokens: torch.Tensor,
                 stream=None) -> StepResult:
        """One verification step: target_logits [B,K+1,V], draft_logits [B,K,V], draft_tokens [B,K]
        (CUDA tensors).  Asynchronous on ``stream``; the returned tensors are ready once it is."""
        T, seq_T = self._split(self.temperature)
        beta, seq_beta = self._split(self.beta)
        out = binding.verify(target_logits, draft_logits, draft_tokens, T, beta if seq_beta is None else 0.0,
                             self.seed, self.offset, b_first=self.b_first, stream=stream,
                             seq_temperature=seq_T, seq_beta=seq_beta,
                             stop_at_first_reject=self.stop_at_first_reject, uncertainty=self.uncertainty,
                             entropy=self.report_entropy)
        res = StepResult(out[0], out[1], self.offset, out[2]["entropy"] if self.report_entropy else None)
        self.offset += 1
        self.steps += 1
        self._pending.append(res.accept_len)
        return res

    def mean_accept_len(self) -> float:
        """Mean accepted length over all steps so far (synchronises: it reads the outputs)."""
        for a in self._pending:
            self.accepted += int(a.clamp(min=0).sum())
            self._seqs = getattr(self, "_seqs", 0) + int((a >= 0).sum())
        self._pending = []
        return self.accepted / max(getattr(self, "_seqs", 0), 1)

    def state(self) -> dict:
        """What a replay needs."""
        return {"seed": self.seed, "offset": self.offset, "steps": self.steps}

"""Seeded synthetic inputs for the EARS verification step.

This module serves both the CUDA path and the CPU oracle in tests and in the
benchmark, so it holds none of the method's arithmetic: it only manufactures
logits and draft tokens with the shapes and value distributions of the five
workload configurations (they stand in for logits a target/draft model pair
would produce during serving; no model or dataset is involved).

Conventions: ``N(0, s)`` means standard deviation ``s``.  bf16 and fp16 tensors are made
in fp32 and rounded *before* the draft tokens are drawn, so every
consumer sees identical bits.  Draft tokens are drawn from the softmax of the
(rounded) draft logits at the call's temperature, as a draft model would.
Generation runs in fixed blocks of sequences so peak memory stays bounded and the
result for a given (config, seed, device type) does not depend on free memory.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Tuple

import torch

_BLOCK = 16  # sequences generated at a time
TORCH_DTYPES = {"fp32": torch.float32, "bf16": torch.bfloat16, "fp16": torch.float16}


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    K: int
    V: int
    dtype: str            # "fp32" | "bf16" | "fp16"
    temperature: float
    beta: float
    recipe: str           # which generator below
    data_seed: int
    verify_seed: int = 0
    temperatures: Tuple[float, ...] = ()   # sweep points (config 2)
    betas: Tuple[float, ...] = ()

    @property
    def rows(self) -> int:
        return self.B * (2 * self.K + 1)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "fp32" else 2

    @property
    def logit_bytes(self) -> int:
        return self.rows * self.V * self.elem_bytes

    def with_batch(self, B: int) -> "Workload":
        return replace(self, B=B)


WORKLOADS = (
    Workload("cfg1_B1_K4_V32000_fp32", 1, 4, 32000, "fp32", 1.0, 0.5, "gauss", 1001,
             ),
    Workload("cfg2_B8_K5_V32000_bf16", 8, 5, 32000, "bf16", 1.0, 0.5, "zipf_jitter", 1002,
             temperatures=(0.7, 1.0, 1.3), betas=(0.0, 0.25, 0.5, 1.0)),
    Workload("cfg3_B32_K7_V128256_bf16", 32, 7, 128256, "bf16", 1.0, 0.5, "peaked_flat", 1003),
    Workload("cfg4_B128_K4_V152064_bf16", 128, 4, 152064, "bf16", 1.0, 0.75, "zipf_rowtemp", 1004),
    Workload("cfg5_B512_K3_V256000_fp32", 512, 3, 256000, "fp32", 1.2, 1.0, "gauss_wide", 1005),
)


def workload(index: int) -> Workload:
    """index 1..5 as the configurations are numbered."""
    return WORKLOADS[index - 1]


def _zipf_logprobs(V: int, s: float, device) -> torch.Tensor:
    ranks = torch.arange(1, V + 1, dtype=torch.float64, device=device)
    w = ranks.pow(-s)
    return (w / w.sum()).log().to(torch.float32)


def _permuted_rows(base: torch.Tensor, nrows: int, gen) -> torch.Tensor:
    out = torch.empty((nrows, base.numel()), dtype=base.dtype, device=base.device)
    for r in range(nrows):
        out[r] = base[torch.randperm(base.numel(), generator=gen, device=base.device)]
    return out


def _block(w: Workload, nb: int, b0: int, gen, device):
    """fp32 target [nb,K+1,V] and draft [nb,K,V] for sequences b0..b0+nb."""
    K, V = w.K, w.V
    rn = lambda *shape: torch.randn(*shape, generator=gen, device=device, dtype=torch.float32)
    if w.recipe == "gauss":            # target N(0,2); draft = target + N(0,0.5)
        t = rn(nb, K + 1, V) * 2.0
        d = t[:, :K] + rn(nb, K, V) * 0.5
    elif w.recipe == "gauss_wide":     # target N(0,3); draft = target + N(0,1.2)
        t = rn(nb, K + 1, V) * 3.0
        d = t[:, :K] + rn(nb, K, V) * 1.2
    elif w.recipe == "zipf_jitter":    # Zipf(1.1) log-probs, permuted per row, + N(0,1); draft + N(0,0.7)
        base = _zipf_logprobs(V, 1.1, device)
        t = _permuted_rows(base, nb * (K + 1), gen).view(nb, K + 1, V) + rn(nb, K + 1, V)
        d = t[:, :K] + rn(nb, K, V) * 0.7
    elif w.recipe == "zipf_rowtemp":   # Zipf(1.0) log-probs / tau_row, tau ~ U[0.5,1.5]; draft = 0.8 t + N(0,0.8)
        base = _zipf_logprobs(V, 1.0, device)
        tau = 0.5 + torch.rand(nb * (K + 1), 1, generator=gen, device=device)
        t = (_permuted_rows(base, nb * (K + 1), gen) / tau).view(nb, K + 1, V)
        d = 0.8 * t[:, :K] + rn(nb, K, V) * 0.8
    elif w.recipe == "peaked_flat":    # even sequences peaked (top logit +8 over N(0,1)), odd flat N(0,0.5)
        t = rn(nb, K + 1, V)
        for i in range(nb):
            if (b0 + i) % 2 == 0:
                rows = t[i]
                j = torch.randint(0, V, (K + 1,), generator=gen, device=device)
                rows[torch.arange(K + 1, device=device), j] = -math.inf
                top = rows.max(dim=1).values
                rows[torch.arange(K + 1, device=device), j] = top + 8.0
            else:
                t[i] *= 0.5
        d = t[:, :K] + rn(nb, K, V)
    else:
        raise ValueError(w.recipe)
    return t, d


def make_inputs(w: Workload, device="cpu", temperature: float | None = None):
    """-> (target_logits [B,K+1,V], draft_logits [B,K,V], draft_tokens [B,K] int32) on `device`.

    Deterministic for a given workload, temperature and device type.
    """
    device = torch.device(device)
    T = w.temperature if temperature is None else float(temperature)
    tdt = TORCH_DTYPES[w.dtype]
    gen = torch.Generator(device=device)
    gen.manual_seed(w.data_seed)
    t_out = torch.empty((w.B, w.K + 1, w.V), dtype=tdt, device=device)
    d_out = torch.empty((w.B, w.K, w.V), dtype=tdt, device=device)
    x_out = torch.empty((w.B, w.K), dtype=torch.int32, device=device)
    for b0 in range(0, w.B, _BLOCK):
        nb = min(_BLOCK, w.B - b0)
        t, d = _block(w, nb, b0, gen, device)
        t_out[b0:b0 + nb] = t.to(tdt)
        d_r = d.to(tdt)
        d_out[b0:b0 + nb] = d_r
        probs = torch.softmax(d_r.to(torch.float32).view(nb * w.K, w.V) / T, dim=1)
        x = torch.multinomial(probs, 1, generator=gen).view(nb, w.K)
        x_out[b0:b0 + nb] = x.to(torch.int32)
    return t_out, d_out, x_out


def tiny_inputs(B: int, K: int, V: int, dtype: str = "fp32", seed: int = 0, scale: float = 2.0,
                noise: float = 0.5, temperature: float = 1.0, device="cpu"):
    """Small gaussian case of arbitrary shape (ragged V, edge sizes) for parity tests."""
    w = Workload(f"tiny_B{B}_K{K}_V{V}_{dtype}", B, K, V, dtype, temperature, 0.5, "gauss", seed)
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    tdt = TORCH_DTYPES[dtype]
    t = (torch.randn(B, K + 1, V, generator=gen, device=device) * scale)
    d = (t[:, :K] + torch.randn(B, K, V, generator=gen, device=device) * noise).to(tdt)
    t = t.to(tdt)
    probs = torch.softmax(d.to(torch.float32).view(B * K, V) / temperature, dim=1)
    x = torch.multinomial(probs, 1, generator=gen).view(B, K).to(torch.int32)
    return w, t, d, x

"""Partitions across GPUs.

Batch: sequences are independent, so a rank verifies a contiguous slice of the batch and passes
the slice's first global index as ``b_first``; no data-path collective is needed and results do
not depend on the split.

Vocabulary (tensor-parallel logits): every rank holds a contiguous range of columns of every row.
``verify_vocab_sharded`` drives the three local phases of a step object (``ShardStep`` of the CUDA
binding) and performs the two small exchanges and the final MAX between them through a
communicator; logits never move."""
from __future__ import annotations

from typing import Tuple


def shard_range(B: int, rank: int, world_size: int) -> Tuple[int, int]:
    """-> (first, count): contiguous, sizes differ by at most one, earlier ranks larger."""
    if world_size < 1 or not 0 <= rank < world_size or B < 0:
        raise ValueError("bad rank / world_size / B")
    base, extra = divmod(B, world_size)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def vocab_range(V: int, rank: int, world_size: int, multiple: int = 8) -> Tuple[int, int]:
    """-> (v_first, Vs): contiguous column ranges in rank order whose sizes are multiples of
    ``multiple`` (16-byte rows for 2-byte logits keep the vector loads) except the last."""
    if world_size < 1 or not 0 <= rank < world_size or V < world_size or multiple < 1:
        raise ValueError("bad rank / world_size / V")
    per = -(-V // world_size)
    per = -(-per // multiple) * multiple
    first = min(V, rank * per)
    count = min(V, first + per) - first if rank < world_size - 1 else V - first
    if count < 1:
        raise ValueError("vocabulary too small for this many ranks")
    return first, count


class TorchDistComm:
    """The two collectives the sharded step needs, over a ``torch.distributed`` process group
    (NCCL for device tensors, gloo for host tensors)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.size = dist.get_world_size(group)

    def all_gather(self, x):
        """x [...] -> [size, ...] with rank r's tensor at index r."""
        import torch
        out = [torch.empty_like(x) for _ in range(self.size)]
        self._dist.all_gather(out, x.contiguous(), group=self.group)
        return torch.stack(out)

    def all_reduce_max_(self, x):
        self._dist.all_reduce(x, op=self._dist.ReduceOp.MAX, group=self.group)
        return x


def verify_vocab_sharded(step, comm):
    """One verification step with the vocabulary split over ``comm.size`` ranks.  ``step`` is this
    rank's ``ShardStep`` (anything with ``stats()``, ``decide(all_stats)``, ``pick(rank, all_stats,
    all_mass)``).  -> (accept_len [B], tokens [B,K+1]), identical on every rank.

    Exchanged per step: 16 bytes per row, 8 bytes per sequence, and the 4 (K+1) bytes per sequence of
    the token array."""
    all_stats = comm.all_gather(step.stats())
    all_mass = comm.all_gather(step.decide(all_stats))
    accept_len, tokens = step.pick(comm.rank, all_stats, all_mass)
    comm.all_reduce_max_(tokens)
    return accept_len, tokens

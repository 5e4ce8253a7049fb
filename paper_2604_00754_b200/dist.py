"""Host-side helpers for running the path on several GPUs, one process per GPU.

The path shards over sequences with no exchange of activations: every (sequence, KV-head
group) is independent, and the permutation of sequence b at a layer is a pure function of
(seed, layer, b), so each rank regenerates exactly the permutations of the sequences it
owns.  The only cross-rank reduction in a batch split is the [2, Hq] gate-logit gradient,
which sums over sequences.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_range(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Half-open range of sequence indices owned by `rank` (contiguous, sizes differ by <= 1)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(B, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def allreduce_gate_grads(dgate: torch.Tensor, group=None) -> torch.Tensor:
    """Sums the per-rank gate-logit gradients in place (no-op without a process group)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(dgate, op=dist.ReduceOp.SUM, group=group)
    return dgate

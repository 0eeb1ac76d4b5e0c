"""Coordinate sharding for more than one GPU.

Every operation of Algorithm 1 is element-wise, so the simulated-workers path needs no exchange
step: rank r owns a contiguous, word-aligned range of coordinates of all M gradient and momentum
buffers and of the parameters, runs the same kernels on its slices, and the packed vote of the
whole model is the concatenation of the ranks' words. This module only computes ranges and
reduces timings; it holds none of the method's arithmetic.
"""

from __future__ import annotations

from typing import Sequence, Tuple

import torch


def shard_range(d: int, rank: int, world: int) -> Tuple[int, int]:
    """Half-open coordinate range [start, stop) of a rank. Starts are multiples of 32 (so packed
    words never straddle two ranks, and slices keep 128-byte alignment); ranges differ by at most
    one word; only the last non-empty range can end in a ragged word."""
    if world < 1 or not 0 <= rank < world or d < 0:
        raise ValueError("bad shard request")
    words = (d + 31) // 32
    base, extra = divmod(words, world)
    w0 = rank * base + min(rank, extra)
    w1 = w0 + base + (1 if rank < extra else 0)
    return min(d, 32 * w0), min(d, 32 * w1)


def shard_slices(tensors: Sequence[torch.Tensor], start: int, stop: int):
    return [t[start:stop] for t in tensors]


def word_range(start: int, stop: int) -> Tuple[int, int]:
    return start // 32, (stop + 31) // 32


def max_over_ranks(value: float, device=None) -> float:
    """Timing reduction used by the benchmark: the slowest rank defines the step time."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())

"""Splitting independent units (batch items, sequences) across ranks.

Every (batch item | sequence, value head) of the gated delta rule is an independent
recurrence, so multi-GPU execution is a partition with no data-path collective: each
rank runs the library on its own contiguous slice and keeps its own states.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def shard_range(n_units: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous balanced slice [lo, hi) of n_units for `rank` (first n % world ranks get one more)."""
    if world_size <= 0 or not (0 <= rank < world_size) or n_units < 0:
        raise ValueError("bad shard arguments")
    base, rem = divmod(n_units, world_size)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def shard_sequences(lengths: Sequence[int], world_size: int) -> List[List[int]]:
    """Longest-processing-time assignment of sequences to ranks by chunk count (the chain
    kernel's cost is the number of 64-token chunks); returns the sequence indices per rank."""
    order = sorted(range(len(lengths)), key=lambda i: -int(lengths[i]))
    load = [0] * world_size
    out: List[List[int]] = [[] for _ in range(world_size)]
    for i in order:
        r = min(range(world_size), key=lambda j: (load[j], j))
        out[r].append(i)
        load[r] += (int(lengths[i]) + 63) // 64
    for r in range(world_size):
        out[r].sort()
    return out

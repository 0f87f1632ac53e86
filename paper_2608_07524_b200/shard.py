"""Data-parallel sharding of a packed batch across GPUs.

Every (sequence, head) of the attention path is independent, so ranks need no data-path
collective: each rank takes whole sequences.  The assignment itself (longest first to the least
loaded rank, load = L^2, the imbalance the paper measures across devices in Section 2.3) is
computed by the library's dcp_shard_sequences; this module only reshapes its answer.
"""
from __future__ import annotations

from typing import List, Sequence

from . import binding


def shard_sequences(lengths: Sequence[int], world_size: int) -> List[List[int]]:
    """Indices of the sequences each rank owns, longest first; deterministic on every rank."""
    if world_size < 1:
        raise ValueError("world_size must be >= 1")
    rank_of, _ = binding.dcp_shard_sequences(lengths, world_size)
    owned: List[List[int]] = [[] for _ in range(world_size)]
    for i in sorted(range(len(lengths)), key=lambda i: (-int(lengths[i]), i)):      # presentation order only
        owned[rank_of[i]].append(i)
    return owned


def imbalance(lengths: Sequence[int], world_size: int) -> float:
    """max over ranks of work / mean work (1.0 = perfectly balanced), from the library's loads."""
    _, load = binding.dcp_shard_sequences(lengths, world_size)
    mean = sum(load) / len(load)
    return max(load) / mean if mean > 0 else 1.0

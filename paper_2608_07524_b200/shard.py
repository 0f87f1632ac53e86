"""Data-parallel sharding of a packed batch across GPUs.

Every (sequence, head) of the attention path is independent, so ranks need no data-path
collective: each rank takes whole sequences.  Sequences are dealt longest first to the rank with
the least accumulated work, work being L^2 (the attention cost) - the same imbalance the paper
measures across devices (Section 2.3), handled here by greedy longest-processing-time assignment.
"""
from __future__ import annotations

from typing import List, Sequence


def shard_sequences(lengths: Sequence[int], world_size: int) -> List[List[int]]:
    """Indices of the sequences each rank owns; deterministic on every rank."""
    if world_size < 1:
        raise ValueError("world_size must be >= 1")
    load = [0] * world_size
    owned: List[List[int]] = [[] for _ in range(world_size)]
    for i in sorted(range(len(lengths)), key=lambda i: (-int(lengths[i]), i)):
        r = min(range(world_size), key=lambda r: (load[r], r))
        owned[r].append(i)
        load[r] += int(lengths[i]) ** 2
    return owned


def imbalance(lengths: Sequence[int], owned: List[List[int]]) -> float:
    """max over ranks of work / mean work (1.0 = perfectly balanced)."""
    loads = [sum(int(lengths[i]) ** 2 for i in idx) for idx in owned]
    mean = sum(loads) / len(loads)
    return max(loads) / mean if mean > 0 else 1.0

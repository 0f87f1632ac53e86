"""Oracle for the assignment of sequences to ranks (longest-processing-time-first on L^2).

TEST INFRASTRUCTURE ONLY: plain Python, exact integers.  The paper gives no algorithm for this (its
Section 2.3 only names the imbalance: per-device work differs because sequence lengths do, and
attention work grows with L^2); the rule is the classical greedy one, taken step by step:
  1. order the sequences by length, longest first, equal lengths by index;
  2. give each in turn to the rank whose accumulated load is smallest, the lowest rank on ties;
  3. a sequence of length L adds L^2 to its rank's load.
Pins (tests/test_shard_gloo.py): a hand-worked case, the partition property, and Graham's bound
against the exhaustive optimum on small inputs (makespan <= (4/3 - 1/(3m)) * optimum).
"""


def shard_lpt(lengths, world_size):
    """(rank_of list[n], load list[world_size])."""
    if world_size < 1:
        raise ValueError("world_size must be >= 1")
    load = [0] * world_size
    rank_of = [0] * len(lengths)
    for i in sorted(range(len(lengths)), key=lambda i: (-int(lengths[i]), i)):
        r = min(range(world_size), key=lambda r: (load[r], r))
        rank_of[i] = r
        load[r] += int(lengths[i]) ** 2
    return rank_of, load


def best_makespan(lengths, world_size):
    """Smallest possible maximum load over all world_size^n assignments (tiny inputs only)."""
    work = [int(L) ** 2 for L in lengths]
    best = [sum(work)]

    def go(i, load):
        if max(load) >= best[0]:
            return
        if i == len(work):
            best[0] = max(load)
            return
        seen = set()
        for r in range(world_size):
            if load[r] in seen:          # ranks with equal load are interchangeable
                continue
            seen.add(load[r])
            load[r] += work[i]
            go(i + 1, load)
            load[r] -= work[i]

    go(0, [0] * world_size)
    return best[0]

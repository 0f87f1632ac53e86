"""Oracle for the DCP-intra selection (Section 3.4, Algorithm 1, Eq. 1 and Eq. 4-6 of the paper).

TEST INFRASTRUCTURE ONLY: plain Python, exact rational arithmetic, exhaustive search.

What is selected.  Every candidate setting (batch size b, sequence-parallel size p) comes with four
profiled numbers taken with ALL layers recomputed: the forward time of one layer, the bytes one
layer keeps when it is not recomputed, the iteration time and the memory footprint.  Switching
recomputation off for `kept` of the n_layers layers adds kept * bytes_per_layer to the footprint
(Eq. 6) and removes kept * layer_fwd_time from the time (Eq. 5).  The selection is the pair
(candidate, kept) with the highest throughput b / (p * time) (Eq. 1) among all pairs whose
footprint stays within the capacity; the recompute count reported is n_layers - kept.

This file does not walk the candidates the way the paper's listing does.  It enumerates every
(candidate, kept) pair with kept = 0 .. n_layers, discards those that do not fit, and takes the
maximum, so that no early exit or closed form can hide a mistake.  For one candidate the time falls
as kept grows, hence the best pair of a candidate is the one with the most layers kept, which is
the smallest recompute count that fits: the quantity Section 3.4's text asks for.

Two readings (paper silent or at odds with itself):
  * taken literally, the listing's inner loop leaves at the first layer count that fits, i.e. it
    would never keep more than one layer; the accompanying text asks for the smallest recompute
    count under the capacity, which is what the maximum over all pairs yields;
  * the listing compares raw times across candidates, the text throughput; the two agree when b and
    p are equal, and throughput is used here.
Ties (the paper states none): higher throughput, then smaller p, larger b, earlier candidate, and
among equal pairs of one candidate (zero layer time) the one keeping more layers.
"""
from fractions import Fraction


class Infeasible(Exception):
    pass


def intra_select(candidates, capacity: int, n_layers: int):
    """candidates: (b, p, layer_fwd_time, bytes_per_layer, time_all_recomputed, bytes_all_recomputed).
    Returns (index, recompute count, time)."""
    pairs = []
    for index, (b, p, layer_fwd_time, bytes_per_layer, time_all, bytes_all) in enumerate(candidates):
        for kept in range(n_layers + 1):
            if bytes_all + kept * bytes_per_layer > capacity:
                continue
            time = time_all - kept * layer_fwd_time
            pairs.append(((Fraction(b, p * time), -p, b, -index, kept), (index, n_layers - kept, time)))
    if not pairs:
        raise Infeasible()
    return max(pairs, key=lambda pair: pair[0])[1]

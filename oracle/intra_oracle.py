"""Oracle for the DCP-intra selection (Algorithm 1 of the paper, Section 3.4).

TEST INFRASTRUCTURE ONLY: plain Python, exact rational arithmetic, the algorithm's steps in the
paper's order and notation.

Input: memory capacity M, model layers L, candidates C = {(b, p): (t_f, m, T_(b,p), M_(b,p))} from a
profile taken with every layer recomputed.  For each candidate the algorithm lets as many layers as
the spare memory allows keep their activations (each costs m bytes more and saves t_f), takes the
resulting time, and keeps the best candidate.

Readings (the listing and the text disagree in two places):
  * the listing's inner loop breaks at the first layer count whose memory fits, which would always
    stop at one layer; its comment ("minimal recompute layer with spare GPU memory") and Section 3.4
    ("computes the minimal r_i under the GPU memory capacity") ask for the largest count of
    non-recomputed layers that still fits.  The loop below therefore runs while the memory fits;
  * the listing keeps the candidate with the smallest time, the text ("compare the throughput
    according to Equation 1") the one with the highest b / (p * time); they agree when b and p are
    equal.  The text is followed.  Ties (the paper gives none): smaller p, larger b, earlier candidate.
"""
from fractions import Fraction


class Infeasible(Exception):
    pass


def intra_select(candidates, M: int, L: int):
    """candidates: list of (b, p, t_f, m, T_bp, M_bp).  Returns (index, recompute layers r, time)."""
    best_key = None
    result = None
    for idx, (b, p, t_f, m, T_bp, M_bp) in enumerate(candidates):
        if M_bp > M:
            continue
        keep = 0
        for layers in range(1, L + 1):          # layers whose recomputation is switched off
            M_opt = M_bp + layers * m
            if M_opt > M:
                break
            keep = layers
        cur_time = T_bp - keep * t_f
        throughput = Fraction(b, p * cur_time)
        key = (throughput, -p, b, -idx)
        if best_key is None or key > best_key:
            best_key = key
            result = (idx, L - keep, cur_time)
    if result is None:
        raise Infeasible()
    return result

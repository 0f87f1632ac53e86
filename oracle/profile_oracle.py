"""Oracle for the profile interpolation and the modelled micro-batch time.

TEST INFRASTRUCTURE ONLY: plain Python integers.
  * interp: the paper's dual-layer profile (Section 3.5) gives t_f, t_b at the profiled candidates only
    and is silent on lengths in between.  The reading: below the first bucket the value is linear in
    L, between two buckets linear, above the last quadratic in L; floor division.
  * model_time: Eq. 4-5, T = Lambda (t_f + t_b) + r t_f + T_C with t_f, t_b summed over the sequences.
  * candidate: Section 3.5's estimate with every layer recomputed, T = Lambda (2 t_f + t_b) + T_C, and
    Eq. 6 at r = Lambda, M = Lambda m_inp + M_C.
Pins (tests/test_profiler.py): hand-computed values at, between, below and above the buckets;
monotonicity; the r = Lambda case of Eq. 4-5 against Section 3.5's closed form.
"""


def interp(bucket_len, bucket_val, L):
    if L < 1:
        raise ValueError("length must be >= 1")
    xs, ys = list(bucket_len), list(bucket_val)
    if L <= xs[0]:
        return ys[0] * L // xs[0]
    if L >= xs[-1]:
        return ys[-1] * L * L // (xs[-1] * xs[-1])
    hi = next(i for i, x in enumerate(xs) if x >= L)
    lo = hi - 1
    return ys[lo] + (ys[hi] - ys[lo]) * (L - xs[lo]) // (xs[hi] - xs[lo])


def model_time(fwd_time, bwd_time, n_layers, recompute, fixed_cost=0):
    tf, tb = sum(fwd_time), sum(bwd_time)
    return n_layers * (tf + tb) + recompute * tf + fixed_cost


def candidate(b, p, t_f, t_b, act_bytes, inp_bytes, n_layers, const_bytes=0, fixed_cost=0):
    return (b, p, t_f, act_bytes, n_layers * (2 * t_f + t_b) + fixed_cost, n_layers * inp_bytes + const_bytes)

// Host-side cost model pieces that sit between the dual-layer profile and the planners:
// interpolation of profiled per-sequence times (Section 3.5 of the paper), the modelled time of a
// micro-batch (Eq. 4-5), the candidate row Algorithm 1 consumes, and the longest-first assignment of
// sequences to ranks.  Definitions are in include/dcp.h.  Integers only.
#include <algorithm>
#include <cstdint>
#include <numeric>
#include <vector>

#include "../../include/dcp.h"
#include "dcp_internal.h"

namespace {
using i128 = __int128;
constexpr i128 kMax = (i128)INT64_MAX;

int check_table(const char* who, const int32_t* bucket_len, const int64_t* bucket_val, int32_t n_buckets) {
    if (!bucket_len || !bucket_val) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer", who);
    if (n_buckets < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: a profile needs at least one bucket", who);
    for (int32_t i = 0; i < n_buckets; ++i) {
        if (bucket_len[i] < 1 || (i > 0 && bucket_len[i] <= bucket_len[i - 1]))
            return dcp::fail(DCP_ERR_INVALID_ARG, "%s: bucket lengths must be positive and strictly ascending", who);
        if (bucket_val[i] < 0) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: negative value in profile", who);
    }
    return DCP_OK;
}

// floor division throughout; values are non-negative except the slope between two buckets
int interp_one(const int32_t* xs, const int64_t* ys, int32_t n, int32_t L, int64_t* out) {
    i128 v;
    if (L <= xs[0]) {
        v = (i128)ys[0] * L / xs[0];
    } else if (L >= xs[n - 1]) {
        v = (i128)ys[n - 1] * L * L / ((i128)xs[n - 1] * xs[n - 1]);
    } else {
        const int32_t hi = (int32_t)(std::lower_bound(xs, xs + n, L) - xs), lo = hi - 1;
        const i128 num = ((i128)ys[hi] - (i128)ys[lo]) * (L - xs[lo]);
        const i128 den = xs[hi] - xs[lo];
        i128 q = num / den;
        if (num % den != 0 && num < 0) --q;                  // floor, not truncation, for a falling table
        v = (i128)ys[lo] + q;
    }
    if (v > kMax) return DCP_ERR_OVERFLOW;
    *out = (int64_t)v;
    return DCP_OK;
}
}  // namespace

extern "C" int dcp_profile_interp(const int32_t* bucket_len, const int64_t* bucket_val, int32_t n_buckets,
                                  const int32_t* lengths, int32_t n, int64_t* out) {
    const char* who = "dcp_profile_interp";
    if (int rc = check_table(who, bucket_len, bucket_val, n_buckets)) return rc;
    if (n < 0 || (n > 0 && (!lengths || !out))) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer or negative n", who);
    for (int32_t i = 0; i < n; ++i) {
        if (lengths[i] < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: lengths[%d] = %d, need >= 1", who, i, lengths[i]);
        if (interp_one(bucket_len, bucket_val, n_buckets, lengths[i], &out[i]) != DCP_OK)
            return dcp::fail(DCP_ERR_OVERFLOW, "%s: value for length %d does not fit in int64", who, lengths[i]);
    }
    return DCP_OK;
}

extern "C" int dcp_model_time(const int64_t* fwd_time, const int64_t* bwd_time, int32_t n, int32_t n_layers,
                              int32_t recompute, int64_t fixed_cost, int64_t* time) {
    const char* who = "dcp_model_time";
    if (!fwd_time || !bwd_time || !time) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer", who);
    if (n < 1 || n_layers < 1 || recompute < 0 || recompute > n_layers || fixed_cost < 0)
        return dcp::fail(DCP_ERR_INVALID_ARG, "%s: need n >= 1, Lambda >= 1, 0 <= r <= Lambda, T_C >= 0", who);
    i128 tf = 0, tb = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (fwd_time[i] < 0 || bwd_time[i] < 0) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: negative time", who);
        tf += fwd_time[i];
        tb += bwd_time[i];
    }
    const i128 t = (i128)n_layers * (tf + tb) + (i128)recompute * tf + fixed_cost;
    if (t > kMax) return dcp::fail(DCP_ERR_OVERFLOW, "%s: time does not fit in int64", who);
    *time = (int64_t)t;
    return DCP_OK;
}

extern "C" int dcp_intra_candidate_from_profile(int32_t batch_size, int32_t sp_size, int64_t t_f, int64_t t_b,
                                                int64_t act_bytes, int64_t inp_bytes, int32_t n_layers,
                                                int64_t const_bytes, int64_t fixed_cost, dcp_intra_candidate* out) {
    const char* who = "dcp_intra_candidate_from_profile";
    if (!out) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer", who);
    if (batch_size < 1 || sp_size < 1 || t_f < 0 || t_b < 0 || act_bytes < 0 || inp_bytes < 0 || n_layers < 1 ||
        const_bytes < 0 || fixed_cost < 0)
        return dcp::fail(DCP_ERR_INVALID_ARG, "%s: sizes must be >= 1 and profile entries >= 0", who);
    const i128 T = (i128)n_layers * (2 * (i128)t_f + (i128)t_b) + fixed_cost;      // every layer recomputed
    const i128 M = (i128)n_layers * inp_bytes + const_bytes;
    if (T > kMax || M > kMax) return dcp::fail(DCP_ERR_OVERFLOW, "%s: time or memory does not fit in int64", who);
    if (T < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: the modelled time is zero", who);
    out->batch_size = batch_size;
    out->sp_size = sp_size;
    out->t_f = t_f;
    out->m = act_bytes;
    out->time_full = (int64_t)T;
    out->mem_full = (int64_t)M;
    return DCP_OK;
}

extern "C" int dcp_activation_bytes(int64_t tokens, int32_t n_heads, int32_t head_dim, int32_t elt_bytes, int64_t* act_bytes,
                                    int64_t* inp_bytes) {
    const char* who = "dcp_activation_bytes";
    if (!act_bytes || !inp_bytes) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer", who);
    if (tokens < 0 || n_heads < 1 || head_dim < 1 || elt_bytes < 1)
        return dcp::fail(DCP_ERR_INVALID_ARG, "%s: need tokens >= 0 and H, d, e >= 1", who);
    const i128 unit = (i128)tokens * n_heads * head_dim * elt_bytes;
    if (4 * unit > kMax) return dcp::fail(DCP_ERR_OVERFLOW, "%s: size does not fit in int64", who);
    *act_bytes = (int64_t)(4 * unit);
    *inp_bytes = (int64_t)unit;
    return DCP_OK;
}

extern "C" int dcp_length_group_plan(int32_t n_seqs, int32_t batch_size, int32_t* mb_id, int32_t* n_mb) {
    const char* who = "dcp_length_group_plan";
    if (!mb_id || !n_mb) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer", who);
    if (n_seqs < 1 || batch_size < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: need n_seqs >= 1 and batch_size >= 1", who);
    for (int32_t i = 0; i < n_seqs; ++i) mb_id[i] = i / batch_size;
    *n_mb = (n_seqs + batch_size - 1) / batch_size;
    return DCP_OK;
}

extern "C" int dcp_shard_sequences(const int32_t* lengths, int32_t n, int32_t world_size, int32_t* rank_of,
                                   int64_t* load) {
    const char* who = "dcp_shard_sequences";
    if (n < 0 || world_size < 1 || (n > 0 && (!lengths || !rank_of)))
        return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer, negative n or world_size < 1", who);
    std::vector<i128> acc(world_size, 0);
    std::vector<int32_t> order(n);
    std::iota(order.begin(), order.end(), 0);
    for (int32_t i = 0; i < n; ++i)
        if (lengths[i] < 0) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: lengths[%d] is negative", who, i);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return lengths[a] > lengths[b]; });
    for (int32_t i : order) {
        int32_t r = 0;
        for (int32_t c = 1; c < world_size; ++c)
            if (acc[c] < acc[r]) r = c;                       // least loaded, lowest rank on ties
        rank_of[i] = r;
        acc[r] += (i128)lengths[i] * lengths[i];
    }
    if (load)
        for (int32_t r = 0; r < world_size; ++r) {
            if (acc[r] > kMax) return dcp::fail(DCP_ERR_OVERFLOW, "%s: load does not fit in int64", who);
            load[r] = (int64_t)acc[r];
        }
    return DCP_OK;
}

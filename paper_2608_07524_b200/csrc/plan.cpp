// Host-side micro-batch / recomputation planner (dcp_plan).
//
// Section 3.4 of the paper models a batch with r recomputed layers as
//     T = T_f + T_b + r * t_f + T_C                        (Eq. 4-5)
//     M = (Lambda - r) * m + Lambda * m_inp + M_C          (Eq. 6)
// and Algorithm 1 picks, per candidate, the smallest r that fits the memory capacity.  On one GPU
// (sequence-parallel size 1) the remaining freedom is how the batch is cut into gradient-
// accumulation micro-batches; sequences are first ordered by length (Section 3.1) and a plan is
// a cut of that order into contiguous blocks.  This file finds the optimum with an O(n^2)
// dynamic programme over suffixes of the sorted order; the definition, cost units and tie rules
// are stated in include/dcp.h.
#include <algorithm>
#include <cstdint>
#include <numeric>
#include <vector>

#include "../../include/dcp.h"
#include "dcp_internal.h"

namespace {

using u128 = unsigned __int128;
constexpr u128 kInt64Max = (u128)INT64_MAX;

struct Key {           // objective of a suffix plan: (cost, number of blocks)
    u128 cost;
    int32_t blocks;
    bool operator<(const Key& o) const { return cost != o.cost ? cost < o.cost : blocks < o.blocks; }
    bool operator==(const Key& o) const { return cost == o.cost && blocks == o.blocks; }
};

// Smallest r in [0, Lambda] whose memory fits, or -1.  mem(r) falls as r grows, so the answer is
// ceil((mem(0) - budget) / m) clamped; computed here without division to keep it obviously exact.
int min_recompute(u128 tok, const dcp_plan_params& p, u128 budget) {
    const u128 unit = (u128)p.n_heads * (u128)p.head_dim * (u128)p.elt_bytes * tok;   // < 2^31*2^31*2^31*2^36
    const u128 base = (u128)p.n_layers * unit + (u128)p.const_bytes;
    if (base > budget) return -1;
    const u128 room = budget - base;           // bytes left for un-recomputed layers
    const u128 m = 4 * unit;
    const u128 keep = m == 0 ? (u128)p.n_layers : std::min<u128>((u128)p.n_layers, room / m);
    return p.n_layers - (int)keep;
}

}  // namespace

namespace {

// Shared body of dcp_plan and dcp_plan_profiled.  weight[i] is the per-layer forward time of
// sequence i in the caller's unit (nullptr: the analytic stand-in 2 * length^2), so a block with
// r recomputed layers adds r * sum(weight) to the objective (Eq. 5).
int plan_impl(const char* who, const int32_t* lengths, const int64_t* weight, int32_t n, int64_t hbm_budget_bytes,
              const dcp_plan_params* params, int32_t* mb_id, int32_t* n_mb, int32_t* recompute, int64_t* cost) {
    static const dcp_plan_params kDefaults = {16, 128, 2, 1, 0, (int64_t)1 << 24};
    const dcp_plan_params p = params ? *params : kDefaults;
    if (!lengths || !mb_id || !n_mb || !recompute) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer", who);
    if (n < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: n = %d, need n >= 1", who, n);
    if (hbm_budget_bytes < 0) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: negative budget", who);
    if (p.n_heads < 1 || p.head_dim < 1 || p.elt_bytes < 1 || p.n_layers < 1 || p.const_bytes < 0 || p.fixed_cost < 0)
        return dcp::fail(DCP_ERR_INVALID_ARG, "%s: bad params (H, d, e, Lambda >= 1; M_C, T_C >= 0)", who);
    for (int32_t i = 0; i < n; ++i) {
        if (lengths[i] < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: lengths[%d] = %d, need >= 1", who, i, lengths[i]);
        if (weight && weight[i] < 0) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: fwd_time[%d] is negative", who, i);
    }

    std::vector<int32_t> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return lengths[a] > lengths[b]; });

    // prefix sums over the sorted order
    std::vector<u128> tok(n + 1, 0), w(n + 1, 0);
    for (int32_t i = 0; i < n; ++i) {
        const u128 L = (u128)lengths[order[i]];
        tok[i + 1] = tok[i] + L;
        w[i + 1] = w[i] + (weight ? (u128)weight[order[i]] : 2 * L * L);
    }
    const u128 budget = (u128)hbm_budget_bytes;
    if (min_recompute(tok[1] - tok[0], p, budget) < 0)
        return dcp::fail(DCP_ERR_INFEASIBLE,
                         "%s: the longest sequence (%d tokens) exceeds the budget even with every layer recomputed", who,
                         lengths[order[0]]);

    // best[i] = optimum for the sorted suffix i..n-1; cut[i] = end of its first block (largest on ties)
    std::vector<Key> best(n + 1);
    std::vector<int32_t> cut(n + 1, n), rec(n + 1, 0);
    best[n] = {0, 0};
    for (int32_t i = n - 1; i >= 0; --i) {
        // If the whole suffix fits without recomputation, one block is optimal: it costs T_C, every other
        // plan costs at least that, and ties go to fewer blocks.  This keeps batches that the budget does
        // not bind (the usual case) linear instead of quadratic in n.
        if (min_recompute(tok[n] - tok[i], p, budget) == 0) {
            best[i] = {(u128)p.fixed_cost, 1};
            cut[i] = n;
            rec[i] = 0;
            continue;
        }
        bool have = false;
        for (int32_t j = i + 1; j <= n; ++j) {
            const int r = min_recompute(tok[j] - tok[i], p, budget);
            if (r < 0) break;                                  // larger blocks only need more memory
            const Key cand = {best[j].cost + (u128)p.fixed_cost + (u128)r * (w[j] - w[i]), best[j].blocks + 1};
            if (!have || cand < best[i] || cand == best[i]) {  // '==' keeps the LARGEST j among ties
                best[i] = cand; cut[i] = j; rec[i] = r; have = true;
            }
        }
        // a single sequence always fits here: the longest one does and memory grows with length
    }
    if (best[0].cost > kInt64Max) return dcp::fail(DCP_ERR_OVERFLOW, "%s: cost does not fit in int64", who);

    int32_t k = 0;
    for (int32_t i = 0; i < n; i = cut[i], ++k) {
        recompute[k] = rec[i];
        for (int32_t a = i; a < cut[i]; ++a) mb_id[order[a]] = k;
    }
    *n_mb = k;
    if (cost) *cost = (int64_t)best[0].cost;
    return DCP_OK;
}

}  // namespace

extern "C" int dcp_plan(const int32_t* lengths, int32_t n, int64_t hbm_budget_bytes, const dcp_plan_params* params,
                        int32_t* mb_id, int32_t* n_mb, int32_t* recompute, int64_t* cost) {
    return plan_impl("dcp_plan", lengths, nullptr, n, hbm_budget_bytes, params, mb_id, n_mb, recompute, cost);
}

extern "C" int dcp_plan_profiled(const int32_t* lengths, const int64_t* fwd_time, int32_t n, int64_t hbm_budget_bytes,
                                 const dcp_plan_params* params, int32_t* mb_id, int32_t* n_mb, int32_t* recompute,
                                 int64_t* cost) {
    if (!fwd_time) return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_plan_profiled: null pointer");
    return plan_impl("dcp_plan_profiled", lengths, fwd_time, n, hbm_budget_bytes, params, mb_id, n_mb, recompute, cost);
}

// Where each sequence of a planned batch lives: in the batch (packed in input order) and in its
// micro-batch's own packed tensors.  The definition is in include/dcp.h.
extern "C" int dcp_plan_segments(const int32_t* lengths, const int32_t* mb_id, int32_t n, int32_t n_mb, int32_t max_rows,
                                 int32_t* mb_seq_offset, int32_t* seq_index, int32_t* mb_cu, int32_t* seg_offset,
                                 int32_t* seg, int32_t seg_capacity, int32_t* n_seg) {
    const char* who = "dcp_plan_segments";
    if (!lengths || !mb_id || !mb_seq_offset || !seq_index || !mb_cu || !seg_offset || !seg || !n_seg)
        return dcp::fail(DCP_ERR_INVALID_ARG, "%s: null pointer", who);
    if (n < 1 || n_mb < 1 || n_mb > n || max_rows < 1 || seg_capacity < 0)
        return dcp::fail(DCP_ERR_INVALID_ARG, "%s: need 1 <= n_mb <= n, max_rows >= 1, seg_capacity >= 0", who);
    std::vector<int64_t> src_row(n + 1, 0);
    std::vector<int32_t> count(n_mb, 0);
    for (int32_t i = 0; i < n; ++i) {
        if (lengths[i] < 0) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: lengths[%d] is negative", who, i);
        if (mb_id[i] < 0 || mb_id[i] >= n_mb) return dcp::fail(DCP_ERR_INVALID_ARG, "%s: mb_id[%d] = %d is not in [0, n_mb)", who, i, mb_id[i]);
        src_row[i + 1] = src_row[i] + lengths[i];
        ++count[mb_id[i]];
    }
    if (src_row[n] > INT32_MAX) return dcp::fail(DCP_ERR_OVERFLOW, "%s: more than 2^31 - 1 tokens", who);
    mb_seq_offset[0] = 0;
    for (int32_t k = 0; k < n_mb; ++k) mb_seq_offset[k + 1] = mb_seq_offset[k] + count[k];
    std::vector<int32_t> fill(mb_seq_offset, mb_seq_offset + n_mb);
    for (int32_t i = 0; i < n; ++i) seq_index[fill[mb_id[i]]++] = i;      // input order inside a micro-batch
    int64_t total_seg = 0;
    for (int32_t k = 0; k < n_mb; ++k) {
        seg_offset[k] = (int32_t)total_seg;
        int64_t dst = 0;
        // micro-batch k's boundary array occupies mb_cu[mb_seq_offset[k] + k ...], count[k] + 1 entries
        int32_t* cu = mb_cu + mb_seq_offset[k] + k;
        cu[0] = 0;
        for (int32_t e = mb_seq_offset[k]; e < mb_seq_offset[k + 1]; ++e) {
            const int32_t i = seq_index[e];
            for (int32_t done = 0; done < lengths[i]; done += max_rows) {
                const int32_t rows = std::min(max_rows, lengths[i] - done);
                if (total_seg < seg_capacity) {
                    seg[3 * total_seg] = (int32_t)(src_row[i] + done);
                    seg[3 * total_seg + 1] = (int32_t)(dst + done);
                    seg[3 * total_seg + 2] = rows;
                }
                ++total_seg;
            }
            dst += lengths[i];
            cu[e - mb_seq_offset[k] + 1] = (int32_t)dst;
        }
    }
    seg_offset[n_mb] = (int32_t)std::min<int64_t>(total_seg, INT32_MAX);
    *n_seg = seg_offset[n_mb];
    if (total_seg > seg_capacity)
        return dcp::fail(DCP_ERR_WORKSPACE, "%s: %lld segments needed, seg holds %d (ask again with that capacity)", who,
                         (long long)total_seg, seg_capacity);
    return DCP_OK;
}

// DCP-inter: gradient-accumulation step counts that balance n concurrently running batches
// (dcp_inter_plan).  Section 3.3 Eq. 3 and Appendix C of the paper; the definition, bounds and tie
// rules are stated in include/dcp.h.
//
// The paper evaluates every combination of step counts.  That is not needed: whatever the optimum
// is, its iteration time M = max_j g_j T_j is attained by some batch j with some count g, and once M
// is fixed every other batch independently wants the largest count with g_i T_i <= M.  So it is
// enough to try each M in { g * T_j } (at most sum_j cap_j values), each in O(n).
#include <cstdint>
#include <vector>

#include "../../include/dcp.h"
#include "dcp_internal.h"

namespace {
using u128 = unsigned __int128;
}

extern "C" int dcp_inter_plan(const int64_t* times, int32_t n, int32_t g_min, int32_t g_max, int32_t* g,
                              int64_t* idle, int64_t* iteration_time) {
    if (!times || !g) return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_inter_plan: null pointer");
    if (n < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_inter_plan: n = %d, need n >= 1", n);
    if (g_min < 1 || g_max < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_inter_plan: G_min and G_max must be >= 1");
    int64_t tmax = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (times[i] < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_inter_plan: times[%d] = %lld, need >= 1", i, (long long)times[i]);
        if (times[i] > tmax) tmax = times[i];
    }
    const u128 limit = (u128)g_max * (u128)tmax;         // longest iteration allowed (Appendix C, G_max)

    // the search must stay light enough to run before every iteration (Appendix C): refuse inputs whose
    // candidate list is out of proportion (times that differ by many orders of magnitude)
    u128 n_candidates = 0;
    for (int32_t j = 0; j < n; ++j) n_candidates += limit / (u128)times[j];
    if (n_candidates > (u128)4000000)
        return dcp::fail(DCP_ERR_UNSUPPORTED, "dcp_inter_plan: more than 4e6 candidate iteration times; rescale the times");

    bool have = false;
    u128 best_idle = 0, best_m = 0;
    std::vector<int64_t> cur(n), best(n);
    for (int32_t j = 0; j < n; ++j) {
        const int64_t cap_j = (int64_t)(limit / (u128)times[j]);
        for (int64_t gj = 1; gj <= cap_j; ++gj) {
            const u128 m = (u128)gj * (u128)times[j];
            u128 sum = 0;
            for (int32_t i = 0; i < n; ++i) {
                const u128 gi = m / (u128)times[i];      // >= 1 only if T_i <= m
                if (gi == 0) { sum = ~(u128)0; break; }  // batch i cannot finish one step within m
                cur[i] = (int64_t)gi;
                sum += gi * (u128)times[i];
            }
            if (sum == ~(u128)0) continue;
            const u128 idle_m = m * (u128)n - sum;
            bool better = false;
            if (!have) better = true;
            else if (idle_m != best_idle) better = idle_m < best_idle;
            else if (m != best_m) better = m < best_m;
            else {
                for (int32_t i = 0; i < n; ++i)
                    if (cur[i] != best[i]) { better = cur[i] < best[i]; break; }
            }
            if (better) { have = true; best_idle = idle_m; best_m = m; best = cur; }
        }
    }
    // g = (1, ..., 1) scaled so that the slowest batch sets m = T_max is always feasible
    if (!have) return dcp::fail(DCP_ERR_INFEASIBLE, "dcp_inter_plan: no feasible step counts (internal error)");

    int64_t gm = 0;
    for (int32_t i = 0; i < n; ++i) if (best[i] > gm) gm = best[i];
    const int64_t factor = gm < g_min ? (g_min + gm - 1) / gm : 1;   // Appendix C, G_min
    for (int32_t i = 0; i < n; ++i) {
        const u128 v = (u128)best[i] * (u128)factor;
        if (v > (u128)INT32_MAX) return dcp::fail(DCP_ERR_OVERFLOW, "dcp_inter_plan: a step count exceeds int32");
        g[i] = (int32_t)v;
    }
    const u128 idle_total = best_idle * (u128)factor, time_total = best_m * (u128)factor;
    if (idle_total > (u128)INT64_MAX || time_total > (u128)INT64_MAX)
        return dcp::fail(DCP_ERR_OVERFLOW, "dcp_inter_plan: idle or iteration time exceeds int64");
    if (idle) *idle = (int64_t)idle_total;
    if (iteration_time) *iteration_time = (int64_t)time_total;
    return DCP_OK;
}

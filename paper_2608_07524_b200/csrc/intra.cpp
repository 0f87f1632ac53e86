// DCP-intra: choice of batch size, sequence-parallel size and recompute count for one sequence
// length from profiled candidates (dcp_intra_select).  Section 3.4, Eq. 4-6 and Algorithm 1 of the
// paper; the definition, the reading of the algorithm's loop and the tie rules are stated in
// include/dcp.h.  Host code, integers only.
#include <cstdint>

#include "../../include/dcp.h"
#include "dcp_internal.h"

namespace {
using i128 = __int128;
}

extern "C" int dcp_intra_select(const dcp_intra_candidate* cands, int32_t n, int64_t mem_capacity, int32_t n_layers,
                                int32_t* best, int32_t* recompute, int64_t* time) {
    if (!cands || !best || !recompute) return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_intra_select: null pointer");
    if (n < 1) return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_intra_select: n = %d, need n >= 1", n);
    if (n_layers < 1 || mem_capacity < 0)
        return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_intra_select: need n_layers >= 1 and mem_capacity >= 0");
    int32_t best_i = -1, best_r = 0;
    i128 best_time = 0;
    for (int32_t i = 0; i < n; ++i) {
        const dcp_intra_candidate& c = cands[i];
        if (c.batch_size < 1 || c.sp_size < 1 || c.t_f < 0 || c.m < 0 || c.time_full < 1 || c.mem_full < 0)
            return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_intra_select: candidate %d has a non-positive size or a negative profile entry", i);
        if (c.mem_full > mem_capacity) continue;                       // does not fit even when every layer recomputes
        // layers that may keep their activations: each costs m more bytes and saves t_f
        const i128 room = (i128)mem_capacity - (i128)c.mem_full;
        i128 keep = c.m == 0 ? (i128)n_layers : room / (i128)c.m;
        if (keep > n_layers) keep = n_layers;
        const i128 cur = (i128)c.time_full - keep * (i128)c.t_f;
        if (cur < 1)
            return dcp::fail(DCP_ERR_INVALID_ARG, "dcp_intra_select: candidate %d: time_full is smaller than the recompute time it contains", i);
        bool better = best_i < 0;
        if (!better) {
            // throughput b / (p * T) (Eq. 1; the sequence length is common to all candidates), compared exactly
            const dcp_intra_candidate& o = cands[best_i];
            const i128 lhs = (i128)c.batch_size * (i128)o.sp_size * best_time;
            const i128 rhs = (i128)o.batch_size * (i128)c.sp_size * cur;
            if (lhs != rhs) better = lhs > rhs;
            else if (c.sp_size != o.sp_size) better = c.sp_size < o.sp_size;
            else if (c.batch_size != o.batch_size) better = c.batch_size > o.batch_size;
        }
        if (better) {
            best_i = i;
            best_r = n_layers - (int32_t)keep;
            best_time = cur;
        }
    }
    if (best_i < 0) return dcp::fail(DCP_ERR_INFEASIBLE, "dcp_intra_select: no candidate fits the memory capacity");
    if (best_time > (i128)INT64_MAX) return dcp::fail(DCP_ERR_OVERFLOW, "dcp_intra_select: time does not fit in int64");
    *best = best_i;
    *recompute = best_r;
    if (time) *time = (int64_t)best_time;
    return DCP_OK;
}

/*
 * Brute-force oracle for the single-GPU micro-batch / recomputation planner.
 *
 * TEST INFRASTRUCTURE ONLY.  The product planner is a dynamic programme; this file instead
 * enumerates every candidate plan and keeps the best, so that the two share neither code nor
 * method.
 *
 * The problem (Section 3.2 at sequence-parallel size p = 1, Section 3.4 Eqs. 4-6 and the rule
 * of Algorithm 1 "smallest recompute count that fits the memory capacity"):
 *
 *   lengths s_0..s_{n-1};  sort indices by (length descending, index ascending)
 *       (Section 3.1: sequences of similar size are grouped together);
 *   a plan cuts the sorted list into K >= 1 contiguous blocks (micro-batches);
 *   for a block:  tok = sum s,  W = sum s^2,
 *       m     = 4 * tok * H * d * e          activations kept by a layer that is not recomputed
 *       m_inp =     tok * H * d * e          layer input kept in any case
 *       M(r)  = (Lambda - r) * m + Lambda * m_inp + M_C                       (Eq. 6)
 *       r*    = min { r in [0, Lambda] : M(r) <= budget }; none => block infeasible
 *       time  = Lambda * 7 W + r* * 2 W + T_C            (Eq. 4-5 with t_f = 2W, t_b = 5W)
 *   objective: minimise the sum of block times.  Lambda * 7 * sum W is the same for every plan,
 *   so the reported cost is   K * T_C + 2 * sum_k r*_k W_k.
 *   ties: smaller cost, then smaller K, then the lexicographically LARGEST vector of block
 *   sizes (the first block takes as many sequences as it can).
 *
 * Profiled variant (Section 3.5: the per-layer forward time t_f comes from a measurement, not
 * from a model): the caller passes t_f of every sequence as weight[i]; a block's recompute term
 * is then r* * sum(weight) (Eq. 5) and the cost  K * T_C + sum_k r*_k sum_{i in k} weight[i].
 * weight == NULL means weight[i] = 2 s_i^2, which is the model above.
 *
 * All arithmetic is exact: unsigned __int128, far beyond what int64 inputs can reach.
 */
#include <stdint.h>
#include <stdlib.h>

typedef unsigned __int128 u128;

typedef struct {
    int32_t n_heads, head_dim, elt_bytes, n_layers;
    int64_t const_bytes, fixed_cost;
} oracle_plan_params;

static int cmp_desc(const void* a, const void* b)
{
    const int64_t* x = a; const int64_t* y = b;       /* pairs (length, index) */
    if (x[0] != y[0]) return x[0] > y[0] ? -1 : 1;
    return x[1] < y[1] ? -1 : (x[1] > y[1]);
}

/* Smallest r in [0, Lambda] with M(r) <= budget, or -1. */
static int min_recompute(u128 tok, const oracle_plan_params* p, u128 budget)
{
    const u128 unit = (u128)p->n_heads * p->head_dim * p->elt_bytes * tok;
    for (int r = 0; r <= p->n_layers; ++r) {
        u128 mem = (u128)(p->n_layers - r) * 4 * unit + (u128)p->n_layers * unit + (u128)p->const_bytes;
        if (mem <= budget) return r;
    }
    return -1;
}

/*
 * returns 0 and fills the outputs, 1 on bad arguments, 3 if no plan is feasible.
 *   mb_id[n]      micro-batch (0-based, in sorted order) of every ORIGINAL index
 *   recompute[n]  first *n_mb entries valid
 *   cost_lo/hi    the 128-bit cost split into two 64-bit halves
 * n <= 24 (2^(n-1) plans are enumerated).
 */
int oracle_plan_bruteforce_weighted(const int32_t* lengths, const int64_t* weight, int32_t n, int64_t budget,
                                    const oracle_plan_params* p, int32_t* mb_id, int32_t* n_mb,
                                    int32_t* recompute, uint64_t* cost_lo, uint64_t* cost_hi)
{
    if (!lengths || !p || n < 1 || n > 24 || budget < 0 || p->n_layers < 1 || p->n_heads < 1 ||
        p->head_dim < 1 || p->elt_bytes < 1 || p->const_bytes < 0 || p->fixed_cost < 0)
        return 1;
    int64_t pairs[24][2];
    for (int i = 0; i < n; ++i) {
        if (lengths[i] < 1 || (weight && weight[i] < 0)) return 1;
        pairs[i][0] = lengths[i]; pairs[i][1] = i;
    }
    qsort(pairs, n, sizeof pairs[0], cmp_desc);

    int have = 0;
    u128 best_cost = 0; int best_K = 0; int best_sizes[24]; int best_r[24];
    /* bit t of `cuts` set  <=>  a block boundary lies between sorted items t and t+1 */
    for (uint32_t cuts = 0; cuts < (1u << (n - 1)); ++cuts) {
        int sizes[24], rs[24], K = 0, feasible = 1, begin = 0;
        u128 cost = 0;
        for (int t = 0; t < n && feasible; ++t) {
            if (t == n - 1 || ((cuts >> t) & 1u)) {
                u128 tok = 0, W = 0;
                for (int a = begin; a <= t; ++a) {
                    tok += (u128)pairs[a][0];
                    W += weight ? (u128)weight[pairs[a][1]] : 2 * (u128)pairs[a][0] * (u128)pairs[a][0];
                }
                int r = min_recompute(tok, p, (u128)budget);
                if (r < 0) { feasible = 0; break; }
                sizes[K] = t - begin + 1; rs[K] = r; ++K;
                cost += (u128)p->fixed_cost + (u128)r * W;
                begin = t + 1;
            }
        }
        if (!feasible) continue;
        int better = 0;
        if (!have) better = 1;
        else if (cost != best_cost) better = cost < best_cost;
        else if (K != best_K) better = K < best_K;
        else {
            for (int b = 0; b < K; ++b)
                if (sizes[b] != best_sizes[b]) { better = sizes[b] > best_sizes[b]; break; }
        }
        if (better) {
            have = 1; best_cost = cost; best_K = K;
            for (int b = 0; b < K; ++b) { best_sizes[b] = sizes[b]; best_r[b] = rs[b]; }
        }
    }
    if (!have) return 3;
    int pos = 0;
    for (int b = 0; b < best_K; ++b) {
        recompute[b] = best_r[b];
        for (int a = 0; a < best_sizes[b]; ++a) mb_id[pairs[pos++][1]] = b;
    }
    *n_mb = best_K;
    if (cost_lo) *cost_lo = (uint64_t)best_cost;
    if (cost_hi) *cost_hi = (uint64_t)(best_cost >> 64);
    return 0;
}

int oracle_plan_bruteforce(const int32_t* lengths, int32_t n, int64_t budget,
                           const oracle_plan_params* p, int32_t* mb_id, int32_t* n_mb,
                           int32_t* recompute, uint64_t* cost_lo, uint64_t* cost_hi)
{
    return oracle_plan_bruteforce_weighted(lengths, NULL, n, budget, p, mb_id, n_mb, recompute, cost_lo, cost_hi);
}

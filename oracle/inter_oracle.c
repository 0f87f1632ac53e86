/*
 * Brute-force oracle for the DCP-inter accumulation-step search.
 *
 * TEST INFRASTRUCTURE ONLY; shares no code with the product.
 *
 * Section 3.3 of the paper: n batches run on n worker groups, batch i taking T_i per accumulation
 * step; choose integer step counts g_i >= 1 that minimise the idle time of Eq. 3,
 *     sum_i ( max_j g_j T_j  -  g_i T_i )            (the constant 1/W is dropped),
 * by evaluating every combination.  Appendix C bounds the search: the iteration may last at most
 * G_max times the slowest batch, i.e. g_i T_i <= G_max * max_j T_j; and if every g_i ends up below
 * G_min all of them are multiplied by ceil(G_min / max_i g_i).
 * Ties (the paper gives none): smaller iteration time max_j g_j T_j, then the lexicographically
 * smallest vector g.  This file enumerates every vector within the bounds.
 */
#include <stdint.h>

typedef unsigned __int128 u128;

/* returns 0 ok, 1 bad arguments, 4 search space too large (> 5e7 vectors) */
int oracle_inter_bruteforce(const int64_t* T, int32_t n, int32_t g_min, int32_t g_max, int32_t* g_out,
                            uint64_t* idle_lo, uint64_t* idle_hi)
{
    if (!T || !g_out || n < 1 || n > 16 || g_min < 1 || g_max < 1) return 1;
    int64_t tmax = 0;
    for (int i = 0; i < n; ++i) {
        if (T[i] < 1) return 1;
        if (T[i] > tmax) tmax = T[i];
    }
    const u128 limit = (u128)g_max * (u128)tmax;
    int64_t cap[16];
    double space = 1.0;
    for (int i = 0; i < n; ++i) {
        cap[i] = (int64_t)(limit / (u128)T[i]);     /* >= g_max >= 1 */
        space *= (double)cap[i];
    }
    if (space > 5e7) return 4;

    int64_t g[16], best_g[16];
    for (int i = 0; i < n; ++i) g[i] = 1;
    int have = 0;
    u128 best_idle = 0, best_max = 0;
    for (;;) {
        u128 mx = 0, sum = 0;
        for (int i = 0; i < n; ++i) {
            u128 t = (u128)g[i] * (u128)T[i];
            sum += t;
            if (t > mx) mx = t;
        }
        const u128 idle = mx * (u128)n - sum;
        int better = 0;
        if (!have) better = 1;
        else if (idle != best_idle) better = idle < best_idle;
        else if (mx != best_max) better = mx < best_max;
        else {
            for (int i = 0; i < n; ++i)
                if (g[i] != best_g[i]) { better = g[i] < best_g[i]; break; }
        }
        if (better) {
            have = 1; best_idle = idle; best_max = mx;
            for (int i = 0; i < n; ++i) best_g[i] = g[i];
        }
        int k = n - 1;                                /* next vector, odometer style */
        while (k >= 0 && g[k] == cap[k]) { g[k] = 1; --k; }
        if (k < 0) break;
        ++g[k];
    }
    int64_t gm = 0;
    for (int i = 0; i < n; ++i) if (best_g[i] > gm) gm = best_g[i];
    int64_t factor = 1;
    if (gm < g_min) factor = (g_min + gm - 1) / gm;
    for (int i = 0; i < n; ++i) {
        int64_t v = best_g[i] * factor;
        if (v > INT32_MAX) return 1;
        g_out[i] = (int32_t)v;
    }
    best_idle *= (u128)factor;
    if (idle_lo) *idle_lo = (uint64_t)best_idle;
    if (idle_hi) *idle_hi = (uint64_t)(best_idle >> 64);
    return 0;
}

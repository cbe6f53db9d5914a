/*
 * CPU oracle for solutions given in the paper's own variables: retention intervals (s, e, a)
 * (Moccasin, arXiv 2304.14463, Section 2, Eqs. 1-8, and the staged event domain of the subsection
 * "Complexity Reduction by Enforcing an Initial Topological Ordering").
 *
 * TEST INFRASTRUCTURE ONLY, like moc_oracle.c: plain loops over the definitions, nothing shared
 * with the CUDA path.  Compiled into the same shared object.
 *
 * A solution holds, for every node v and slot i in 0..C-1, a start s_v^i, an end e_v^i (events,
 * 1-based, domain D = {1..D}) and a flag a_v^i (1 active, 0 inactive), each as int32 in [n][C]
 * order.  Every constraint is taken as printed:
 *   Eq. 1  duration = sum of w_v over the active intervals;
 *   Eq. 2  s <= e for every interval, active or not;
 *   Eq. 3  e_v^i <= s_v^{i+1} for every node and i < C, active or not;
 *   Eq. 4  usage(t) = sum of m_v over the ACTIVE intervals with s <= t <= e, for t in D;
 *          peak = max_t usage(t); the constraint is peak <= M;
 *   Eq. 5  for every edge (u,v) and every ACTIVE interval i of v there is an ACTIVE interval j of
 *          u with s_u^j + 1 <= s_v^i <= e_u^j;
 *   Eq. 6  s_v^i != s_u^j for v != u and all i, j, active or not (the alldifferent constraint over
 *          the start variables); not part of the staged model;
 *   Eq. 7  a_v^0 = 1 for every node;
 *   Eq. 8  s, e in D and a in {0, 1}.
 * Staged model: with k = 1-based index of node v in the input topological order, an active interval
 * of v may start only at event k of a stage j >= k, i.e. s = j(j-1)/2 + k (stage j holds the events
 * j(j-1)/2 + 1 .. j(j+1)/2), and the first interval starts at the last event of stage k:
 * s_v^0 = k(k+1)/2.  D = n(n+1)/2.
 *
 * Result: a mask with bit (q-2) set when Eq. q (q = 2..8) is violated (bit 0 = Eq. 2 ... bit 6 =
 * Eq. 8) and bit 7 set when the staged rule is violated.  When Eq. 8 fails nothing else is
 * evaluated: mask = 64, peak = dur = -1.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "moc_oracle_graph.h"

enum { BIT_EQ2 = 1, BIT_EQ3 = 2, BIT_EQ4 = 4, BIT_EQ5 = 8, BIT_EQ6 = 16, BIT_EQ7 = 32, BIT_EQ8 = 64, BIT_STAGE = 128 };

/*
 * topo_index: NULL for the plain model (then D is the caller's domain size, normally C*n); for the
 * staged model the 1-based index of every node in the input topological order (then D must be
 * n(n+1)/2).  out_usage (may be NULL): D entries, usage(t) of Eq. 4 for t = 1..D (untouched when
 * Eq. 8 fails).
 */
void moc_oracle_check_intervals(const void *graph, const int32_t *s, const int32_t *e, const int32_t *a,
                                int64_t D, const int32_t *topo_index, int64_t M, int64_t *out_peak,
                                int64_t *out_dur, int32_t *out_mask, int64_t *out_usage) {
    const ograph *g = (const ograph *)graph;
    const int32_t n = g->n, C = g->C;
    int32_t mask = 0;
    *out_peak = -1;
    *out_dur = -1;
    /* Eq. 8 */
    for (int32_t k = 0; k < n * C; ++k)
        if (s[k] < 1 || s[k] > D || e[k] < 1 || e[k] > D || (a[k] != 0 && a[k] != 1)) mask |= BIT_EQ8;
    if (mask) {
        *out_mask = mask;
        return;
    }
    /* Eq. 1 */
    int64_t dur = 0;
    for (int32_t v = 0; v < n; ++v)
        for (int32_t i = 0; i < C; ++i)
            if (a[v * C + i]) dur += g->w[v];
    /* Eqs. 2, 3, 7 */
    for (int32_t v = 0; v < n; ++v) {
        if (a[v * C] != 1) mask |= BIT_EQ7;
        for (int32_t i = 0; i < C; ++i) {
            if (s[v * C + i] > e[v * C + i]) mask |= BIT_EQ2;
            if (i + 1 < C && e[v * C + i] > s[v * C + i + 1]) mask |= BIT_EQ3;
        }
    }
    /* Eq. 4 */
    int64_t peak = 0;
    for (int64_t t = 1; t <= D; ++t) {
        int64_t use = 0;
        for (int32_t v = 0; v < n; ++v)
            for (int32_t i = 0; i < C; ++i)
                if (a[v * C + i] && s[v * C + i] <= t && t <= e[v * C + i]) use += g->m[v];
        if (use > peak) peak = use;
        if (out_usage) out_usage[t - 1] = use;
    }
    if (peak > M) mask |= BIT_EQ4;
    /* Eq. 5 */
    for (int32_t v = 0; v < n; ++v)
        for (int64_t k = g->pred_start[v]; k < g->pred_start[v + 1]; ++k) {
            const int32_t u = g->pred[k];
            for (int32_t i = 0; i < C; ++i) {
                if (!a[v * C + i]) continue;
                int found = 0;
                for (int32_t j = 0; j < C; ++j)
                    if (a[u * C + j] && s[u * C + j] + 1 <= s[v * C + i] && s[v * C + i] <= e[u * C + j]) found = 1;
                if (!found) mask |= BIT_EQ5;
            }
        }
    if (!topo_index) {
        /* Eq. 6 */
        for (int32_t v = 0; v < n; ++v)
            for (int32_t u = v + 1; u < n; ++u)
                for (int32_t i = 0; i < C; ++i)
                    for (int32_t j = 0; j < C; ++j)
                        if (s[v * C + i] == s[u * C + j]) mask |= BIT_EQ6;
    } else {
        /* staged model */
        for (int32_t v = 0; v < n; ++v) {
            const int64_t k = topo_index[v];
            if (s[v * C] != k * (k + 1) / 2) mask |= BIT_STAGE;
            for (int32_t i = 0; i < C; ++i) {
                if (!a[v * C + i]) continue;
                int ok = 0;
                for (int64_t j = k; j <= n; ++j)
                    if (s[v * C + i] == j * (j - 1) / 2 + k) ok = 1;
                if (!ok) mask |= BIT_STAGE;
            }
        }
    }
    *out_peak = peak;
    *out_dur = dur;
    *out_mask = mask;
}

/*
 * The execution sequence a solution stands for: its active intervals in the order of their starts
 * (each active interval is one computation of its node, in its first event).  Returns the number of
 * steps written to out_seq (room for n*C), or -1 when two active intervals start at the same event
 * (no sequential execution) or Eq. 8 fails.
 */
int32_t moc_oracle_intervals_to_sequence(const void *graph, const int32_t *s, const int32_t *e, const int32_t *a,
                                         int64_t D, int32_t *out_seq) {
    const ograph *g = (const ograph *)graph;
    const int32_t K = g->n * g->C;
    for (int32_t k = 0; k < K; ++k)
        if (s[k] < 1 || s[k] > D || e[k] < 1 || e[k] > D || (a[k] != 0 && a[k] != 1)) return -1;
    int32_t len = 0;
    for (int64_t t = 1; t <= D; ++t) {
        int32_t here = 0;
        for (int32_t k = 0; k < K; ++k)
            if (a[k] && s[k] == t) {
                if (here++) return -1;
                out_seq[len++] = k / g->C;
            }
    }
    return len;
}

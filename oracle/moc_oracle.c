/*
 * CPU oracle for the evaluation of rematerialization sequences (Moccasin, arXiv 2304.14463).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, sequential statement of what one
 * schedule evaluates to.  It is used by the tests, by the smoke check and by the timed CPU
 * baseline of the benchmark; the CUDA library never calls, includes or links it, and it shares
 * no code, header, table or helper with the CUDA path.
 *
 * What is evaluated (paper, Section 1 problem statement and Section 2, Eqs. 1-8):
 *   a schedule is a sequence seq[0..T) of node ids of a DAG G=(V,E); position t is the t-th
 *   filled compute event (empty events change neither duration nor peak, Section 2), each
 *   occurrence of a node is one "copy" = one active retention interval [s,e] with s = its
 *   position.  An edge (u,v) means v consumes the output of u.
 *
 *   duration   Eq. 1      : sum of w over every executed copy, recomputations included.
 *   precedence Eq. 5      : when v runs at step t every predecessor u needs an active interval
 *                           with s_u + 1 <= t <= e_u.  Among the copies of u before t the most
 *                           recent one is charged (by Eq. 3 intervals of one node do not overlap,
 *                           so this choice keeps every interval as short as the sequence allows;
 *                           the result is the least memory the sequence can be run in).
 *   interval end          : e = last step that consumes the copy before the node is recomputed;
 *                           a copy nobody consumes has e = s (Eq. 2 allows s = e).  The output of
 *                           a sink (a node without successors) is the result of the computation:
 *                           its LAST copy is retained to the final step T-1.
 *   memory     Eq. 4      : usage at step t = sum of m over the copies with s <= t <= e (both
 *                           ends inclusive); peak = maximum over the steps (Section 2).
 *   budget     Eq. 4      : feasible iff peak <= M.
 *   well-formedness       : every node at least once (Eq. 7), at most C_v copies of node v
 *                           (Section 2, parameter C_v: uniform C unless per-node caps <= C are
 *                           set), hence n <= T <= C*n, ids in range.
 *
 * Status codes: 1 feasible, 0 peak over budget, -1 a precedence constraint is violated
 * (peak = -1, duration still reported), -2 malformed sequence (peak = duration = -1).
 *
 * Every function is pinned by tests/test_oracle_*.py: the paper's worked 4-node example, closed
 * forms (chain, star), an independent set-definition brute force and a direct check of
 * Eqs. 2-5 on the intervals this file produces.
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "moc_oracle_graph.h"

/* Builds the predecessor lists of G=(V,E) (Section 1: (u,v) in E, v needs the output of u). */
ograph *moc_oracle_graph_create(int32_t n, int64_t n_edges, const int32_t *edges, const int64_t *w,
                                const int64_t *m, int32_t C) {
    if (n <= 0 || n_edges < 0 || C < 1) return NULL;
    for (int64_t e = 0; e < n_edges; ++e) {
        int32_t u = edges[2 * e], v = edges[2 * e + 1];
        if (u < 0 || u >= n || v < 0 || v >= n || u == v) return NULL;
    }
    ograph *g = (ograph *)calloc(1, sizeof(ograph));
    g->n = n;
    g->C = C;
    g->n_edges = n_edges;
    g->pred_start = (int64_t *)calloc((size_t)n + 1, sizeof(int64_t));
    g->pred = (int32_t *)calloc((size_t)(n_edges > 0 ? n_edges : 1), sizeof(int32_t));
    g->has_succ = (uint8_t *)calloc((size_t)n, 1);
    g->w = (int64_t *)malloc((size_t)n * sizeof(int64_t));
    g->m = (int64_t *)malloc((size_t)n * sizeof(int64_t));
    memcpy(g->w, w, (size_t)n * sizeof(int64_t));
    memcpy(g->m, m, (size_t)n * sizeof(int64_t));
    for (int64_t e = 0; e < n_edges; ++e) g->pred_start[edges[2 * e + 1] + 1]++;
    for (int32_t v = 0; v < n; ++v) g->pred_start[v + 1] += g->pred_start[v];
    int64_t *fill = (int64_t *)malloc((size_t)n * sizeof(int64_t));
    memcpy(fill, g->pred_start, (size_t)n * sizeof(int64_t));
    for (int64_t e = 0; e < n_edges; ++e) {
        int32_t u = edges[2 * e], v = edges[2 * e + 1];
        g->pred[fill[v]++] = u;
        g->has_succ[u] = 1;
    }
    free(fill);
    return g;
}

/* Per-node caps C_v (Section 2: node v has at most C_v retention intervals), each in [1, C];
 * NULL restores the uniform cap C.  Returns 0, or -1 for a cap outside [1, C]. */
int32_t moc_oracle_graph_set_caps(ograph *g, const int32_t *caps) {
    free(g->cap);
    g->cap = NULL;
    if (!caps) return 0;
    for (int32_t v = 0; v < g->n; ++v)
        if (caps[v] < 1 || caps[v] > g->C) return -1;
    g->cap = (int32_t *)malloc((size_t)g->n * sizeof(int32_t));
    memcpy(g->cap, caps, (size_t)g->n * sizeof(int32_t));
    return 0;
}

void moc_oracle_graph_destroy(ograph *g) {
    if (!g) return;
    free(g->cap);
    free(g->pred_start);
    free(g->pred);
    free(g->has_succ);
    free(g->w);
    free(g->m);
    free(g);
}

/*
 * Evaluates one sequence.  out_profile (T entries) and out_free (T entries) may be NULL.
 * On status -1 / -2 the two arrays are filled with -1.
 */
void moc_oracle_eval(const ograph *g, const int32_t *seq, int32_t T, int64_t M, int64_t *out_peak,
                     int64_t *out_dur, int32_t *out_status, int64_t *out_profile, int32_t *out_free) {
    const int32_t n = g->n;
    *out_peak = -1;
    *out_dur = -1;
    *out_status = -2;
    if (out_profile) for (int32_t t = 0; t < T; ++t) out_profile[t] = -1;
    if (out_free) for (int32_t t = 0; t < T; ++t) out_free[t] = -1;

    /* well-formedness: Eq. 7 (each node at least once), at most C copies, ids in range */
    if (T < n || (int64_t)T > (int64_t)g->C * n) return;
    int32_t *count = (int32_t *)calloc((size_t)n, sizeof(int32_t));
    int ok = 1;
    for (int32_t t = 0; t < T && ok; ++t) {
        if (seq[t] < 0 || seq[t] >= n) ok = 0;
        else count[seq[t]]++;
    }
    for (int32_t v = 0; v < n && ok; ++v)
        if (count[v] < 1 || count[v] > (g->cap ? g->cap[v] : g->C)) ok = 0;
    free(count);
    if (!ok) return;

    /* Eq. 1: total duration */
    int64_t dur = 0;
    for (int32_t t = 0; t < T; ++t) dur += g->w[seq[t]];
    *out_dur = dur;

    /* Eq. 5 by sequential simulation: last[u] = position of the most recent copy of u */
    int32_t *last = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    int32_t *fr = (int32_t *)malloc((size_t)T * sizeof(int32_t));
    for (int32_t v = 0; v < n; ++v) last[v] = -1;
    int violated = 0;
    for (int32_t t = 0; t < T; ++t) {
        const int32_t v = seq[t];
        fr[t] = t; /* Eq. 2: an interval holds at least its own compute step */
        for (int64_t k = g->pred_start[v]; k < g->pred_start[v + 1]; ++k) {
            const int32_t u = g->pred[k];
            if (last[u] < 0) violated = 1;          /* no copy of u with s_u + 1 <= t */
            else if (fr[last[u]] < t) fr[last[u]] = t; /* keep that copy until step t */
        }
        last[v] = t;
    }
    if (violated) {
        *out_status = -1;
        free(last);
        free(fr);
        return;
    }
    /* results of the computation stay resident to the end */
    for (int32_t v = 0; v < n; ++v)
        if (!g->has_succ[v]) fr[last[v]] = T - 1;

    /* Eq. 4: usage(t) = sum of m over copies p with p <= t <= free[p]; difference array */
    int64_t *delta = (int64_t *)calloc((size_t)T + 1, sizeof(int64_t));
    for (int32_t p = 0; p < T; ++p) {
        delta[p] += g->m[seq[p]];
        delta[fr[p] + 1] -= g->m[seq[p]];
    }
    int64_t run = 0, peak = 0;
    for (int32_t t = 0; t < T; ++t) {
        run += delta[t];
        if (out_profile) out_profile[t] = run;
        if (run > peak) peak = run;
    }
    if (out_free) memcpy(out_free, fr, (size_t)T * sizeof(int32_t));
    *out_peak = peak;
    *out_status = (peak <= M) ? 1 : 0;
    free(delta);
    free(last);
    free(fr);
}

/* Batch: schedule b occupies seqs[offs[b] .. offs[b]+lens[b]) with offs the exclusive sum of lens. */
typedef struct {
    const ograph *g;
    const int32_t *seqs;
    const int32_t *lens;
    const int64_t *offs;
    int64_t b0, b1;
    int64_t M;
    int64_t *peak, *dur;
    int32_t *status;
} batch_job;

static void *batch_worker(void *arg) {
    batch_job *j = (batch_job *)arg;
    for (int64_t b = j->b0; b < j->b1; ++b)
        moc_oracle_eval(j->g, j->seqs + j->offs[b], j->lens[b], j->M, &j->peak[b], &j->dur[b],
                        &j->status[b], NULL, NULL);
    return NULL;
}

/* Independent schedules are split into contiguous blocks, one per thread; returns threads used. */
int32_t moc_oracle_eval_batch(const ograph *g, const int32_t *seqs, const int32_t *lens, int64_t B,
                              int64_t M, int64_t *out_peak, int64_t *out_dur, int32_t *out_status,
                              int32_t n_threads) {
    if (B <= 0) return 0;
    if (n_threads < 1) n_threads = 1;
    if (n_threads > B) n_threads = (int32_t)B;
    int64_t *offs = (int64_t *)malloc((size_t)(B + 1) * sizeof(int64_t));
    offs[0] = 0;
    for (int64_t b = 0; b < B; ++b) offs[b + 1] = offs[b] + (lens[b] > 0 ? lens[b] : 0);
    batch_job *jobs = (batch_job *)calloc((size_t)n_threads, sizeof(batch_job));
    pthread_t *th = (pthread_t *)calloc((size_t)n_threads, sizeof(pthread_t));
    for (int32_t i = 0; i < n_threads; ++i) {
        jobs[i] = (batch_job){g, seqs, lens, offs, B * i / n_threads, B * (i + 1) / n_threads,
                              M, out_peak, out_dur, out_status};
        if (i > 0) pthread_create(&th[i], NULL, batch_worker, &jobs[i]);
    }
    batch_worker(&jobs[0]);
    for (int32_t i = 1; i < n_threads; ++i) pthread_join(th[i], NULL);
    free(th);
    free(jobs);
    free(offs);
    return n_threads;
}

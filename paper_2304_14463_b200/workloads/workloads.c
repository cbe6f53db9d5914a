/*
 * Seeded synthetic inputs: compute DAGs, node weights and batches of candidate execution
 * sequences.  Pure data generation -- nothing here evaluates a sequence (no free steps, no memory
 * profile, no peak); the evaluator and its CPU checker both receive these arrays as plain inputs.
 *
 * Random numbers: xoshiro256** (Blackman & Vigna) seeded through splitmix64; every schedule of a
 * batch has its own stream (seed, index), so the output does not depend on the thread count.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct { uint64_t s[4]; } rng_t;

static uint64_t splitmix64(uint64_t *x) {
    uint64_t z = (*x += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static void rng_seed(rng_t *r, uint64_t seed, uint64_t stream) {
    uint64_t x = seed * 0xD1342543DE82EF95ull + stream * 0x2545F4914F6CDD1Dull + 0x1234567ull;
    for (int i = 0; i < 4; ++i) r->s[i] = splitmix64(&x);
}
static inline uint64_t rotl64(uint64_t x, int k) { return (x << k) | (x >> (64 - k)); }
static uint64_t rng_next(rng_t *r) {
    uint64_t *s = r->s;
    const uint64_t result = rotl64(s[1] * 5, 7) * 9, t = s[1] << 17;
    s[2] ^= s[0]; s[3] ^= s[1]; s[1] ^= s[2]; s[0] ^= s[3];
    s[2] ^= t; s[3] = rotl64(s[3], 45);
    return result;
}
/* uniform in [0, k), k >= 1 */
static uint32_t rng_below(rng_t *r, uint32_t k) {
    return (uint32_t)(((unsigned __int128)rng_next(r) * k) >> 64);
}
/* uniform in (0, 1] */
static double rng_unit(rng_t *r) { return ((double)(rng_next(r) >> 11) + 1.0) * (1.0 / 9007199254740992.0); }
static double rng_normal(rng_t *r) {
    const double u1 = rng_unit(r), u2 = rng_unit(r);
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925 * u2);
}

/* ------------------------------------------------------------------ weights */
void wl_weights_uniform(int32_t n, int64_t lo, int64_t hi, uint64_t seed, uint64_t stream, int64_t *out) {
    rng_t r; rng_seed(&r, seed, stream);
    for (int32_t v = 0; v < n; ++v) out[v] = lo + (int64_t)rng_below(&r, (uint32_t)(hi - lo + 1));
}
void wl_weights_lognormal(int32_t n, double mu, double sigma, uint64_t seed, uint64_t stream, int64_t *out) {
    rng_t r; rng_seed(&r, seed, stream);
    for (int32_t v = 0; v < n; ++v) {
        const double x = exp(mu + sigma * rng_normal(&r));
        int64_t k = (int64_t)llround(x);
        out[v] = k < 1 ? 1 : k;
    }
}

/* ------------------------------------------------------------------ edge set helper */
typedef struct { uint64_t *slot; uint64_t mask; int32_t *edges; int64_t count, cap; } edgeset;
static void es_init(edgeset *s, int64_t cap, int32_t *edges) {
    uint64_t sz = 16; while (sz < (uint64_t)cap * 4) sz <<= 1;
    s->slot = (uint64_t *)malloc(sz * sizeof(uint64_t));
    memset(s->slot, 0xFF, sz * sizeof(uint64_t));
    s->mask = sz - 1; s->edges = edges; s->count = 0; s->cap = cap;
}
/* returns 1 if (u,v) was new and has been appended, 0 if present, -1 if full */
static int es_add(edgeset *s, int32_t u, int32_t v) {
    const uint64_t key = ((uint64_t)(uint32_t)u << 32) | (uint32_t)v;
    uint64_t x = key, h = splitmix64(&x) & s->mask;
    while (s->slot[h] != ~0ull) { if (s->slot[h] == key) return 0; h = (h + 1) & s->mask; }
    if (s->count >= s->cap) return -1;
    s->slot[h] = key;
    s->edges[2 * s->count] = u; s->edges[2 * s->count + 1] = v; s->count++;
    return 1;
}

/* ------------------------------------------------------------------ graphs
 * All generators number the nodes in a topological order (u < v for every edge). */

/* Random layered DAG: n nodes in L layers whose sizes differ by at most one; (i) every node outside
 * layer 0 gets one predecessor drawn from the previous layer, (ii) every node outside the last
 * layer that still has no successor gets one in the next layer, (iii) distinct uniform pairs with
 * layer(u) < layer(v) are added until there are exactly m edges.  Returns m, or -1 if (i)+(ii)
 * already exceed m or m exceeds the number of admissible pairs. */
int64_t wl_layered_dag(int32_t n, int64_t m, int32_t L, uint64_t seed, int32_t *edges) {
    if (n < L || L < 2) return -1;
    int32_t *start = (int32_t *)malloc((size_t)(L + 1) * sizeof(int32_t));
    int32_t *layer = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    uint8_t *has_succ = (uint8_t *)calloc((size_t)n, 1);
    start[0] = 0;
    for (int32_t l = 0; l < L; ++l) start[l + 1] = start[l] + n / L + (l < n % L ? 1 : 0);
    for (int32_t l = 0; l < L; ++l) for (int32_t v = start[l]; v < start[l + 1]; ++v) layer[v] = l;
    int64_t pairs = 0;
    for (int32_t l = 0; l < L; ++l) pairs += (int64_t)(start[l + 1] - start[l]) * (n - start[l + 1]);
    int64_t ret = -1;
    edgeset s; es_init(&s, m, edges);
    rng_t r; rng_seed(&r, seed, 0);
    if (m > pairs) goto done;
    for (int32_t v = start[1]; v < n; ++v) {
        const int32_t l = layer[v];
        const int32_t u = start[l - 1] + (int32_t)rng_below(&r, (uint32_t)(start[l] - start[l - 1]));
        if (es_add(&s, u, v) < 0) goto done;
        has_succ[u] = 1;
    }
    for (int32_t u = 0; u < start[L - 1]; ++u) {
        if (has_succ[u]) continue;
        const int32_t l = layer[u];
        const int32_t v = start[l + 1] + (int32_t)rng_below(&r, (uint32_t)(start[l + 2] - start[l + 1]));
        if (es_add(&s, u, v) < 0) goto done;
        has_succ[u] = 1;
    }
    while (s.count < m) {
        int32_t u = (int32_t)rng_below(&r, (uint32_t)n), v = (int32_t)rng_below(&r, (uint32_t)n);
        if (layer[u] == layer[v]) continue;
        if (layer[u] > layer[v]) { int32_t t = u; u = v; v = t; }
        es_add(&s, u, v);
    }
    ret = s.count;
done:
    free(s.slot); free(start); free(layer); free(has_succ);
    return ret;
}

/* Training-shaped DAG on 2F nodes: forward chain f_0..f_{F-1} (ids 0..F-1), backward ops
 * b_{F-1}..b_0 (ids F..2F-1, b_i = 2F-1-i) with f_i -> b_i and b_{i+1} -> b_i, plus n_skips
 * distinct forward skips f_i -> f_{i+s}, s uniform in [smin, smax], each mirrored as
 * b_{i+s} -> b_i.  Edge count 3F - 2 + 2*n_skips.  Returns it, or -1. */
int64_t wl_training_dag(int32_t F, int32_t n_skips, int32_t smin, int32_t smax, uint64_t seed,
                        int32_t *edges) {
    if (F < smax + 1 || smin < 2 || smax < smin) return -1;
    int64_t possible = 0;
    for (int32_t s = smin; s <= smax; ++s) possible += F - s;
    if (n_skips > possible) return -1;
    const int64_t m = 3 * (int64_t)F - 2 + 2 * (int64_t)n_skips;
    edgeset s; es_init(&s, m, edges);
    rng_t r; rng_seed(&r, seed, 0);
#define B_ID(i) (2 * F - 1 - (i))
    for (int32_t i = 0; i + 1 < F; ++i) es_add(&s, i, i + 1);
    for (int32_t i = 0; i < F; ++i) es_add(&s, i, B_ID(i));
    for (int32_t i = 0; i + 1 < F; ++i) es_add(&s, B_ID(i + 1), B_ID(i));
    int32_t placed = 0;
    while (placed < n_skips) {
        const int32_t span = smin + (int32_t)rng_below(&r, (uint32_t)(smax - smin + 1));
        const int32_t i = (int32_t)rng_below(&r, (uint32_t)(F - span));
        if (es_add(&s, i, i + span) == 1) { es_add(&s, B_ID(i + span), B_ID(i)); placed++; }
    }
#undef B_ID
    const int64_t cnt = s.count;
    free(s.slot);
    return cnt;
}

/* ResNet-like forward+backward DAG on 2F nodes (deterministic): forward chain, a skip
 * f_{3k} -> f_{3k+3} per block of three ops, both mirrored in the backward pass (b_i = 2F-1-i),
 * and the cross edges f_i -> b_i, f_{i-1} -> b_i, f_{i+1} -> b_i, f_{3k} -> b_{3k+3}. */
int64_t wl_resnet_dag(int32_t F, int64_t cap, int32_t *edges) {
    edgeset s; es_init(&s, cap, edges);
    int bad = 0;
#define B_ID(i) (2 * F - 1 - (i))
#define ADD(u, v) do { if (es_add(&s, (u), (v)) < 0) bad = 1; } while (0)
    for (int32_t i = 0; i + 1 < F; ++i) ADD(i, i + 1);
    for (int32_t k = 0; 3 * k + 3 < F; ++k) ADD(3 * k, 3 * k + 3);
    for (int32_t i = 0; i + 1 < F; ++i) ADD(B_ID(i + 1), B_ID(i));
    for (int32_t k = 0; 3 * k + 3 < F; ++k) ADD(B_ID(3 * k + 3), B_ID(3 * k));
    for (int32_t i = 0; i < F; ++i) ADD(i, B_ID(i));
    for (int32_t i = 1; i < F; ++i) ADD(i - 1, B_ID(i));
    for (int32_t i = 0; i + 1 < F; ++i) ADD(i + 1, B_ID(i));
    for (int32_t k = 0; 3 * k + 3 < F; ++k) ADD(3 * k, B_ID(3 * k + 3));
#undef ADD
#undef B_ID
    const int64_t cnt = bad ? -1 : s.count;
    free(s.slot);
    return cnt;
}

/* ------------------------------------------------------------------ schedules
 * One schedule: a topological order produced by Kahn's algorithm that draws the next node
 * uniformly among the ready ones; then, node by node in id order and for each of its C-1 spare
 * copies, with probability p one more copy is inserted at an index uniform in
 * (first position of the node, current length]; insertion stops once the length reaches t_cap. */
typedef struct {
    int32_t n, C, t_cap;
    double p;
    const int64_t *succ_start; const int32_t *succ; const int32_t *indeg;
    uint64_t seed;
    int64_t b0, b1, stride;
    int32_t *seqs, *lens;
} sched_job;

static void *sched_worker(void *arg) {
    sched_job *j = (sched_job *)arg;
    const int32_t n = j->n;
    int32_t *deg = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    int32_t *ready = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    for (int64_t b = j->b0; b < j->b1; ++b) {
        rng_t r; rng_seed(&r, j->seed, (uint64_t)b + 1);
        int32_t *seq = j->seqs + b * j->stride;
        int32_t len = 0, n_ready = 0;
        memcpy(deg, j->indeg, (size_t)n * sizeof(int32_t));
        for (int32_t v = 0; v < n; ++v) if (deg[v] == 0) ready[n_ready++] = v;
        while (n_ready > 0) {
            const uint32_t k = rng_below(&r, (uint32_t)n_ready);
            const int32_t v = ready[k];
            ready[k] = ready[--n_ready];
            seq[len++] = v;
            for (int64_t e = j->succ_start[v]; e < j->succ_start[v + 1]; ++e)
                if (--deg[j->succ[e]] == 0) ready[n_ready++] = j->succ[e];
        }
        for (int32_t v = 0; v < n; ++v) {
            for (int32_t c = 1; c < j->C; ++c) {
                if (rng_unit(&r) > j->p) continue;
                if (len >= j->t_cap) continue;
                int32_t first = 0;
                while (seq[first] != v) ++first;
                const int32_t idx = first + 1 + (int32_t)rng_below(&r, (uint32_t)(len - first));
                memmove(seq + idx + 1, seq + idx, (size_t)(len - idx) * sizeof(int32_t));
                seq[idx] = v;
                ++len;
            }
        }
        j->lens[b] = len;
    }
    free(deg); free(ready);
    return NULL;
}

/* Writes schedule b to seqs_strided[b*stride .. b*stride+lens[b]) (stride >= min(C*n, t_cap)).
 * The graph must be acyclic.  Returns 0, or -1 on bad arguments. */
int32_t wl_schedules(int32_t n, int64_t n_edges, const int32_t *edges, int32_t C, double p,
                     int32_t t_cap, int64_t B, uint64_t seed, int32_t n_threads, int64_t stride,
                     int32_t *seqs_strided, int32_t *lens) {
    if (n <= 0 || C < 1 || B < 0 || t_cap < n) return -1;
    int64_t *succ_start = (int64_t *)calloc((size_t)n + 1, sizeof(int64_t));
    int32_t *succ = (int32_t *)malloc((size_t)(n_edges > 0 ? n_edges : 1) * sizeof(int32_t));
    int32_t *indeg = (int32_t *)calloc((size_t)n, sizeof(int32_t));
    for (int64_t e = 0; e < n_edges; ++e) { succ_start[edges[2 * e] + 1]++; indeg[edges[2 * e + 1]]++; }
    for (int32_t v = 0; v < n; ++v) succ_start[v + 1] += succ_start[v];
    int64_t *fill = (int64_t *)malloc((size_t)n * sizeof(int64_t));
    memcpy(fill, succ_start, (size_t)n * sizeof(int64_t));
    for (int64_t e = 0; e < n_edges; ++e) succ[fill[edges[2 * e]]++] = edges[2 * e + 1];
    free(fill);
    if (n_threads < 1) n_threads = 1;
    if (n_threads > B) n_threads = (int32_t)(B > 0 ? B : 1);
    sched_job *jobs = (sched_job *)calloc((size_t)n_threads, sizeof(sched_job));
    pthread_t *th = (pthread_t *)calloc((size_t)n_threads, sizeof(pthread_t));
    for (int32_t i = 0; i < n_threads; ++i) {
        jobs[i] = (sched_job){n, C, t_cap, p, succ_start, succ, indeg, seed,
                              B * i / n_threads, B * (i + 1) / n_threads, stride, seqs_strided, lens};
        if (i > 0) pthread_create(&th[i], NULL, sched_worker, &jobs[i]);
    }
    sched_worker(&jobs[0]);
    for (int32_t i = 1; i < n_threads; ++i) pthread_join(th[i], NULL);
    free(th); free(jobs); free(succ_start); free(succ); free(indeg);
    return 0;
}

/* Packs strided schedules back to back: out[offs[b] .. offs[b]+lens[b]). Returns the total. */
int64_t wl_pack(int64_t B, int64_t stride, const int32_t *seqs_strided, const int32_t *lens, int32_t *out) {
    int64_t off = 0;
    for (int64_t b = 0; b < B; ++b) {
        memcpy(out + off, seqs_strided + b * stride, (size_t)lens[b] * sizeof(int32_t));
        off += lens[b];
    }
    return off;
}

/*
 * CPU oracle for the local search over rematerialization sequences (Moccasin, arXiv 2304.14463,
 * Section 3, "Optimization in Two Phases").
 *
 * TEST INFRASTRUCTURE ONLY, like moc_oracle.c: plain, sequential, shares nothing with the CUDA
 * path.  It is compiled into the same shared object as moc_oracle.c and calls its evaluator.
 *
 * What is computed.  P independent chains each hold one sequence with its evaluation (peak,
 * duration, status).  One generation proposes, per chain, one edited copy of the chain's sequence
 * (insert a further copy of a node, delete a copy, or move a copy), evaluates it with the
 * evaluator of moc_oracle.c and keeps it when it is not worse.  "Not worse" is the paper's two
 * phases folded into one lexicographic key:
 *     key(sequence) = ( max(peak, M), duration )            for status >= 0,  +infinity otherwise.
 * Phase 1 of the paper minimises max(M_var, M) with M_var the peak; Phase 2 minimises the duration
 * (Eq. 1) subject to peak <= M (Eq. 4).  While a chain is over budget the first component
 * decreases (Phase 1); once peak <= M it equals M for every accepted sequence, a proposal over
 * budget has a larger key and is refused, and only the duration decides (Phase 2).
 *
 * Random draws: one call of Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers:
 * as easy as 1, 2, 3", SC 2011) per chain and generation, counter = (generation, chain, 0, 0),
 * key = (low, high) 32 bits of the seed; "chain" is the chain's global number chain0 + c, so that a
 * population split over several runs (one per device) draws what the unsplit population draws.  The four output words r0..r3 select the edit:
 *     op = r0 mod 3                 0 insert, 1 delete, 2 move   (with all three kinds enabled; with
 *                                   a mask of k enabled kinds: the (r0 mod k)-th enabled one in
 *                                   this order.  "move" alone searches over the orders of a
 *                                   sequence without adding or removing copies.)
 *     q  = r1 mod T                 position of the copy the edit refers to
 *     insert:  j = r2 mod (T+1);  the node seq[q] is inserted in front of index j     (T+1 steps)
 *     delete:  element q is removed                                                   (T-1 steps)
 *     move:    element q is removed, then inserted in front of index j = r2 mod T
 *              of the shortened sequence                                              (T steps)
 * Several proposals per chain and generation ("samples" = E >= 1): proposal e = 0..E-1 uses counter
 * (generation, chain, e, 0); the chain's candidate is the proposal with the smallest key among those
 * with status >= 0 (the lowest e among equals), and it replaces the chain's sequence when it is not
 * worse than it.  E = 1 is the single proposal described above.
 * A chain with T = 0 proposes nothing.  Proposals are judged by the evaluator alone: a length
 * outside [n, C*n], a node left without a copy or with more than C copies all give status -2
 * there, and such a proposal is refused.
 *
 * Pins (tests/test_search_oracle.py): the generator against the known-answer vectors published
 * with its reference implementation; the edits against hand-written cases and a list-based
 * restatement; the acceptance rule against exhaustive enumeration on a tiny graph and the
 * invariants (key never increases, accepted sequences are valid, chains are independent).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* the evaluator of moc_oracle.c (same shared object) */
void moc_oracle_eval(const void *g, const int32_t *seq, int32_t T, int64_t M, int64_t *out_peak,
                     int64_t *out_dur, int32_t *out_status, int64_t *out_profile, int32_t *out_free);

/* ---- Philox4x32-10 (Salmon et al., SC 2011, Section 3.3 and Table 2: multipliers and Weyl
 * increments of the 4x32 variant; ten rounds).  One round maps (c0,c1,c2,c3) with round key
 * (k0,k1) to ( hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0) ); the key is
 * advanced by (W0, W1) between rounds. */
void moc_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += W0;
            k1 += W1;
        }
        const uint64_t p0 = M0 * c0, p1 = M1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * Applies the edit selected by (r0, r1, r2) among the enabled kinds to seq[0..T) and writes the
 * proposal to child (room for T+1 ints).  Returns the proposal's length, or -1 when T = 0 or no
 * kind is enabled (nothing to edit).
 */
int32_t moc_oracle_mutate(const int32_t *seq, int32_t T, uint32_t r0, uint32_t r1, uint32_t r2,
                          uint32_t kinds, int32_t *child) {
    if (T <= 0) return -1;
    /* kinds: bit 0 insert, bit 1 delete, bit 2 move; at least one is set */
    uint32_t enabled[3], k = 0;
    for (uint32_t o = 0; o < 3; ++o)
        if (kinds & (1u << o)) enabled[k++] = o;
    if (k == 0) return -1;
    const uint32_t op = enabled[r0 % k];
    const int32_t q = (int32_t)(r1 % (uint32_t)T);
    if (op == 0) { /* insert a further copy of seq[q] in front of index j */
        const int32_t j = (int32_t)(r2 % ((uint32_t)T + 1u));
        for (int32_t t = 0; t < j; ++t) child[t] = seq[t];
        child[j] = seq[q];
        for (int32_t t = j; t < T; ++t) child[t + 1] = seq[t];
        return T + 1;
    }
    /* delete and move both start by taking element q out */
    int32_t len = 0;
    for (int32_t t = 0; t < T; ++t)
        if (t != q) child[len++] = seq[t];
    if (op == 1) return len; /* T - 1 */
    const int32_t j = (int32_t)(r2 % (uint32_t)T); /* T = len + 1 insertion points */
    for (int32_t t = len; t > j; --t) child[t] = child[t - 1];
    child[j] = seq[q];
    return T;
}

/* 1 iff a sequence with evaluation (peak_c, dur_c, st_c) is not worse than (peak_p, dur_p, st_p)
 * under key = (max(peak, M), duration), invalid sequences (status < 0) ranking last; an invalid
 * proposal is never accepted. */
int32_t moc_oracle_accept(int64_t peak_c, int64_t dur_c, int32_t st_c, int64_t peak_p,
                          int64_t dur_p, int32_t st_p, int64_t M) {
    if (st_c < 0) return 0;
    if (st_p < 0) return 1;
    const int64_t a = peak_c > M ? peak_c : M, b = peak_p > M ? peak_p : M;
    if (a != b) return a < b;
    return dur_c <= dur_p;
}

/*
 * Runs generations gen0 .. gen0+n_gen-1 on P chains, in place.
 *   pop     P rows of `stride` ints, stride >= C*n (a proposal longer than the evaluator admits
 *           is refused before it is stored)
 *   lens    P lengths;  peak, dur, status: the evaluation of every chain's current sequence
 *           (the caller evaluates the initial population).
 *   chain0  global number of chain 0 (enters the random draws only).
 *   kinds   enabled kinds of edit (bit 0 insert, bit 1 delete, bit 2 move).
 *   samples proposals per chain and generation (>= 1).
 *   n_accepted (may be NULL) receives the number of accepted proposals.
 */
void moc_oracle_search_run(const void *g, int32_t *pop, int32_t *lens, int64_t *peak, int64_t *dur,
                           int32_t *status, int32_t P, int32_t stride, int64_t M, uint64_t seed,
                           uint32_t gen0, uint32_t n_gen, uint32_t chain0, uint32_t kinds, uint32_t samples,
                           int64_t *n_accepted) {
    int32_t *child = (int32_t *)malloc(((size_t)stride + 2) * sizeof(int32_t));
    int32_t *cand = (int32_t *)malloc(((size_t)stride + 2) * sizeof(int32_t));
    const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    int64_t acc = 0;
    for (uint32_t gen = gen0; gen < gen0 + n_gen; ++gen) {
        for (int32_t c = 0; c < P; ++c) {
            int32_t *row = pop + (size_t)c * stride;
            const int32_t T = lens[c];
            /* the chain's candidate: best valid proposal of this generation */
            int have = 0;
            int32_t cand_T = 0, cand_st = -2;
            int64_t cand_pk = -1, cand_du = -1;
            for (uint32_t e = 0; e < samples; ++e) {
                const uint32_t ctr[4] = {gen, chain0 + (uint32_t)c, e, 0u};
                uint32_t r[4];
                moc_oracle_philox4x32_10(ctr, key, r);
                const int32_t Tc = moc_oracle_mutate(row, T, r[0], r[1], r[2], kinds, child);
                if (Tc < 0) continue;
                int64_t pk, du;
                int32_t st;
                moc_oracle_eval(g, child, Tc, M, &pk, &du, &st, NULL, NULL);
                if (st < 0) continue;
                /* strictly better than the candidate so far: the lowest e wins among equals */
                if (!have || (moc_oracle_accept(pk, du, st, cand_pk, cand_du, cand_st, M) &&
                              !moc_oracle_accept(cand_pk, cand_du, cand_st, pk, du, st, M))) {
                    have = 1;
                    cand_T = Tc;
                    cand_pk = pk;
                    cand_du = du;
                    cand_st = st;
                    memcpy(cand, child, (size_t)Tc * sizeof(int32_t));
                }
            }
            if (!have) continue;
            if (!moc_oracle_accept(cand_pk, cand_du, cand_st, peak[c], dur[c], status[c], M)) continue;
            /* status >= 0 implies cand_T <= C*n <= stride */
            memcpy(row, cand, (size_t)cand_T * sizeof(int32_t));
            lens[c] = cand_T;
            peak[c] = cand_pk;
            dur[c] = cand_du;
            status[c] = cand_st;
            ++acc;
        }
    }
    if (n_accepted) *n_accepted = acc;
    free(child);
    free(cand);
}

/* Index of the best chain: smallest key (max(peak, M), duration), valid chains only, lowest index
 * among equals; -1 when no chain is valid. */
int32_t moc_oracle_search_best(const int64_t *peak, const int64_t *dur, const int32_t *status,
                               int32_t P, int64_t M) {
    int32_t best = -1;
    for (int32_t c = 0; c < P; ++c) {
        if (status[c] < 0) continue;
        if (best < 0) { best = c; continue; }
        const int64_t a = peak[c] > M ? peak[c] : M, b = peak[best] > M ? peak[best] : M;
        if (a < b || (a == b && dur[c] < dur[best])) best = c;
    }
    return best;
}

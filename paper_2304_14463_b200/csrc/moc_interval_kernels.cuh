// Device code of the interval-form checker: a batch of solutions in the paper's own variables
// (starts s, ends e, activity flags a of the retention intervals; Section 2, Eqs. 1-8, and the staged
// event domain of "Complexity Reduction by Enforcing an Initial Topological Ordering") is checked
// constraint by constraint, with the duration (Eq. 1) and the peak of the usage of Eq. 4.
//
// One block per solution at a time.  The event domain can be far larger than the number of intervals
// (n(n+1)/2 staged events for n*C intervals), so usage is not accumulated per event.  It can only
// rise at the start of an active interval, hence the peak is the largest usage over those start
// events.  A bitmap over the domain marks them, a prefix count over its words turns an event t into
// rank(t) = number of marked events <= t, and every active interval [s, e] with s <= e adds m to the
// marked events rank(s) .. rank(e): a difference array over at most n*C ranks and one prefix sum.
// The same ranks order the active intervals into the execution sequence the solution stands for.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace moc {

constexpr int kIvThreads = 256;
constexpr int32_t kIvEq2 = 1, kIvEq3 = 2, kIvEq4 = 4, kIvEq5 = 8, kIvEq6 = 16, kIvEq7 = 32, kIvEq8 = 64, kIvStage = 128;

struct IntervalParams {
    int32_t n, C;
    const int32_t* succ_start;   // n+1, successor lists (CSR)
    const int32_t* succ;
    const int64_t* w;            // n durations
    const int64_t* m;            // n output sizes
    const int32_t* s;            // B * n * C each, [B][n][C]
    const int32_t* e;
    const int32_t* a;
    int32_t B;
    int64_t D;                   // events are 1..D
    const int32_t* topo_index;   // n (1-based index in the input topological order): staged model; nullptr: plain
    int64_t M;
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_mask;
    int32_t* out_seqs;           // B rows of n*C ints, or nullptr
    int32_t* out_lens;           // B, or nullptr
    uint32_t words;              // bitmap words: (D + 32) / 32  (bit t of the bitmap = event t, bit 0 unused)
};

// Shared memory, in this order: bitmap of active starts [words], bitmap of all starts [words] (plain
// model only, else absent), rank base per word [words], difference array [n*C + 2] int64.
__host__ __device__ inline size_t interval_smem_bytes(uint32_t words, int64_t K, bool plain) {
    size_t b = (size_t)words * 4 * (plain ? 3 : 2);
    b = (b + 15) & ~size_t(15);
    return b + (size_t)(K + 2) * 8;
}

// exact test "x = j(j-1)/2 for an integer j >= jmin"; x >= 0
__device__ __forceinline__ bool is_triangular_from(int64_t x, int64_t jmin) {
    // j = (1 + sqrt(1 + 8x)) / 2, corrected to the integer root
    int64_t j = (int64_t)((1.0 + sqrt(1.0 + 8.0 * (double)x)) * 0.5);
    while (j * (j - 1) / 2 > x) --j;
    while ((j + 1) * j / 2 <= x) ++j;
    return j * (j - 1) / 2 == x && j >= jmin;
}

__global__ void __launch_bounds__(kIvThreads) check_intervals_kernel(const IntervalParams p) {
    extern __shared__ __align__(16) char smem[];
    __shared__ int32_t s_mask;
    __shared__ int32_t s_nactive;
    __shared__ int64_t s_red[kIvThreads / 32], s_red2[kIvThreads / 32];
    const bool plain = p.topo_index == nullptr;
    const int32_t n = p.n, C = p.C;
    const int64_t K = (int64_t)n * C;
    uint32_t* bm_act = reinterpret_cast<uint32_t*>(smem);
    uint32_t* bm_all = bm_act + p.words;                               // plain model only
    uint32_t* rbase = bm_act + (size_t)p.words * (plain ? 2 : 1);
    int64_t* delta = reinterpret_cast<int64_t*>(smem + ((((size_t)p.words * 4 * (plain ? 3 : 2)) + 15) & ~size_t(15)));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int32_t b = blockIdx.x; b < p.B; b += gridDim.x) {
        const int32_t* __restrict__ S = p.s + (int64_t)b * K;
        const int32_t* __restrict__ E = p.e + (int64_t)b * K;
        const int32_t* __restrict__ A = p.a + (int64_t)b * K;
        // ---- clear
        for (uint32_t i = tid; i < p.words * (plain ? 2u : 1u); i += kIvThreads) bm_act[i] = 0;
        for (int64_t i = tid; i < K + 2; i += kIvThreads) delta[i] = 0;
        if (tid == 0) { s_mask = 0; s_nactive = 0; }
        __syncthreads();

        // ---- per node: Eq. 8, then Eqs. 1, 2, 3, 7
        int32_t mask = 0;
        int64_t dur = 0;
        for (int32_t v = tid; v < n; v += kIvThreads) {
            const int64_t wv = __ldg(&p.w[v]);
            for (int32_t i = 0; i < C; ++i) {
                const int32_t sv = S[v * C + i], ev = E[v * C + i], av = A[v * C + i];
                if (sv < 1 || sv > p.D || ev < 1 || ev > p.D || (av != 0 && av != 1)) mask |= kIvEq8;
                if (sv > ev) mask |= kIvEq2;
                if (i + 1 < C && ev > S[v * C + i + 1]) mask |= kIvEq3;
                if (av == 1) dur += wv;
            }
            if (A[v * C] != 1) mask |= kIvEq7;
        }
        if (mask) atomicOr(&s_mask, mask);
        __syncthreads();
        if (s_mask & kIvEq8) {          // nothing else is evaluated (uniform: s_mask is shared)
            if (tid == 0) {
                p.out_mask[b] = kIvEq8;
                p.out_peak[b] = -1;
                p.out_dur[b] = -1;
                if (p.out_lens) p.out_lens[b] = -1;
            }
            __syncthreads();
            continue;
        }
        mask = 0;

        // ---- per node: mark the active starts; Eq. 6 (plain) or the staged rule
        for (int32_t v = tid; v < n; v += kIvThreads) {
            const int64_t k = plain ? 0 : (int64_t)__ldg(&p.topo_index[v]);
            if (!plain && (int64_t)S[v * C] != k * (k + 1) / 2) mask |= kIvStage;
            for (int32_t i = 0; i < C; ++i) {
                const int32_t sv = S[v * C + i];
                if (A[v * C + i] == 1) {
                    atomicOr(&bm_act[sv >> 5], 1u << (sv & 31));
                    if (!plain && !((int64_t)sv >= k && is_triangular_from((int64_t)sv - k, k))) mask |= kIvStage;
                }
                if (plain) {
                    // each node marks each of its distinct starts once: a bit found set belongs to another node
                    bool seen = false;
                    for (int32_t i2 = 0; i2 < i; ++i2) seen |= S[v * C + i2] == sv;
                    if (!seen) {
                        const uint32_t bit = 1u << (sv & 31);
                        if (atomicOr(&bm_all[sv >> 5], bit) & bit) mask |= kIvEq6;
                    }
                }
            }
        }
        __syncthreads();

        // ---- rank base of every bitmap word: exclusive prefix sum of the popcounts
        {
            const uint32_t per = (p.words + kIvThreads - 1) / kIvThreads;
            const uint32_t w0 = min(p.words, (uint32_t)tid * per), w1 = min(p.words, w0 + per);
            uint32_t cnt = 0;
            for (uint32_t i = w0; i < w1; ++i) cnt += __popc(bm_act[i]);
            uint32_t incl = cnt;
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d) incl += o;
            }
            if (lane == 31) s_red[warp] = incl;
            __syncthreads();
            uint32_t base = 0;
            for (int k2 = 0; k2 < warp; ++k2) base += (uint32_t)s_red[k2];
            uint32_t run = base + incl - cnt;
            for (uint32_t i = w0; i < w1; ++i) {
                rbase[i] = run;
                run += __popc(bm_act[i]);
            }
            if (tid == kIvThreads - 1) s_nactive = (int32_t)run;     // number of distinct active starts
        }
        __syncthreads();
        const int32_t R = s_nactive;
        auto rank = [&](int32_t t) -> int32_t {   // marked events <= t
            const uint32_t wd = bm_act[t >> 5];
            const uint32_t upto = (t & 31) == 31 ? wd : (wd & ((2u << (t & 31)) - 1u));
            return (int32_t)(rbase[t >> 5] + __popc(upto));
        };

        // ---- Eq. 4: every active interval with s <= e covers the marked events rank(s)..rank(e)
        int32_t total_active = 0;
        for (int64_t k = tid; k < K; k += kIvThreads) {
            if (A[k] != 1) continue;
            ++total_active;
            const int32_t sv = S[k], ev = E[k];
            const int32_t r = rank(sv);
            if (sv <= ev) {
                const int64_t mv = __ldg(&p.m[k / C]);
                atomicAdd(reinterpret_cast<unsigned long long*>(&delta[r]), (unsigned long long)mv);
                atomicAdd(reinterpret_cast<unsigned long long*>(&delta[rank(ev) + 1]), (unsigned long long)(-mv));
            }
        }
        // total number of active intervals (for the sequence: defined iff all their starts differ)
        {
            int32_t t = total_active;
            for (int d = 16; d > 0; d >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, d);
            if (lane == 0) s_red2[warp] = t;
        }
        __syncthreads();
        int32_t n_act_total = 0;
        for (int k2 = 0; k2 < kIvThreads / 32; ++k2) n_act_total += (int32_t)s_red2[k2];
        __syncthreads();

        // ---- prefix sum over the ranks 1..R and its maximum
        int64_t peak = 0;
        {
            const int32_t per = (R + kIvThreads - 1) / kIvThreads;
            const int32_t r0 = min(R, tid * per) + 1, r1 = min(R, tid * per + per) + 1;   // ranks [r0, r1)
            int64_t sum = 0, top = INT64_MIN;
            for (int32_t r = r0; r < r1; ++r) {
                sum += delta[r];
                top = sum > top ? sum : top;
            }
            int64_t incl = sum;
            for (int d = 1; d < 32; d <<= 1) {
                const int64_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d) incl += o;
            }
            if (lane == 31) s_red[warp] = incl;
            __syncthreads();
            int64_t base = 0;
            for (int k2 = 0; k2 < warp; ++k2) base += s_red[k2];
            int64_t best = r1 > r0 ? base + incl - sum + top : 0;
            for (int d = 16; d > 0; d >>= 1) {
                const int64_t o = __shfl_xor_sync(0xFFFFFFFFu, best, d);
                best = o > best ? o : best;
            }
            __syncthreads();
            if (lane == 0) s_red[warp] = best;
            __syncthreads();
            for (int k2 = 0; k2 < kIvThreads / 32; ++k2) peak = s_red[k2] > peak ? s_red[k2] : peak;
        }
        if (peak > p.M) mask |= kIvEq4;

        // ---- Eq. 5: every active interval of a successor starts inside an active interval of the producer
        for (int32_t u = tid; u < n; u += kIvThreads) {
            const int32_t e0 = __ldg(&p.succ_start[u]), e1 = __ldg(&p.succ_start[u + 1]);
            for (int32_t q = e0; q < e1; ++q) {
                const int32_t v = __ldg(&p.succ[q]);
                for (int32_t i = 0; i < C; ++i) {
                    if (A[v * C + i] != 1) continue;
                    const int32_t t = S[v * C + i];
                    bool found = false;
                    for (int32_t j = 0; j < C; ++j)
                        found |= A[u * C + j] == 1 && S[u * C + j] + 1 <= t && t <= E[u * C + j];
                    if (!found) mask |= kIvEq5;
                }
            }
        }

        // ---- the execution sequence: active intervals by rank of their start
        const bool has_seq = R == n_act_total;
        if (p.out_seqs != nullptr && has_seq) {
            int32_t* row = p.out_seqs + (int64_t)b * K;
            for (int64_t k = tid; k < K; k += kIvThreads)
                if (A[k] == 1) row[rank(S[k]) - 1] = (int32_t)(k / C);
        }

        // ---- duration, flags, outputs
        for (int d = 16; d > 0; d >>= 1) dur += __shfl_xor_sync(0xFFFFFFFFu, dur, d);
        __syncthreads();
        if (lane == 0) s_red[warp] = dur;
        if (mask) atomicOr(&s_mask, mask);
        __syncthreads();
        if (tid == 0) {
            int64_t total = 0;
            for (int k2 = 0; k2 < kIvThreads / 32; ++k2) total += s_red[k2];
            p.out_mask[b] = s_mask;
            p.out_peak[b] = peak;
            p.out_dur[b] = total;
            if (p.out_lens) p.out_lens[b] = has_seq ? R : -1;
        }
        __syncthreads();
    }
}

}  // namespace moc

// Device code of the interval-form checker: a batch of solutions in the paper's own variables
// (starts s, ends e, activity flags a of the retention intervals; Section 2, Eqs. 1-8, and the staged
// event domain of "Complexity Reduction by Enforcing an Initial Topological Ordering") is checked
// constraint by constraint, with the duration (Eq. 1) and the peak of the usage of Eq. 4.
//
// One warp per solution at a time, warp-synchronous (no block barriers); a block is a few warps that
// share nothing but the launch.  The event domain can be far larger than the number of intervals
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

constexpr int kIvMaxWarps = 8;   // warps (solutions in flight) per block, fewer when shared memory is short
constexpr int32_t kIvEq2 = 1, kIvEq3 = 2, kIvEq4 = 4, kIvEq5 = 8, kIvEq6 = 16, kIvEq7 = 32, kIvEq8 = 64, kIvStage = 128;
constexpr int kIvMaxC = 8;       // slots per node held in registers

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
    int32_t D;                   // events are 1..D
    const int32_t* topo_index;   // n (1-based index in the input topological order): staged model; nullptr: plain
    int64_t M;
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_mask;
    int32_t* out_seqs;           // B rows of n*C ints, or nullptr
    int32_t* out_lens;           // B, or nullptr
    uint32_t words;              // bitmap words: (D + 32) / 32  (bit t of the bitmap = event t, bit 0 unused)
    uint32_t warp_bytes;         // shared memory of one warp
    int32_t byte_marks;          // plain model, and two bytes per event fit the space of the difference array
};

// Shared memory of one warp, in this order: bitmap of active starts [words], bitmap of all starts
// [words] (plain model only, else absent), rank base per word [words], difference array [n*C + 2]
// (MemT), then -- when it fits -- the solution: start of every active slot (0 = inactive) and end of
// every slot, [n*C] int32 each, written while the solution is read from HBM for the only time.
__host__ __device__ inline size_t interval_bitmap_bytes(uint32_t words, bool plain) {
    return (((size_t)words * 4 * (plain ? 3 : 2)) + 15) & ~size_t(15);
}
__host__ __device__ inline size_t interval_clear_bytes(uint32_t words, int64_t K, bool plain, size_t mem_sz) {
    return interval_bitmap_bytes(words, plain) + (((size_t)(K + 2) * mem_sz + 15) & ~size_t(15));
}
__host__ __device__ inline size_t interval_stage_bytes(int64_t K, size_t pos_sz) { return ((size_t)K * 2 * pos_sz + 15) & ~size_t(15); }

// exact test "x = j(j-1)/2 for an integer j >= jmin"; x >= 0
__device__ __forceinline__ bool is_triangular_from(int64_t x, int64_t jmin) {
    // j = (1 + sqrt(1 + 8x)) / 2, corrected to the integer root
    int64_t j = (int64_t)((1.0 + sqrt(1.0 + 8.0 * (double)x)) * 0.5);
    while (j * (j - 1) / 2 > x) --j;
    while ((j + 1) * j / 2 <= x) ++j;
    return j * (j - 1) / 2 == x && j >= jmin;
}

__device__ __forceinline__ void iv_add(int32_t* p, int32_t v) { atomicAdd(p, v); }
__device__ __forceinline__ void iv_add(int64_t* p, int64_t v) {
    atomicAdd(reinterpret_cast<unsigned long long*>(p), (unsigned long long)v);
}

// kPlain: plain model (Eq. 6) or staged model; CP: slots per node held in registers (>= C); MemT: type
// of the usage sums (int32 when C * sum(m) < 2^31); kStage: the solution is kept in shared memory
// after the first pass (otherwise the second pass reads it again through L1/L2), as PosT (uint16 when
// D < 65536).
template <bool kPlain, int CP, typename MemT, bool kStage, typename PosT>
__global__ void __launch_bounds__(32 * kIvMaxWarps) check_intervals_kernel(const IntervalParams p) {
    extern __shared__ __align__(16) char smem[];
    const int lane = threadIdx.x & 31;
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const int wpb = blockDim.x >> 5;
    const int32_t n = p.n, C = p.C, K = n * C;
    char* ws = smem + (size_t)warp * p.warp_bytes;
    uint32_t* bm_act = reinterpret_cast<uint32_t*>(ws);
    uint32_t* bm_all = bm_act + p.words;                               // plain model only
    uint32_t* rbase = bm_act + p.words * (kPlain ? 2u : 1u);
    MemT* delta = reinterpret_cast<MemT*>(ws + interval_bitmap_bytes(p.words, kPlain));
    PosT* sS = reinterpret_cast<PosT*>(ws + interval_clear_bytes(p.words, K, kPlain, sizeof(MemT)));
    PosT* sE = sS + K;
    // plain model: two bytes per event during pass 1 (active start, any start), in the space of the difference
    // array when it is large enough (byte_marks)
    const uint32_t by_stride = ((uint32_t)p.D + 1u + 15u) & ~15u;
    uint8_t* by_act = reinterpret_cast<uint8_t*>(delta);
    constexpr uint32_t kFull = 0xFFFFFFFFu;
    const int nz = (int)(interval_clear_bytes(p.words, K, kPlain, sizeof(MemT)) >> 4);

    for (int32_t b = blockIdx.x * wpb + warp; b < p.B; b += gridDim.x * wpb) {
        const int32_t* __restrict__ gs = p.s + (int64_t)b * K;
        const int32_t* __restrict__ ge = p.e + (int64_t)b * K;
        const int32_t* __restrict__ ga = p.a + (int64_t)b * K;
        {
            int4* z4 = reinterpret_cast<int4*>(ws);
            for (int i = lane; i < nz; i += 32) z4[i] = make_int4(0, 0, 0, 0);
        }
        __syncwarp();
        // C = 2 and the three rows of this solution start on 8 bytes: slots are read in pairs
        const bool pairs = C == 2 && ((reinterpret_cast<uintptr_t>(gs) | reinterpret_cast<uintptr_t>(ge) | reinterpret_cast<uintptr_t>(ga)) & 7) == 0;

        // ---- pass 1, per node: read the C slots; Eq. 8; Eqs. 1, 2, 3, 7; mark the starts in the bitmaps
        // (Eq. 6 / staged rule).  A start outside the domain marks nothing; the marks are used only when
        // Eq. 8 holds everywhere.
        int32_t mask = 0, n_act = 0, n_distinct = 0;
        int64_t dur = 0;
        for (int32_t v = lane; v < n; v += 32) {
            int32_t sv[CP], ev[CP], av[CP];
            if (CP == 2 && pairs) {                         // two slots per node: one 8-byte load per array
                const int2 s2 = __ldg(reinterpret_cast<const int2*>(gs) + v), e2 = __ldg(reinterpret_cast<const int2*>(ge) + v),
                           a2 = __ldg(reinterpret_cast<const int2*>(ga) + v);
                sv[0] = s2.x; sv[1] = s2.y;
                ev[0] = e2.x; ev[1] = e2.y;
                av[0] = a2.x; av[1] = a2.y;
            } else {
#pragma unroll
                for (int i = 0; i < CP; ++i) {
                    const bool in = i < C;
                    sv[i] = in ? __ldg(gs + v * C + i) : 0;
                    ev[i] = in ? __ldg(ge + v * C + i) : 0;
                    av[i] = in ? __ldg(ga + v * C + i) : 0;
                }
            }
            const int64_t wv = __ldg(&p.w[v]);
            int64_t k = 0;
            if (!kPlain) {
                k = (int64_t)__ldg(&p.topo_index[v]);
                if ((int64_t)sv[0] != k * (k + 1) / 2) mask |= kIvStage;
            }
            if (av[0] != 1) mask |= kIvEq7;
            if (kStage && CP == 2 && sizeof(PosT) == 2 && C == 2) {       // both slots in one 32-bit store per array
                reinterpret_cast<uint32_t*>(sS)[v] = (uint32_t)(uint16_t)(av[0] == 1 ? sv[0] : 0) | (uint32_t)(uint16_t)(av[1] == 1 ? sv[1] : 0) << 16;
                reinterpret_cast<uint32_t*>(sE)[v] = (uint32_t)(uint16_t)ev[0] | (uint32_t)(uint16_t)ev[1] << 16;
            }
#pragma unroll
            for (int i = 0; i < CP; ++i) {
                if (i < C) {
                    const bool in_dom = sv[i] >= 1 && sv[i] <= p.D;
                    if (!in_dom || ev[i] < 1 || ev[i] > p.D || (av[i] != 0 && av[i] != 1)) mask |= kIvEq8;
                    if (sv[i] > ev[i]) mask |= kIvEq2;
                    if (i + 1 < CP && i + 1 < C && ev[i] > sv[i + 1]) mask |= kIvEq3;
                    const bool act = av[i] == 1;
                    if (act) { dur += wv; ++n_act; }
                    if (kStage && !(CP == 2 && sizeof(PosT) == 2 && C == 2)) {
                        sS[v * C + i] = (PosT)(act ? sv[i] : 0);
                        sE[v * C + i] = (PosT)ev[i];
                    }
                    if (in_dom) {
                        // Each node marks its distinct starts; Eq. 6 holds iff no two nodes marked the same event,
                        // i.e. iff as many events end up marked as marks were made.  With byte marks (plain
                        // stores: marks of neighbouring events share a word without colliding) the two bitmaps
                        // are made from the bytes below; otherwise the marks go straight into them.
                        const uint32_t bit = 1u << (sv[i] & 31);
                        if (act) {
                            if (kPlain && p.byte_marks) by_act[2 * sv[i]] = 1;
                            else atomicOr(&bm_act[sv[i] >> 5], bit);
                            if (!kPlain && !((int64_t)sv[i] >= k && is_triangular_from((int64_t)sv[i] - k, k))) mask |= kIvStage;
                        }
                        if (kPlain) {
                            bool seen = false;
#pragma unroll
                            for (int i2 = 0; i2 < i; ++i2) seen |= sv[i2] == sv[i];
                            if (!seen) {
                                if (p.byte_marks) by_act[2 * sv[i] + 1] = 1;
                                else atomicOr(&bm_all[sv[i] >> 5], bit);
                                ++n_distinct;
                            }
                        }
                    }
                }
            }
        }
        if (__any_sync(kFull, mask & kIvEq8)) {     // nothing else is evaluated
            if (lane == 0) {
                p.out_mask[b] = kIvEq8;
                p.out_peak[b] = -1;
                p.out_dur[b] = -1;
                if (p.out_lens) p.out_lens[b] = -1;
            }
            __syncwarp();
            continue;
        }
        __syncwarp();
        if (kPlain && p.byte_marks) {
            // bytes -> bitmaps: the warp reads the byte pairs of 32 consecutive events, the two ballots are their
            // bitmap words, kept by lane (word mod 32) and stored 32 words at a time; then the bytes, which
            // borrowed the difference array, are cleared again
            const uint16_t* by2 = reinterpret_cast<const uint16_t*>(by_act);
            for (uint32_t w0 = 0; w0 < p.words; w0 += 32) {
                uint32_t keep_a = 0, keep_l = 0;
                const uint32_t w1 = min(p.words, w0 + 32u);
                for (uint32_t wd = w0; wd < w1; ++wd) {
                    const int32_t t = (int32_t)(wd * 32u) + lane;
                    const uint32_t pr = t <= p.D ? (uint32_t)by2[t] : 0u;
                    const uint32_t ba = __ballot_sync(kFull, (pr & 0xFFu) != 0), bl = __ballot_sync(kFull, (pr >> 8) != 0);
                    if (lane == (int)(wd - w0)) {
                        keep_a = ba;
                        keep_l = bl;
                    }
                }
                if (w0 + lane < w1) {
                    bm_act[w0 + lane] = keep_a;
                    bm_all[w0 + lane] = keep_l;
                }
            }
            __syncwarp();
            int4* z4 = reinterpret_cast<int4*>(by_act);
            for (uint32_t i = lane; i < (2u * by_stride + 15u) / 16u; i += 32) z4[i] = make_int4(0, 0, 0, 0);
            __syncwarp();
        }

        // ---- rank base of every bitmap word: exclusive prefix sum of the popcounts
        int32_t R;
        {
            const uint32_t per = (p.words + 31) / 32;
            const uint32_t w0 = min(p.words, (uint32_t)lane * per), w1 = min(p.words, w0 + per);
            uint32_t cnt = 0;
            for (uint32_t i = w0; i < w1; ++i) cnt += __popc(bm_act[i]);
            uint32_t incl = cnt;
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_up_sync(kFull, incl, d);
                if (lane >= d) incl += o;
            }
            uint32_t run = incl - cnt;
            for (uint32_t i = w0; i < w1; ++i) {
                rbase[i] = run;
                run += __popc(bm_act[i]);
            }
            R = (int32_t)__shfl_sync(kFull, incl, 31);       // number of distinct active starts
        }
        int32_t total_act = n_act;
        for (int d = 16; d > 0; d >>= 1) total_act += __shfl_xor_sync(kFull, total_act, d);
        if (kPlain) {
            int32_t bits = 0;
            for (uint32_t i = lane; i < p.words; i += 32) bits += __popc(bm_all[i]);
            bits = __reduce_add_sync(kFull, bits);
            if (bits != __reduce_add_sync(kFull, n_distinct)) mask |= kIvEq6;
        }
        const bool has_seq = R == total_act;
        int32_t* row = (p.out_seqs != nullptr && has_seq) ? p.out_seqs + (int64_t)b * K : nullptr;
        __syncwarp();
        auto rank = [&](int32_t t) -> int32_t {   // marked events <= t
            const uint32_t wd = bm_act[t >> 5];
            return (int32_t)(rbase[t >> 5] + __popc(wd & (0xFFFFFFFFu >> (31 - (t & 31)))));
        };
        // start (0 = inactive) and end of slot i of node v
        // both slots of node v at once (C = 2, positions staged in 16 bits)
        constexpr bool kPairStage = kStage && CP == 2 && sizeof(PosT) == 2;
        auto start_pair = [&](int32_t v) -> uint32_t { return reinterpret_cast<const uint32_t*>(sS)[v]; };
        auto end_pair = [&](int32_t v) -> uint32_t { return reinterpret_cast<const uint32_t*>(sE)[v]; };
        auto slot = [&](int32_t v, int32_t i, int32_t& s_out, int32_t& e_out) {
            if (kStage) {
                s_out = (int32_t)sS[v * C + i];
                e_out = (int32_t)sE[v * C + i];
            } else {
                s_out = __ldg(ga + v * C + i) == 1 ? __ldg(gs + v * C + i) : 0;
                e_out = __ldg(ge + v * C + i);
            }
        };

        // ---- pass 2, per node u: Eq. 4 (its active intervals with s <= e cover the marked events
        // rank(s)..rank(e)), the sequence, and Eq. 5 for its successors
        for (int32_t u = lane; u < n; u += 32) {
            int32_t us[CP], ue[CP];
            const MemT mv = (MemT)__ldg(&p.m[u]);
            if (kPairStage && C == 2) {
                const uint32_t sp = start_pair(u), ep = end_pair(u);
                us[0] = (int32_t)(sp & 0xFFFFu); us[1] = (int32_t)(sp >> 16);
                ue[0] = (int32_t)(ep & 0xFFFFu); ue[1] = (int32_t)(ep >> 16);
            } else {
#pragma unroll
                for (int j = 0; j < CP; ++j) {
                    us[j] = 0;
                    ue[j] = 0;
                    if (j < C) slot(u, j, us[j], ue[j]);
                }
            }
#pragma unroll
            for (int j = 0; j < CP; ++j) {
                if (us[j] != 0) {
                    const int32_t r = rank(us[j]);
                    if (us[j] <= ue[j]) {
                        iv_add(&delta[r], mv);
                        iv_add(&delta[rank(ue[j]) + 1], (MemT)(-mv));
                    }
                    if (row) row[r - 1] = u;
                } else {
                    us[j] = INT32_MAX - 1;      // an inactive slot serves nobody
                    ue[j] = 0;
                }
            }
            // Eq. 5: every active start t of a successor lies in (us, ue] of one slot of u, tested as
            // (t - lo) <= len in unsigned arithmetic with lo = us + 1, len = ue - lo; a slot that serves nobody
            // (inactive, or ue <= us) gets lo = 2^32 - 1, len = 0, which no t >= 1 satisfies
            uint32_t lo5[CP], len5[CP];
#pragma unroll
            for (int j = 0; j < CP; ++j) {
                const bool serves = ue[j] > us[j];
                lo5[j] = serves ? (uint32_t)us[j] + 1u : 0xFFFFFFFFu;
                len5[j] = serves ? (uint32_t)(ue[j] - us[j] - 1) : 0u;
            }
            const int32_t e0 = __ldg(&p.succ_start[u]), e1 = __ldg(&p.succ_start[u + 1]);
            for (int32_t q = e0; q < e1; ++q) {
                const int32_t v = __ldg(&p.succ[q]);
                uint32_t tp = 0;
                if (kPairStage && C == 2) tp = start_pair(v);
#pragma unroll
                for (int i = 0; i < CP; ++i) {
                    if (i < C) {
                        int32_t t, te = 0;
                        if (kPairStage && C == 2) t = (int32_t)(i == 0 ? tp & 0xFFFFu : tp >> 16);
                        else slot(v, i, t, te);
                        bool found = t == 0;                    // an inactive slot of the successor asks for nothing
#pragma unroll
                        for (int j = 0; j < CP; ++j) found |= (uint32_t)t - lo5[j] <= len5[j];
                        if (!found) mask |= kIvEq5;
                    }
                }
            }
        }
        __syncwarp();

        // ---- prefix sum over the ranks 1..R and its maximum: lane owns a run of consecutive ranks
        int64_t peak;
        {
            const int32_t per = (R + 31) / 32;
            const int32_t r0 = min(R, lane * per) + 1, r1 = min(R, lane * per + per) + 1;   // ranks [r0, r1)
            int64_t sum = 0, top = INT64_MIN;
            for (int32_t r = r0; r < r1; ++r) {
                sum += (int64_t)delta[r];
                top = sum > top ? sum : top;
            }
            int64_t incl = sum;
            for (int d = 1; d < 32; d <<= 1) {
                const int64_t o = __shfl_up_sync(kFull, incl, d);
                if (lane >= d) incl += o;
            }
            peak = r1 > r0 ? incl - sum + top : 0;
            for (int d = 16; d > 0; d >>= 1) {
                const int64_t o = __shfl_xor_sync(kFull, peak, d);
                peak = o > peak ? o : peak;
            }
        }
        if (peak > p.M) mask |= kIvEq4;

        // ---- duration, flags, outputs
        for (int d = 16; d > 0; d >>= 1) dur += __shfl_xor_sync(kFull, dur, d);
        mask = __reduce_or_sync(kFull, mask);
        if (lane == 0) {
            p.out_mask[b] = mask;
            p.out_peak[b] = peak;
            p.out_dur[b] = dur;
            if (p.out_lens) p.out_lens[b] = has_seq ? R : -1;
        }
        __syncwarp();
    }
}

}  // namespace moc

// Block-per-sequence path of the evaluator for up to four copies per node (the paper's cap C_v,
// Section 2; its experiments use 2, larger caps trade more recomputation for memory): a thread
// block evaluates one sequence at a time with the positions of a node's copies packed into one
// 64-bit word, so that a consumer reads all copies of a successor with one load and compares them
// two at a time with packed 16-bit arithmetic.
//
// Representation.  Positions are 1-based and 16 bits wide (sequences of at most 32766 steps: the packed
// comparisons tell earlier from later by the sign of a 16-bit difference).  After
// stage 1b a node's word holds its copies in ascending order; a node with fewer than four copies
// repeats its last copy in the remaining quarters, so that no quarter is empty.
//
// Stages for one sequence seq[0..T) (paper: Section 2, Eqs. 1-8):
//   1a. occurrence words  step t takes the next free quarter of its node's word (a 16-bit counter per
//                         node, two counters per 32-bit atomic) and stores t + 1 there.
//   1b. per node          count in [1, min(C, C_v)] (Eq. 7 and the cap), duration += count * w
//                         (Eq. 1); the quarters are sorted with a five-comparator network on packed
//                         halves (empty quarters last) and the empty ones filled with the last copy;
//                         delta[p - 1] = m for every copy p ("+m at the copy's own step" of stage 3:
//                         a plain store, every step belongs to exactly one copy).
//   2.  free steps        one thread per node u with copies a_1 <= ... <= a_4, nodes taken in order of
//                         falling out-degree so that the lanes of a warp run about the same number of
//                         rounds; per successor word r (both halves, two packed operations each):
//                           G_0 = max (r - a_1) mod 2^16        2^15 or more: a successor copy before
//                                                               the first copy (Eq. 5 violated); else
//                                                               a_1 + G_0 is the latest successor copy,
//                                                               until which the last copy is kept;
//                           G_i = max (r - a_{i+1}) mod 2^16    ranks the successor copies below
//                                                               a_{i+1} above all others: the latest
//                                                               one inside (a_i, a_{i+1}), until which
//                                                               copy i is kept (Eqs. 2, 3, 5); seeded
//                                                               with a_i - a_{i+1}: else a_i itself.
//                         A sink's only successor is a made-up word that holds T in every quarter.
//   3.  memory profile    delta[free + 1] -= m_u per copy, prefix sum over the steps (Eq. 4).
//   4.  reductions        peak (Section 2), status against the budget.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "moc_pair_kernel.cuh"

namespace moc {

struct QuadParams {
    int32_t n;
    int32_t C;                 // 3 or 4 accumulators are compiled; C itself bounds the copy count
    int32_t max_T;             // C * n
    int32_t B;
    int64_t M;
    const uint4* order;        // n records of 32 bytes in order of falling out-degree (below)
    const uint16_t* succ;      // the successors beyond the eighth of the nodes that have more
    const void* m;             // n output sizes, int32 or int64
    const int64_t* w;          // n durations
    const int32_t* cap;        // n per-node caps, or nullptr
    const int32_t* seqs;
    const int32_t* lens;
    const int64_t* offs;       // B + 1 row offsets
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_status;
    uint32_t word_bytes;       // 8 (n + 2), rounded to 16
    uint32_t cnt_bytes;        // 2 (n + 2), rounded to 16
};

// Node record: word 0 = node | out-degree << 16 (a sink: 1, its successor the id n + 1), word 1 = index
// of its ninth successor in `succ`, words 2-3 = m (int32: word 2), words 4-7 = its first eight successor
// ids, 16 bits each.

__device__ __forceinline__ void sts_u64(uint32_t addr, uint64_t v) {
    asm volatile("st.shared.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t atom_add_shared_u32(uint32_t addr, uint32_t v) {
    uint32_t old;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}

// Ascending sort of four 16-bit keys held as (k0, k1) in lo and (k2, k3) in hi: comparators (0,2)(1,3),
// (0,1)(2,3), (1,2), each on packed halves.
__device__ __forceinline__ void sort4_u16(uint32_t& lo, uint32_t& hi) {
    const uint32_t a = min_u16x2(lo, hi), b = max_u16x2(lo, hi);
    const uint32_t as = swap_halves(a), bs = swap_halves(b);
    const uint32_t a2 = __byte_perm(min_u16x2(a, as), max_u16x2(a, as), 0x7610);   // (min, max) of a
    const uint32_t b2 = __byte_perm(min_u16x2(b, bs), max_u16x2(b, bs), 0x7610);
    const uint32_t x = __byte_perm(a2, b2, 0x5432), y = swap_halves(x);            // (a2.hi, b2.lo) and swapped
    lo = __byte_perm(a2, min_u16x2(x, y), 0x5410);
    hi = __byte_perm(max_u16x2(x, y), b2, 0x7610);
}
__device__ __forceinline__ uint32_t max_halves(uint32_t v) { return max_u16x2(v, swap_halves(v)) & 0xFFFFu; }

// kAcc: number of copies the node pass keeps apart (3 or 4).
template <typename MemT, int kAcc>
__global__ void __launch_bounds__(1024) eval_quad_kernel(const QuadParams p) {
    extern __shared__ __align__(16) char smem[];
    __shared__ int64_t s_dur[32];
    __shared__ MemT s_sum[32], s_top[32];
    __shared__ uint32_t s_flags;
    constexpr int kShift = sizeof(MemT) == 4 ? 2 : 3;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, n_warps = nthr >> 5;
    int n = p.n;
    MOC_KEEP(n);
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(smem);
    uint32_t wa = sbase, ca = sbase + p.word_bytes, da = ca + p.cnt_bytes;   // words | counters | delta[0..]
    MOC_KEEP(wa);
    MOC_KEEP(ca);
    MOC_KEEP(da);
    const MemT* gm = reinterpret_cast<const MemT*>(p.m);

    for (int b = blockIdx.x; b < p.B; b += gridDim.x) {
        const int64_t off = __ldg(p.offs + b);
        const int32_t T = __ldg(p.lens + b);
        int64_t out_pk = -1, out_du = -1;
        int32_t out_st = -2;
        if (T >= n && T <= p.max_T) {      // uniform over the block
            // ---- clear words and counters (stage 1a writes every delta the prefix sum reads)
            {
                const int4 z = make_int4(0, 0, 0, 0);
                int4* s4 = reinterpret_cast<int4*>(smem);
                const int nz = (int)((p.word_bytes + p.cnt_bytes) >> 4);
                for (int i = tid; i < nz; i += nthr) s4[i] = z;
                if (tid == 0) s_flags = 0;
            }
            __syncthreads();
            // ---- stage 1a
            uint32_t flags = 0;    // bit 0: malformed, bit 1: precedence violated
            {
                const int32_t* row = p.seqs + off;
                auto put = [&](uint32_t id, int t) {
                    if (id < (uint32_t)n) {
                        const uint32_t sh = (id & 1u) << 4;
                        const uint32_t k = (atom_add_shared_u32(ca + ((id >> 1) << 2), 1u << sh) >> sh) & 0xFFFFu;
                        if (k < 4) sts_u16(wa + (id << 3) + (k << 1), (uint32_t)t + 1u);
                    } else {
                        flags = 1;
                    }
                };
                int t = tid;
                for (; t + 3 * nthr < T; t += 4 * nthr) {      // four loads in flight per thread
                    const uint32_t i0 = (uint32_t)__ldg(row + t), i1 = (uint32_t)__ldg(row + t + nthr),
                                   i2 = (uint32_t)__ldg(row + t + 2 * nthr), i3 = (uint32_t)__ldg(row + t + 3 * nthr);
                    put(i0, t);
                    put(i1, t + nthr);
                    put(i2, t + 2 * nthr);
                    put(i3, t + 3 * nthr);
                }
                for (; t < T; t += nthr) put((uint32_t)__ldg(row + t), t);
                if (tid == 0) sts_u64(wa + ((uint32_t)(n + 1) << 3), (uint64_t)(uint32_t)T * 0x0001000100010001ull);
            }
            __syncthreads();
            // ---- stage 1b
            int64_t dur = 0;
            for (int v = tid; v < n; v += nthr) {
                const uint32_t c = (lds_u32(ca + ((uint32_t)(v >> 1) << 2)) >> ((v & 1) << 4)) & 0xFFFFu;
                uint32_t limit = (uint32_t)p.C;
                if (p.cap != nullptr) limit = min(limit, (uint32_t)__ldg(p.cap + v));
                if (c < 1 || c > limit) flags |= 1;
                dur += (int64_t)c * __ldg(p.w + v);
                const uint2 q = lds_v2(wa + ((uint32_t)v << 3));
                // keys x - 1: an empty quarter becomes the largest key and sorts last
                uint32_t lo = __viaddmin_u16x2(q.x, 0xFFFFFFFFu, 0xFFFFFFFFu), hi = __viaddmin_u16x2(q.y, 0xFFFFFFFFu, 0xFFFFFFFFu);
                const uint32_t top = max_halves(max_u16x2(q.x, q.y));                  // the last copy
                const uint32_t cap_key = (top - 1u) * 0x10001u;
                sort4_u16(lo, hi);
                lo = __viaddmax_u16x2(min_u16x2(lo, cap_key), 0x00010001u, 0u);        // back to positions, empties = last copy
                hi = __viaddmax_u16x2(min_u16x2(hi, cap_key), 0x00010001u, 0u);
                sts_u64(wa + ((uint32_t)v << 3), (uint64_t)lo | ((uint64_t)hi << 32));
                // +m at every copy's own step; repeated quarters write the same value to the same place.  Only
                // for a node with a valid count: then every quarter is a step of the row (1..T); the word of an
                // absent or overfull node holds no usable positions and the sequence is malformed anyway.
                if (c >= 1 && c <= limit) {
                    const MemT mv = __ldg(gm + v);
                    const uint32_t dm1 = da - (uint32_t)sizeof(MemT);
                    sts_mem(dm1 + ((lo & 0xFFFFu) << kShift), mv);
                    sts_mem(dm1 + ((lo >> 16) << kShift), mv);
                    sts_mem(dm1 + ((hi & 0xFFFFu) << kShift), mv);
                    sts_mem(dm1 + ((hi >> 16) << kShift), mv);
                }
            }
            flags = __reduce_or_sync(0xFFFFFFFFu, flags);
            dur = warp_sum64(dur);
            if (lane == 0) {
                if (flags) atomicOr(&s_flags, flags);
                s_dur[warp] = dur;
            }
            __syncthreads();
            const bool malformed = (s_flags & 1u) != 0;
            if (!malformed) {
                // ---- stage 2 and the scatter of stage 3
                uint32_t depw = 0;
                const int n_round = (n + 31) & ~31;
                for (int i = tid; i < n_round; i += nthr) {
                    uint32_t node = 0, deg = 0, e8 = 0;
                    uint4 inl = make_uint4(0, 0, 0, 0);
                    MemT neg_m = 0;
                    if (i < n) {
                        const uint4 r = __ldg(p.order + 2 * i);
                        inl = __ldg(p.order + 2 * i + 1);
                        node = r.x & 0xFFFFu;
                        deg = r.x >> 16;
                        e8 = r.y;
                        if constexpr (sizeof(MemT) == 4) neg_m = -(MemT)r.z;
                        else neg_m = -(MemT)((uint64_t)r.z | ((uint64_t)r.w << 32));
                    }
                    const int rounds = __reduce_max_sync(0xFFFFFFFFu, (int)deg);
                    const uint2 own = lds_v2(wa + (node << 3));
                    // copies a_1..a_4 ascending: own.x = (a_1, a_2), own.y = (a_3, a_4)
                    uint32_t base[kAcc], na[kAcc], G[kAcc];
                    base[0] = own.x & 0xFFFFu;
                    base[1] = own.x >> 16;
                    base[2] = own.y & 0xFFFFu;
                    if constexpr (kAcc == 4) base[3] = own.y >> 16;
                    const uint32_t last = own.y >> 16;
#pragma unroll
                    for (int j = 0; j < kAcc; ++j) na[j] = 0x00010000u - base[j] * 0x10001u;     // (-a, -a) mod 2^16
                    G[0] = (last - base[0]) * 0x10001u;                                          // the last copy ends at itself at least
#pragma unroll
                    for (int j = 1; j < kAcc; ++j) G[j] = ((base[j - 1] - base[j]) & 0xFFFFu) * 0x10001u;   // copy j ends at itself at least
                    auto visit = [&](uint32_t sid) {
                        const uint2 r = lds_v2(wa + (sid << 3));
#pragma unroll
                        for (int j = 0; j < kAcc; ++j) {
                            G[j] = __viaddmax_u16x2(r.x, na[j], G[j]);
                            G[j] = __viaddmax_u16x2(r.y, na[j], G[j]);
                        }
                    };
                    const uint32_t in8[4] = {inl.x, inl.y, inl.z, inl.w};
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (k < rounds) {
                            if ((uint32_t)k < deg) visit((k & 1) ? in8[k >> 1] >> 16 : in8[k >> 1] & 0xFFFFu);
                        }
                    }
                    for (int k = 8; k < rounds; ++k)
                        if ((uint32_t)k < deg) visit((uint32_t)__ldg(p.succ + e8 + (k - 8)));
                    if (i < n) {
                        const uint32_t g0 = max_halves(G[0]);
                        depw |= g0;                                           // bit 15: a successor copy before a_1
                        red_add_shared(da + (((base[0] + g0) & 0xFFFFu) << kShift), neg_m);
#pragma unroll
                        for (int j = 1; j < kAcc; ++j) {
                            if (base[j] != base[j - 1]) {                    // copy j exists apart from copy j + 1
                                const uint32_t x = (base[j] + max_halves(G[j])) & 0xFFFFu;
                                red_add_shared(da + (x << kShift), neg_m);
                            }
                        }
                    }
                }
                if (__any_sync(0xFFFFFFFFu, (depw & 0x8000u) != 0) && lane == 0) atomicOr(&s_flags, 2u);
            }
            __syncthreads();
            const uint32_t fl = s_flags;
            if (!(fl & 1u)) {
                out_du = 0;
                for (int k = 0; k < n_warps; ++k) out_du += s_dur[k];
                out_st = -1;
            }
            if (fl == 0) {
                // ---- stages 3 and 4: prefix sum, each thread a chunk of consecutive steps (odd length: no bank conflicts)
                const int chunk = ((T + nthr - 1) / nthr) | 1;
                const int tb = min(tid * chunk, T), te = min(tb + chunk, T);
                MemT run = 0, top = 0;
                uint32_t ad = da + ((uint32_t)tb << kShift);
                for (int t = tb; t < te; ++t, ad += (uint32_t)sizeof(MemT)) {
                    run += lds_mem(ad, MemT());
                    top = (t == tb || run > top) ? run : top;
                }
                // chunk sums -> usage in front of every chunk; a thread without steps passes its prefix on
                MemT incl = warp_inclusive_sum(run, lane);
                if (lane == 31) s_sum[warp] = incl;
                __syncthreads();
                MemT before = incl - run;
                for (int k = 0; k < warp; ++k) before += s_sum[k];
                MemT peak = tb < te ? before + top : MemT(0);
                peak = warp_max_t(peak);
                if (lane == 0) s_top[warp] = peak;
                __syncthreads();
                if (tid == 0) {
                    for (int k = 1; k < n_warps; ++k) peak = s_top[k] > peak ? s_top[k] : peak;
                    out_pk = (int64_t)peak;
                    out_st = out_pk <= p.M ? 1 : 0;
                }
            }
        }
        if (tid == 0) {
            p.out_peak[b] = out_pk;
            p.out_dur[b] = out_du;
            p.out_status[b] = out_st;
        }
        __syncthreads();    // the state is reused by the next sequence
    }
}

}  // namespace moc

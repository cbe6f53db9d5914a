// Sequence-per-lane path of the evaluator for C <= 2 copies per node and graphs whose state for a
// whole group of sequences fits in shared memory (the paper's experiments: C_v = 2, Section 4.3).
//
// A block works on a group of g = 8, 16 or 32 sequences at a time and keeps ALL of them on chip in
// transposed form: row u of the word array holds the occurrence word of node u for each of the g
// sequences, row t of the delta array the change of usage at step t for each of them.  In stages
// 2-4 a warp's lanes are (sequence j, sub-lane h), j < g, h < S = 32 / g: the g lanes of one
// sub-lane touch g consecutive 32-bit words of one row, so neither the word gathers of stage 2 nor
// the reductions of stage 3 collide on a bank, and everything that depends only on the graph
// (node, successor list, m, w) is the same for all lanes of a sub-lane and is fetched once for g
// sequences.  Stage 1 turns the roles around: a warp takes one row of the batch and its lanes take
// consecutive steps, so that the row is read from global memory in whole 512-byte pieces; rows of
// the word array are g + 1 words apart, which spreads the words of one sequence over all banks.
// The warps of the block share the work of the group: rows in stage 1, nodes in stage 2, chunks
// of steps in the prefix sum, sequences in stage 4.
//
// Representation.  Positions are 1-based and 16 bits wide; a node's word holds its two positions in
// any order, a node computed once the same position twice, an absent node 0.
//
// Stages for the sequences of one group (paper: Section 2, Eqs. 1-8):
//   1. occurrence words   step t exchanges (t+1, t+1) into its node's word; a non-zero return is
//                         the other copy and goes into the high half.  Ids outside [0, n) land in
//                         a spare row.  Well-formed (Eq. 7 and C_v) iff every node's word is
//                         non-zero and the number of words with two positions is T - n.
//   2. free steps         for node u with copies a <= b, over the words r of its successors, two
//                         packed 16-bit reductions (both halves of r take part in both):
//                           Ga = max (r - a) mod 2^16   no successor copy before a (Eq. 5) iff the
//                                                       result is below 2^15; then a + Ga is the
//                                                       latest successor copy: b is kept until there;
//                           Gb = max (r - b) mod 2^16   ranks the copies below b above all others:
//                                                       the latest successor copy inside (a, b),
//                                                       until which the first copy is kept
//                                                       (Eqs. 2, 3, 5).  Seeded with a - b, so that
//                                                       with no such copy the result is a itself.
//                         A sink's only successor is a made-up word that holds T.
//   3. memory profile     delta[p] += m_u, delta[free + 1] -= m_u per copy, then a prefix sum over
//                         the steps, one chunk of steps per sub-lane (Eq. 4).
//   4. reductions         peak (Section 2); duration = sum of all w + w of the second copies (Eq. 1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "moc_pair_kernel.cuh"

namespace moc {

struct LaneParams {
    int32_t n;
    int32_t max_T;             // C * n
    int32_t B;
    int32_t n_bundles;         // ceil(n / S): nodes in order of falling out-degree, S per bundle
    int64_t M;
    int64_t base_dur;          // sum of all w
    const uint4* rec;          // S * n_bundles node records of 32 bytes (below)
    const uint32_t* succ;      // successor rows: byte offsets into the word array
    const int32_t* seqs;
    const int32_t* lens;
    const int64_t* offs;       // row offsets, or nullptr: rows are packed back to back
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_status;
    // shared-memory layout, bytes (multiples of 16)
    uint32_t rec_bytes, succ_bytes;
    uint32_t word_bytes;       // two special rows (T, the constant (1, 1)), then n + 1 rows of g + 1 words
    uint32_t delta_bytes;      // (max_T + 3) rows of g sums: steps -1 .. max_T + 1
};

// Word array: rows of g + 1 words.  The n node rows and one spare row (ids out of range) start at
// a 16-byte boundary; kLaneSpecial(g) bytes in front of them lie the row that holds T (the made-up
// successor of sinks) and, after it, a row of constant words (1, 1) read by empty node slots.
__host__ __device__ constexpr uint32_t lane_word_row(int g) { return 4u * ((uint32_t)g + 1u); }
__host__ __device__ constexpr uint32_t lane_special(int g) { return (2u * lane_word_row(g) + 15u) & ~15u; }

// Node record, 32 bytes: word 0 = byte offset of the node's row from the first node row, word 1 =
// byte offset of its first successor entry | rows of its bundle << 24, words 2-3 = m (int32: word 2
// = m, word 3 = -m), words 4-5 = w | 1 << 40 | (C_v == 1) << 52, words 6-7 = -m (int64 only).  Entry (k, h) of a bundle sits S * k + h
// entries after the bundle's first entry and is itself the byte offset of a row; lists shorter than the
// bundle's rows are padded with the node's own row, which is neutral for both reductions.
constexpr uint64_t kLaneDurMask = (uint64_t(1) << 40) - 1;   // bits 0..39: sum of w over second copies
constexpr int kLaneCntShift = 40;                             // bits 40..51: number of nodes with two copies
constexpr int kLaneCapShift = 52;                             // bits 52..63: of those, nodes with C_v = 1

// if (x != y): red.shared.add [a0], v0; red.shared.add [a1], v1; acc += inc
__device__ __forceinline__ void lane_second_copy(uint32_t x, uint32_t y, uint32_t a0, int32_t v0, uint32_t a1, int32_t v1,
                                                 uint32_t& acc_lo, uint32_t& acc_hi, uint32_t inc_lo, uint32_t inc_hi) {
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, %3;\n\t@q red.shared.add.s32 [%4], %5;\n\t@q red.shared.add.s32 [%6], %7;\n\t"
                 "@q add.cc.u32 %0, %0, %8;\n\t@q addc.u32 %1, %1, %9;\n\t}"
                 : "+r"(acc_lo), "+r"(acc_hi) : "r"(x), "r"(y), "r"(a0), "r"(v0), "r"(a1), "r"(v1), "r"(inc_lo), "r"(inc_hi) : "memory");
}
__device__ __forceinline__ void lane_second_copy(uint32_t x, uint32_t y, uint32_t a0, int64_t v0, uint32_t a1, int64_t v1,
                                                 uint32_t& acc_lo, uint32_t& acc_hi, uint32_t inc_lo, uint32_t inc_hi) {
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, %3;\n\t@q red.shared.add.u64 [%4], %5;\n\t@q red.shared.add.u64 [%6], %7;\n\t"
                 "@q add.cc.u32 %0, %0, %8;\n\t@q addc.u32 %1, %1, %9;\n\t}"
                 : "+r"(acc_lo), "+r"(acc_hi) : "r"(x), "r"(y), "r"(a0), "l"(v0), "r"(a1), "l"(v1), "r"(inc_lo), "r"(inc_hi) : "memory");
}

// Vector k of a row covers the steps 4k - a .. 4k - a + 3 (a = ints between the 16-byte boundary
// below the row and the row).  Steps outside [0, T) come back as -1, which stage 1 sends to the spare row.
__device__ __forceinline__ int4 lane_load_vec(const int32_t* row, int k, int a, int T) {
    const int t0 = 4 * k - a;
    if (t0 >= 0 && t0 + 4 <= T) return __ldg(reinterpret_cast<const int4*>(row + t0));
    int4 v;
    v.x = (t0 >= 0 && t0 < T) ? __ldg(row + t0) : -1;
    v.y = (t0 + 1 >= 0 && t0 + 1 < T) ? __ldg(row + t0 + 1) : -1;
    v.z = (t0 + 2 >= 0 && t0 + 2 < T) ? __ldg(row + t0 + 2) : -1;
    v.w = (t0 + 3 >= 0 && t0 + 3 < T) ? __ldg(row + t0 + 3) : -1;
    return v;
}

// LG: log2 of the sequences per group.  KP: pieces of a row (32 vectors of 4 steps) per warp that are
// fetched into registers one group ahead; further pieces are loaded in place.
template <typename MemT, int LG, int KP>
__global__ void __launch_bounds__(1024, 1) eval_lane_kernel(const LaneParams p) {
    constexpr int g = 1 << LG, S = 32 >> LG;
    constexpr uint32_t kWordRow = lane_word_row(g), kSpecial = lane_special(g);
    constexpr uint32_t kMemRow = (uint32_t)sizeof(MemT) * g, kPartRow = (uint32_t)sizeof(MemT) * (g + 1);
    extern __shared__ __align__(16) char smem[];
    __shared__ int64_t s_red[32];
    __shared__ int64_t s_off[2][g];
    __shared__ int32_t s_T[2][g];
    __shared__ uint32_t s_vmin[g], s_dep[g];
    __shared__ unsigned long long s_acc[g];

    const int lane = threadIdx.x & 31, j = lane & (g - 1), h = lane >> LG;
    int W = blockDim.x >> 5;
    MOC_KEEP(W);
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const int Q = W * S, q = warp * S + h;
    const int QS = min(Q, 32);                 // chunks of the prefix sum (one warp puts them together)
    int n = p.n, n_bundles = p.n_bundles;
    MOC_KEEP(n);
    MOC_KEEP(n_bundles);

    // ---- shared-memory map: graph | chunk sums | chunk maxima | special rows, words | deltas
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t a_rec = sbase;
    uint32_t a_succ = a_rec + p.rec_bytes;
    const uint32_t part_bytes = (32u * kPartRow + 15u) & ~15u;
    const uint32_t a_run = a_succ + p.succ_bytes, a_top = a_run + part_bytes;
    uint32_t a_word = a_top + part_bytes + kSpecial;                          // first node row
    const uint32_t a_delta = a_word - kSpecial + p.word_bytes;
    uint32_t wlane = a_word + 4u * j;                                         // word of sequence j in the first node row
    uint32_t dlane = a_delta + kMemRow + (uint32_t)sizeof(MemT) * j;          // delta of sequence j at step 0
    uint32_t dlane1 = dlane - kMemRow;                                        // ... at step -1
    MOC_KEEP(a_succ);
    MOC_KEEP(a_word);
    MOC_KEEP(wlane);
    MOC_KEEP(dlane);
    MOC_KEEP(dlane1);

    // ---- this block's groups: [grp, grp_end) of ceil(B / g); sum of the lengths in front of them
    const int n_groups = (p.B + g - 1) >> LG;
    int grp = (int)((int64_t)blockIdx.x * n_groups / gridDim.x);
    const int grp_end = (int)(((int64_t)blockIdx.x + 1) * n_groups / gridDim.x);
    const bool self = p.offs == nullptr;
    int64_t base = 0;     // self mode, kept by the last warp: offset of the next group's first row
    if (self) {
        const int c0 = grp << LG;
        int64_t sum = 0;
        if ((reinterpret_cast<uintptr_t>(p.lens) & 15) == 0) {
            const int4* l4 = reinterpret_cast<const int4*>(p.lens);
            const int n4 = c0 >> 2, st = blockDim.x;
            int i = threadIdx.x;
            for (; i + 3 * st < n4; i += 4 * st) {      // four loads in flight per thread
                const int4 v0 = __ldg(l4 + i), v1 = __ldg(l4 + i + st), v2 = __ldg(l4 + i + 2 * st), v3 = __ldg(l4 + i + 3 * st);
                sum += (int64_t)max(v0.x, 0) + max(v0.y, 0) + max(v0.z, 0) + max(v0.w, 0);
                sum += (int64_t)max(v1.x, 0) + max(v1.y, 0) + max(v1.z, 0) + max(v1.w, 0);
                sum += (int64_t)max(v2.x, 0) + max(v2.y, 0) + max(v2.z, 0) + max(v2.w, 0);
                sum += (int64_t)max(v3.x, 0) + max(v3.y, 0) + max(v3.z, 0) + max(v3.w, 0);
            }
            for (; i < n4; i += st) {
                const int4 v = __ldg(l4 + i);
                sum += (int64_t)max(v.x, 0) + max(v.y, 0) + max(v.z, 0) + max(v.w, 0);
            }
            for (int k = (c0 & ~3) + threadIdx.x; k < c0; k += blockDim.x) sum += max(__ldg(p.lens + k), 0);
        } else {
            for (int k = threadIdx.x; k < c0; k += blockDim.x) sum += max(__ldg(p.lens + k), 0);
        }
        sum = warp_sum64(sum);
        if (lane == 0) s_red[warp] = sum;
    }
    // ---- graph -> shared memory; zero words and deltas; constant row
    {
        const uint32_t n_rec16 = p.rec_bytes >> 4, graph16 = (p.rec_bytes + p.succ_bytes) >> 4;
        int4* s4 = reinterpret_cast<int4*>(smem);
        for (uint32_t i = threadIdx.x; i < graph16; i += blockDim.x)
            s4[i] = i < n_rec16 ? __ldg(reinterpret_cast<const int4*>(p.rec) + i)
                                : __ldg(reinterpret_cast<const int4*>(p.succ) + (i - n_rec16));
        const uint32_t z0 = (a_run - sbase) >> 4, z1 = (a_delta + p.delta_bytes - sbase) >> 4;
        const int4 z = make_int4(0, 0, 0, 0);
        for (uint32_t i = z0 + threadIdx.x; i < z1; i += blockDim.x) s4[i] = z;
        if (threadIdx.x < g) {
            s_vmin[threadIdx.x] = 0xFFFFFFFFu;
            s_dep[threadIdx.x] = 0;
            s_acc[threadIdx.x] = 0;
        }
    }
    __syncthreads();
    if (threadIdx.x < g) sts_u32(a_word - kSpecial + kWordRow + 4u * threadIdx.x, 0x00010001u);   // read by empty node slots
    if (self)
        for (int k = 0; k < W; ++k) base += s_red[k];

    // Place and length of the rows of group `gi`, written to buffer gi & 1 by one warp.  A row is
    // usable iff it exists and n <= T <= C n; the others are recorded with T = 0.
    auto publish_group = [&](int gi) {
        const int b = (gi << LG) + j;
        const int32_t len = (gi < grp_end && b < p.B) ? __ldg(p.lens + b) : 0;
        int64_t off;
        if (self) {
            const int64_t pos = (h == 0 && len > 0) ? len : 0;
            const int64_t incl = warp_inclusive_sum(pos, lane);     // lanes of sub-lane 0 come first
            off = base + incl - pos;
            base += __shfl_sync(0xFFFFFFFFu, incl, 31);
        } else {
            off = (gi < grp_end && b < p.B) ? __ldg(p.offs + b) : 0;
        }
        if (h == 0) {
            s_off[gi & 1][j] = off;
            s_T[gi & 1][j] = (len >= n && len <= p.max_T) ? len : 0;
        }
    };
    // Stage 1 works in pieces of 32 vectors (128 steps).  The block has a whole number of warps per
    // row: this warp takes row rj and of its pieces number pk0, pk0 + pstep, ...; lane l takes vector l
    // of a piece.  The warp's first KP pieces are requested one group ahead so that they arrive behind
    // other work.
    const int rj = warp & (g - 1), pk0 = warp >> LG, pstep = W >> LG;
    int4 pre[KP];
    auto prefetch_group = [&](int gi) {
        const int32_t Tj = s_T[gi & 1][rj];
        const int32_t* row = p.seqs + s_off[gi & 1][rj];
        const int a = (int)((reinterpret_cast<uintptr_t>(row) >> 2) & 3);
        const int nvec = Tj ? (Tj + a + 3) >> 2 : 0;
#pragma unroll
        for (int i = 0; i < KP; ++i) {
            const int k = ((pk0 + i * pstep) << 5) + lane;
            if (k < nvec) pre[i] = lane_load_vec(row, k, a, Tj);
        }
    };
    if (grp < grp_end) {
        if (warp == W - 1) publish_group(grp);
        __syncthreads();
        if (warp == 0 && h == 0) sts_u32(wlane - kSpecial, (uint32_t)s_T[grp & 1][j] * 0x10001u);
        prefetch_group(grp);
    }

    for (; grp < grp_end; ++grp) {
        const int buf = grp & 1;
        const int32_t T = s_T[buf][j];      // 0: nothing to evaluate in this lane
        // ---- stage 1: occurrence words
        {
            const int32_t Tj = s_T[buf][rj];
            const int32_t* row = p.seqs + s_off[buf][rj];
            const int a = (int)((reinterpret_cast<uintptr_t>(row) >> 2) & 3);
            const int nvec = Tj ? (Tj + a + 3) >> 2 : 0;
            const uint32_t wj = a_word + 4u * (uint32_t)rj;
            auto put4 = [&](const int4 v, const int k) {
                uint32_t val = (uint32_t)(4 * k - a + 1) * 0x10001u;
                const int32_t id[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t addr = wj + min((uint32_t)id[e], (uint32_t)n) * kWordRow;
                    const uint32_t old = exch_shared(addr, val);
                    sts_u16_if_nonzero(old, addr + 2, old);
                    val += 0x10001u;
                }
            };
#pragma unroll
            for (int i = 0; i < KP; ++i) {
                const int k = ((pk0 + i * pstep) << 5) + lane;
                if (k < nvec) put4(pre[i], k);
            }
            for (int k = ((pk0 + KP * pstep) << 5) + lane; k < nvec; k += pstep << 5) put4(lane_load_vec(row, k, a, Tj), k);
        }
        __syncthreads();

        // ---- stage 2 and the scatter of stage 3: one node per sub-lane and round
        if (warp == W - 1) publish_group(grp + 1);
        {
            uint32_t vmin = 0xFFFFFFFFu, depw = 0, acc_lo = 0, acc_hi = 0;
            uint32_t prec = a_rec + 32u * (uint32_t)q;
            uint32_t rec_step = 32u * (uint32_t)Q, rec_end = a_rec + 32u * (uint32_t)(n_bundles * S);
            MOC_KEEP(rec_step);
            MOC_KEEP(rec_end);
            for (; prec < rec_end; prec += rec_step) {
                const uint4 rec = lds_v4(prec);
                const uint4 rec2 = lds_v4(prec + 16);      // w and flags; -m of 64 bits
                const uint32_t own = lds_u32(wlane + rec.x);
                const uint32_t sw = swap_halves(own);
                const uint32_t mn = min_u16x2(own, sw), mx = max_u16x2(own, sw);   // (a, a), (b, b)
                const uint32_t naa = 0x00010000u - mn, nbb = 0x00010000u - mx;     // (-a, -a), (-b, -b) mod 2^16
                uint32_t Ga = mx - mn;                                             // (b - a, b - a)
                uint32_t Gb = 0x00010000u - Ga;                                    // (a - b, a - b) mod 2^16 when a < b
                int rows = (int)(rec.y >> 24);
                if (S > 1) rows = __shfl_sync(0xFFFFFFFFu, rows, 0);
                uint32_t pe = a_succ + (rec.y & 0xFFFFFFu);
#pragma unroll 2
                for (int k = 0; k < rows; ++k) {
                    const uint32_t r = lds_u32(wlane + lds_u32_nv(pe));
                    pe += 4u * S;
                    Ga = __viaddmax_u16x2(r, naa, Ga);
                    Gb = __viaddmax_u16x2(r, nbb, Gb);
                }
                depw |= Ga;                                                        // bit 15 or 31: a successor copy before a
                const uint32_t gg = max_u16x2(__byte_perm(Ga, Gb, 0x5410), __byte_perm(Ga, Gb, 0x7632));  // (best Ga, best Gb)
                const uint32_t ab = __byte_perm(mn, mx, 0x7610);                   // (a, b)
                const uint32_t v = gg + ab;                                        // (end of b, end of a) mod 2^16
                MemT m, neg_m;
                if constexpr (sizeof(MemT) == 4) {
                    m = (MemT)rec.z;
                    neg_m = (MemT)rec.w;
                } else {
                    m = (MemT)((uint64_t)rec.z | ((uint64_t)rec.w << 32));
                    neg_m = (MemT)((uint64_t)rec2.z | ((uint64_t)rec2.w << 32));
                }
                red_add_shared(dlane1 + (ab >> 16) * kMemRow, m);
                red_add_shared(dlane + (v & 0xFFFFu) * kMemRow, neg_m);
                lane_second_copy(mn, mx, dlane1 + (ab & 0xFFFFu) * kMemRow, m, dlane + (v >> 16) * kMemRow, neg_m,
                                 acc_lo, acc_hi, rec2.x, rec2.y);
                vmin = min(vmin, own);
            }
            atomicMin(&s_vmin[j], vmin);
            if (depw & 0x80008000u) atomicOr(&s_dep[j], 1u);
            atomicAdd(&s_acc[j], (unsigned long long)acc_lo | ((unsigned long long)acc_hi << 32));
        }
        __syncthreads();

        // ---- next group's rows on their way; prefix sum of this group's deltas, chunk per sub-lane;
        // words and deltas back to zero
        const bool more = grp + 1 < grp_end;
        if (more) prefetch_group(grp + 1);
        {
            const int E = __reduce_max_sync(0xFFFFFFFFu, T) + 2;      // steps 0 .. Tmax + 1 can hold something
            const int L = (E + QS - 1) / QS;
            if (q < QS) {
                const int t0 = q * L, t1 = min(t0 + L, E);
                MemT run = 0, top = 0;
                uint32_t ad = dlane + (uint32_t)t0 * kMemRow;
                if (t0 < t1) {
                    run = lds_mem(ad, MemT());
                    sts_mem(ad, MemT(0));
                    top = run;
                    ad += kMemRow;
                }
#pragma unroll 4
                for (int t = t0 + 1; t < t1; ++t) {
                    const MemT d = lds_mem(ad, MemT());
                    sts_mem(ad, MemT(0));
                    run += d;
                    top = run > top ? run : top;
                    ad += kMemRow;
                }
                sts_mem(a_run + (uint32_t)q * kPartRow + (uint32_t)sizeof(MemT) * j, run);
                sts_mem(a_top + (uint32_t)q * kPartRow + (uint32_t)sizeof(MemT) * j, top);
            }
            // words of the n nodes and the spare row (whole 16-byte vectors: up to 12 bytes of the
            // deltas' step -1, which only collects the additions of absent nodes, go with them)
            const int4 z = make_int4(0, 0, 0, 0);
            int4* w4 = reinterpret_cast<int4*>(smem + (a_word - sbase));
            const int nw4 = (int)(((uint32_t)(n + 1) * kWordRow + 15u) >> 4);
            for (int i = threadIdx.x; i < nw4; i += blockDim.x) w4[i] = z;
            if (warp == 0 && h == 0) {
                if (more) sts_u32(wlane - kSpecial, (uint32_t)s_T[buf ^ 1][j] * 0x10001u);
                sts_mem(dlane1, MemT(0));
            }
        }
        __syncthreads();

        // ---- stage 4: a warp per sequence puts the chunks together (lane = chunk) and writes the results
        for (int jj = warp; jj < g; jj += W) {
            const int b = (grp << LG) + jj;
            if (b >= p.B) break;
            MemT r = 0, tp = 0;
            if (lane < QS) {
                r = lds_mem(a_run + (uint32_t)lane * kPartRow + (uint32_t)sizeof(MemT) * jj, MemT());
                tp = lds_mem(a_top + (uint32_t)lane * kPartRow + (uint32_t)sizeof(MemT) * jj, MemT());
            }
            // an empty chunk has r = tp = 0: its candidate is the usage in front of it, never above the peak
            const MemT cand = warp_inclusive_sum(r, lane) - r + tp;
            const int64_t peak = (int64_t)warp_max_t(cand);
            if (lane == 0) {
                const int32_t Tj = s_T[buf][jj];
                const uint32_t vmin = s_vmin[jj], dep = s_dep[jj];
                const unsigned long long acc = s_acc[jj];
                s_vmin[jj] = 0xFFFFFFFFu;
                s_dep[jj] = 0;
                s_acc[jj] = 0;
                int64_t out_pk = -1, out_du = -1;
                int32_t out_st = -2;
                const bool well_formed = Tj != 0 && vmin != 0 && (int)((acc >> kLaneCntShift) & 0xFFFu) == Tj - n &&
                                         (acc >> kLaneCapShift) == 0;
                if (well_formed) {
                    out_du = p.base_dur + (int64_t)(acc & kLaneDurMask);
                    out_st = -1;
                    if (!dep) {
                        out_pk = peak;
                        out_st = peak <= p.M ? 1 : 0;
                    }
                }
                p.out_peak[b] = out_pk;
                p.out_dur[b] = out_du;
                p.out_status[b] = out_st;
            }
        }
    }
}

}  // namespace moc

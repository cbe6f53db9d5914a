// Fast path of the sequence evaluator for C <= 2 copies per node (the paper's experiments all use
// C_v = 2, Section 4.3): one warp evaluates one sequence, warp-synchronously, with the graph staged
// once per block in shared memory.
//
// Representation.  Positions are 1-based and 16 bits wide.  Each node owns one 32-bit word with
// its two positions; a node computed once holds the same position in both halves, an absent node
// holds 0.  A consumer reads both copies of a successor with one load.  Lane l of a warp works on
// the nodes with id = l (mod 32): a node's word then sits in bank l, so the lanes' reads of their
// own words never collide.  The nodes of each residue class are sorted by out-degree
// (descending); "half" j holds the j-th node of every class and a tile is two consecutive halves,
// so a lane treats two nodes per tile.  The successor lists are stored per tile as a dense
// [rows][32] matrix of 32-bit entries: entry (k, l) packs the word offsets of the k-th successor
// of lane l's two nodes, 16 bits each; rows = largest out-degree in the tile; missing successors
// point at a dummy word that stays zero, which is neutral for every reduction below.  A sink has
// one made-up successor: a word that holds the sequence length T, which keeps its last copy to
// the end.  Every lane of a warp runs the same trip count.  Node slots beyond the last node of a
// class read a constant word and carry m = w = 0, so they need no special case.
//
// Stages for one sequence seq[0..T) (paper: Section 2, Eqs. 1-8):
//   1. occurrence words   step t exchanges (t+1, t+1) into its node's word; if the word was taken,
//                         the previous low half is stored into the high half.  An id outside
//                         [0, n) lands in the dummy word.  A third copy, or an id out of range,
//                         loses a position, which the check "sum of stored positions = T(T+1)/2"
//                         detects; an absent node (Eq. 7) shows as a zero word.
//   2. free steps         one lane per node u with copies a <= b (a = b if computed once), one pass
//                         over its successors' words r with three packed 16-bit reductions:
//                           F = max(b, r)        latest successor copy: b is kept until F;
//                           D = min(a-1, r-1)    below a-1 iff a successor copy precedes a: Eq. 5
//                                                violated;
//                           G = max (r - b)      mod 2^16 this ranks the copies below b above all
//                                                others, in order: the latest successor copy inside
//                                                (a, b), until which the first copy a is kept
//                                                (Eqs. 2, 3, 5).
//   3. memory profile     delta[p] += m_u, delta[free+1] -= m_u, prefix sum (Eq. 4).
//   4. reductions         peak (Section 2), duration = sum_v w_v + sum over second copies (Eq. 1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "moc_kernels.cuh"

namespace moc {

struct PairParams {
    int32_t n;
    int32_t n_tiles;           // tiles of 64 node slots (two halves of 32)
    int32_t sell_len;          // 32-bit entries of the successor tiles
    int32_t max_T;             // C * n
    uint32_t sum_bias;         // number of empty node slots (each reads a word holding (1, 1))
    const void* rec;           // 64 * n_tiles node records (NodeRec<MemT>), slot = half * 32 + lane
    const int64_t* wslot;      // 64 * n_tiles durations, same slots; bit 63 set: the node's cap C_v is 1
    const uint32_t* sell;      // sell_len entries: successor word offsets of the two halves, 16 bits each
    const uint32_t* tile;      // n_tiles: first entry of the tile | rows of the tile << 20
    int64_t base_dur;          // sum of all w
    const int32_t* seqs;
    const int32_t* lens;
    const int64_t* offs;       // exclusive prefix sum of the lengths, or nullptr: the kernel finds the rows itself
    int32_t B;
    int64_t M;
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_status;
    // shared-memory layout, bytes (multiples of 16)
    uint32_t rec_bytes, w_bytes, tile_bytes, sell_bytes;  // graph, once per block
    uint32_t word_bytes, delta_bytes;            // per warp; 16 bytes after the words hold the constant 1
};

constexpr int kPairDeltaFront = 16;  // bytes in front of delta[0]: lands writes of absent nodes
constexpr int kPairWordTail = 16;    // bytes after the words: the word read by empty node slots

__device__ __forceinline__ int64_t warp_sum64(int64_t v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}
__device__ __forceinline__ int32_t warp_max_t(int32_t v) { return __reduce_max_sync(0xFFFFFFFFu, v); }
__device__ __forceinline__ int64_t warp_max_t(int64_t v) { return warp_max(v); }

// per-halfword unsigned max of two packed 16-bit pairs (one instruction on sm_90 and later)
__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t min_u16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("min.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t swap_halves(uint32_t a) { return __byte_perm(a, 0, 0x1032); }

// ---- shared-memory accesses by 32-bit shared address
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_u16(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"((uint16_t)v) : "memory");
}
__device__ __forceinline__ uint32_t exch_shared(uint32_t addr, uint32_t v) {
    uint32_t old;
    asm volatile("atom.shared.exch.b32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void red_add_shared(uint32_t addr, int32_t v) {
    asm volatile("red.shared.add.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void red_add_shared(uint32_t addr, int64_t v) {
    asm volatile("red.shared.add.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}

// Node record: byte offset of the node's word, and the output size.
template <typename MemT> struct NodeRec;
template <> struct __align__(8) NodeRec<int32_t> { uint32_t nd; int32_t m; };
template <> struct __align__(16) NodeRec<int64_t> { uint32_t nd; uint32_t pad; int64_t m; };

// kPre: how many 16-byte vectors of the next row each lane fetches ahead (rows of about 128*kPre
// steps; 0 for short rows, where the extra registers cost more than the wait).  Blocks have up to 16
// warps and two of them share an SM (62 registers per thread, no spills).
template <typename MemT, int kPre>
__global__ void __launch_bounds__(512, 2) eval_pair_kernel(const PairParams p) {
    extern __shared__ __align__(16) char smem[];
    __shared__ int64_t s_part[16];
    using Rec = NodeRec<MemT>;
    // ---- graph -> shared memory, once per block
    Rec* s_rec = reinterpret_cast<Rec*>(smem);
    int64_t* s_w = reinterpret_cast<int64_t*>(smem + p.rec_bytes);
    uint32_t* s_tile = reinterpret_cast<uint32_t*>(smem + p.rec_bytes + p.w_bytes);
    uint32_t* s_sell = reinterpret_cast<uint32_t*>(smem + p.rec_bytes + p.w_bytes + p.tile_bytes);
    const uint32_t graph_bytes = p.rec_bytes + p.w_bytes + p.tile_bytes + p.sell_bytes;
    {
        const int4* g4 = reinterpret_cast<const int4*>(p.rec);
        int4* s4 = reinterpret_cast<int4*>(s_rec);
        const int n4 = (int)sizeof(Rec) * 64 * p.n_tiles / 16;
        for (int i = threadIdx.x; i < n4; i += blockDim.x) s4[i] = __ldg(&g4[i]);
        for (int i = threadIdx.x; i < 64 * p.n_tiles; i += blockDim.x) s_w[i] = __ldg(&p.wslot[i]);
        for (int i = threadIdx.x; i < p.n_tiles; i += blockDim.x) s_tile[i] = __ldg(&p.tile[i]);
        for (int i = threadIdx.x; i < p.sell_len; i += blockDim.x) s_sell[i] = __ldg(&p.sell[i]);
    }
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    // broadcast from lane 0 so that the compiler knows the warp index is uniform across the warp
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    char* ws = smem + graph_bytes + (size_t)warp * (p.word_bytes + kPairWordTail + p.delta_bytes);
    uint32_t* word = reinterpret_cast<uint32_t*>(ws);
    char* delta_base = ws + p.word_bytes + kPairWordTail;          // includes the front pad
    const uint32_t wa = (uint32_t)__cvta_generic_to_shared(word);
    const uint32_t da = (uint32_t)__cvta_generic_to_shared(delta_base) + kPairDeltaFront;  // &delta[0]
    const uint32_t da1 = da - (uint32_t)sizeof(MemT);                                     // &delta[-1]
    if (lane == 0) *reinterpret_cast<uint32_t*>(ws + p.word_bytes) = 0x00010001u;   // read by empty node slots
    __syncthreads();

    const int n = p.n;
    const int n_warps = gridDim.x * wpb;
    constexpr int kPerVec = 16 / (int)sizeof(MemT);  // delta entries per 16-byte vector
    constexpr int kShift = sizeof(MemT) == 4 ? 2 : 3;

    // Two ways to find the rows.  With p.offs (written by the offsets kernel) warps stride over the
    // whole batch.  Without it (p.offs == nullptr) block c takes the contiguous range
    // [c*B/grid, (c+1)*B/grid): it adds up the lengths in front of its range once, and every warp then
    // walks the range with the lengths themselves -- no scratch, no second kernel.
    const bool self = p.offs == nullptr;
    int b, b_end, b_step;
    int64_t off = 0;
    int32_t T = 0;
    // self mode: lanes 0..wpb-1 hold the lengths of sequences b .. b+wpb-1 (next: of the following wpb)
    int32_t len_raw = 0;
    auto group_sum = [&](int32_t raw, int lanes) -> int64_t {   // sum of max(raw, 0) over lanes < `lanes`
        const uint32_t v = (lane < lanes && raw > 0) ? (uint32_t)raw : 0u;
        const uint32_t lo = __reduce_add_sync(0xFFFFFFFFu, v & 0xFFFFu), hi = __reduce_add_sync(0xFFFFFFFFu, v >> 16);
        return (int64_t)lo + ((int64_t)hi << 16);
    };
    if (!self) {
        b = blockIdx.x * wpb + warp;
        b_end = p.B;
        b_step = n_warps;
        if (b < b_end) { off = __ldg(&p.offs[b]); T = __ldg(&p.lens[b]); }
    } else {
        const int c0 = (int)((int64_t)blockIdx.x * p.B / gridDim.x);
        b_end = (int)(((int64_t)blockIdx.x + 1) * p.B / gridDim.x);
        b_step = wpb;
        int64_t sum = 0;
        if ((reinterpret_cast<uintptr_t>(p.lens) & 15) == 0) {
            const int4* l4 = reinterpret_cast<const int4*>(p.lens);
            for (int i = threadIdx.x; i < (c0 >> 2); i += blockDim.x) {
                const int4 q = __ldg(l4 + i);
                sum += (int64_t)max(q.x, 0) + max(q.y, 0) + max(q.z, 0) + max(q.w, 0);
            }
            for (int i = (c0 & ~3) + threadIdx.x; i < c0; i += blockDim.x) sum += max(__ldg(p.lens + i), 0);
        } else {
            for (int i = threadIdx.x; i < c0; i += blockDim.x) sum += max(__ldg(p.lens + i), 0);
        }
        sum = warp_sum64(sum);
        if (lane == 0) s_part[warp] = sum;
        __syncthreads();
        for (int k = 0; k < wpb; ++k) off += s_part[k];
        // lengths of the first wpb sequences of the range; this warp starts at the warp-th of them
        len_raw = (c0 + lane < p.B) ? __ldg(p.lens + c0 + lane) : 0;
        off += group_sum(len_raw, warp);
        b = c0 + warp;
        // shift so that lane k holds the length of sequence b + k
        len_raw = (b + lane < p.B) ? __ldg(p.lens + b + lane) : 0;
        T = __shfl_sync(0xFFFFFFFFu, len_raw, 0);
    }
    // The first kPre 16-byte vectors per lane of the NEXT row are loaded into registers while the
    // current sequence is still being worked on, so that stage 1 does not wait for HBM.
    int4 pre[kPre > 0 ? kPre : 1];
    bool have_pre = false;
    while (b < b_end) {
        // fetch the next sequence's place early: its latency hides behind this sequence's work
        const int b_next = b + b_step;
        int64_t off_next = 0;
        int32_t T_next = 0, len_next = 0;
        if (!self) {
            if (b_next < b_end) { off_next = __ldg(&p.offs[b_next]); T_next = __ldg(&p.lens[b_next]); }
        } else {
            if (b_next < b_end) len_next = (b_next + lane < p.B) ? __ldg(p.lens + b_next + lane) : 0;
        }

        const bool use_pre = have_pre;   // pre[] holds this row only if the previous iteration fetched it
        have_pre = false;
        int64_t out_pk = -1, out_du = -1;
        int32_t out_st = -2;
        if (T >= n && T <= p.max_T) {
            // ---- clear: words, and the deltas the scan will read (whole vectors per lane)
            const int nvec_d = (T + 1 + kPerVec - 1) / kPerVec;        // vectors covering delta[0..T]
            const int V = ((nvec_d + 31) >> 5) | 1;                      // vectors per lane, odd
            {
                const int4 z = make_int4(0, 0, 0, 0);
                int4* w4 = reinterpret_cast<int4*>(word);
                for (int i = lane; i < (int)(p.word_bytes >> 4); i += 32) w4[i] = z;
                int4* d4 = reinterpret_cast<int4*>(delta_base);
                const int nd4 = 32 * V + 1;                              // front pad + 32*V vectors
                for (int i = lane; i < nd4; i += 32) d4[i] = z;
            }
            __syncwarp();
            if (lane == 0) word[n + 1] = (uint32_t)T * 0x10001u;   // the made-up successor of sinks

            // ---- stage 1: occurrence words
            {
                const int32_t* row = p.seqs + off;
                const int a = (int)((reinterpret_cast<uintptr_t>(row) & 15) >> 2);
                const int nvec = (T + a + 3) >> 2;
                auto put = [&](int node, uint32_t t1) {
                    // ids outside [0, n) go to the dummy word n; the position sum exposes them
                    const uint32_t addr = wa + 4u * min((uint32_t)node, (uint32_t)n);
                    const uint32_t old = exch_shared(addr, t1 * 0x10001u);
                    if (old) sts_u16(addr + 2, old);
                };
                // vectors that lie completely inside the row (the first kPre per lane may already be here)
#pragma unroll
                for (int j = 0; j < kPre; ++j) {
                    const int i = lane + 32 * j;
                    const int t0 = 4 * i - a;
                    if (i < nvec && t0 >= 0 && t0 + 4 <= T) {
                        int4 v = pre[j];
                        if (!use_pre) v = __ldg(reinterpret_cast<const int4*>(row + t0));
                        put(v.x, (uint32_t)t0 + 1);
                        put(v.y, (uint32_t)t0 + 2);
                        put(v.z, (uint32_t)t0 + 3);
                        put(v.w, (uint32_t)t0 + 4);
                    }
                }
                for (int i = lane + 32 * kPre; i < nvec; i += 32) {
                    const int t0 = 4 * i - a;
                    if (t0 >= 0 && t0 + 4 <= T) {
                        const int4 v = __ldg(reinterpret_cast<const int4*>(row + t0));
                        put(v.x, (uint32_t)t0 + 1);
                        put(v.y, (uint32_t)t0 + 2);
                        put(v.z, (uint32_t)t0 + 3);
                        put(v.w, (uint32_t)t0 + 4);
                    }
                }
                // the ragged first and last vectors, element by element
                if (lane < 2) {
                    const int i = lane == 0 ? 0 : nvec - 1;
                    const int t0 = 4 * i - a;
                    if ((lane == 0 || nvec > 1) && !(t0 >= 0 && t0 + 4 <= T)) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int t = t0 + k;
                            if (t >= 0 && t < T) put(__ldg(row + t), (uint32_t)t + 1);
                        }
                    }
                }
            }
            __syncwarp();

            // request the next row now: the loads complete behind stages 2-4
            if (kPre > 0 && b_next < b_end) {
                const int64_t off_n = self ? off + group_sum(len_raw, wpb) : off_next;
                const int32_t T_n = self ? __shfl_sync(0xFFFFFFFFu, len_next, 0) : T_next;
                if (T_n >= n && T_n <= p.max_T) {
                    const int32_t* nrow = p.seqs + off_n;
                    const int an = (int)((reinterpret_cast<uintptr_t>(nrow) & 15) >> 2);
                    const int nvn = (T_n + an + 3) >> 2;
#pragma unroll
                    for (int j = 0; j < kPre; ++j) {
                        const int i = lane + 32 * j;
                        const int t0 = 4 * i - an;
                        if (i < nvn && t0 >= 0 && t0 + 4 <= T_n) pre[j] = __ldg(reinterpret_cast<const int4*>(nrow + t0));
                    }
                    have_pre = true;
                }
            }

            // ---- stage 2 and the scatter of stage 3: two node slots per lane and tile
            uint32_t vmin = 0xFFFFFFFFu, vsum = 0;
            uint32_t depw = 0, capw = 0;
            int64_t dur_extra = 0;
            for (int d = 0; d < p.n_tiles; ++d) {
                Rec rec[2];
                uint32_t mn[2], mx[2], nbb[2], aa1[2], F[2], D[2], G[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    rec[h] = s_rec[(2 * d + h) * 32 + lane];
                    const uint32_t own = lds_u32(wa + rec[h].nd);
                    const uint32_t sw = swap_halves(own);
                    mn[h] = min_u16x2(own, sw);        // (a, a)
                    mx[h] = max_u16x2(own, sw);        // (b, b)
                    nbb[h] = 0x00010000u - mx[h];      // (-b, -b) mod 2^16 for b >= 1
                    aa1[h] = mn[h] - 0x00010001u;      // (a-1, a-1) for a >= 1
                    F[h] = mx[h]; D[h] = aa1[h]; G[h] = 0;
                }
                // successors of the tile: uniform trip count, padded entries read the dummy word
                const uint32_t tl = __shfl_sync(0xFFFFFFFFu, s_tile[d], 0);
                const uint32_t* pj = s_sell + (tl & 0xFFFFFu) + lane;
                const int rows = (int)(tl >> 20);
#pragma unroll 2
                for (int k = 0; k < rows; ++k) {
                    const uint32_t e = pj[k * 32];
                    const uint32_t r0 = lds_u32(wa + (e & 0xFFFFu));
                    const uint32_t r1 = lds_u32(wa + (e >> 16));
                    F[0] = max_u16x2(F[0], r0);
                    F[1] = max_u16x2(F[1], r1);
                    D[0] = __viaddmin_u16x2(r0, 0xFFFFFFFFu, D[0]);   // min(r - 1): empty half -> 0xFFFF
                    D[1] = __viaddmin_u16x2(r1, 0xFFFFFFFFu, D[1]);
                    G[0] = __viaddmax_u16x2(r0, nbb[0], G[0]);        // max(r - b)
                    G[1] = __viaddmax_u16x2(r1, nbb[1], G[1]);
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t a = mn[h] & 0xFFFFu, bpos = mx[h] & 0xFFFFu;
                    vmin = min(vmin, a);
                    vsum += bpos;
                    depw |= D[h] ^ aa1[h];     // some successor copy lies before the first copy of u
                    const uint32_t fb = max_u16x2(F[h], swap_halves(F[h])) & 0xFFFFu;
                    red_add_shared(da1 + (bpos << kShift), rec[h].m);
                    red_add_shared(da + (fb << kShift), (MemT)(-rec[h].m));
                    if (a != bpos) {
                        vsum += a;
                        // bit 63 of the duration marks a node that may have one copy only (C_v = 1): the
                        // sequence is then malformed and the sum below is never reported
                        const int64_t wv = s_w[(2 * d + h) * 32 + lane];
                        capw |= (uint32_t)((uint64_t)wv >> 32);
                        dur_extra += wv;
                        // latest successor copy x with a < x < b, if any: (x - b) mod 2^16 is the largest
                        const uint32_t x = (max_u16x2(G[h], swap_halves(G[h])) + bpos) & 0xFFFFu;
                        const uint32_t fa = (x - 1u < bpos - 1u) ? x : a;
                        red_add_shared(da1 + (a << kShift), rec[h].m);
                        red_add_shared(da + (fa << kShift), (MemT)(-rec[h].m));
                    }
                }
            }
            vmin = __reduce_min_sync(0xFFFFFFFFu, vmin);
            vsum = __reduce_add_sync(0xFFFFFFFFu, vsum);
            const bool cap_ok = !__any_sync(0xFFFFFFFFu, (int32_t)capw < 0);
            const bool well_formed = cap_ok && vmin != 0 && vsum == (uint32_t)T * ((uint32_t)T + 1u) / 2u + p.sum_bias;
            const bool dep = __any_sync(0xFFFFFFFFu, depw != 0);
            __syncwarp();

            if (!well_formed) {
                // status -2, sentinels already set
            } else if (dep) {
                out_st = -1;
                out_du = p.base_dur + warp_sum64(dur_extra);
            } else {
                // ---- stage 3 + 4: prefix sum and running maximum; lane owns V consecutive vectors
                // One pass: the lane's running prefix and the largest prefix it sees; the largest
                // usage inside the lane's chunk is then (sum of the chunks before it) + that maximum.
                const int4* d4 = reinterpret_cast<const int4*>(delta_base + kPairDeltaFront) + lane * V;
                MemT run = 0, top;
                {
                    const int4 q = d4[0];
                    if constexpr (sizeof(MemT) == 4) {
                        run = q.x; top = run;
                        run += q.y; top = max(top, run);
                        run += q.z; top = max(top, run);
                        run += q.w; top = max(top, run);
                    } else {
                        const longlong2 l = *reinterpret_cast<const longlong2*>(&q);
                        run = (MemT)l.x; top = run;
                        run += (MemT)l.y; top = run > top ? run : top;
                    }
                }
                for (int j = 1; j < V; ++j) {
                    const int4 q = d4[j];
                    if constexpr (sizeof(MemT) == 4) {
                        run += q.x; top = max(top, run);
                        run += q.y; top = max(top, run);
                        run += q.z; top = max(top, run);
                        run += q.w; top = max(top, run);
                    } else {
                        const longlong2 l = *reinterpret_cast<const longlong2*>(&q);
                        run += (MemT)l.x; top = run > top ? run : top;
                        run += (MemT)l.y; top = run > top ? run : top;
                    }
                }
                const MemT peak = warp_inclusive_sum(run, lane) - run + top;
                out_pk = (int64_t)warp_max_t(peak);
                out_du = p.base_dur + warp_sum64(dur_extra);
                out_st = out_pk <= p.M ? 1 : 0;
            }
            __syncwarp();
        }
        if (lane == 0) {
            p.out_peak[b] = out_pk;
            p.out_dur[b] = out_du;
            p.out_status[b] = out_st;
        }
        if (self) {
            off_next = off + group_sum(len_raw, wpb);   // skip the wpb sequences b .. b+wpb-1
            len_raw = len_next;
            T_next = __shfl_sync(0xFFFFFFFFu, len_next, 0);
        }
        b = b_next;
        off = off_next;
        T = T_next;
    }
}

}  // namespace moc

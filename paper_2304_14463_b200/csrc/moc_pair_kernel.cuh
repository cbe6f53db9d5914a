// Fast path of the sequence evaluator for C <= 2 copies per node (the paper's experiments all use
// C_v = 2, Section 4.3): one warp evaluates one sequence, warp-synchronously, with the graph staged
// once per block in shared memory.
//
// Representation.  Positions are 1-based and 16 bits wide.  Each node owns one 32-bit word with
// its two positions in any order; a node computed once holds the same position in both halves, an
// absent node holds 0.  A consumer reads both copies of a successor with one load.  Lane l of a
// warp works on the nodes with id = l (mod 32): a node's word then sits in bank l, so the lanes'
// reads of their own words never collide.  The nodes of each residue class are sorted by out-degree
// (descending); "half" j holds the j-th node of every class and a tile is two consecutive halves,
// so a lane treats two nodes per tile.  The successor lists are stored per tile as a dense
// [rows][32] matrix of 32-bit entries: entry (k, l) packs the byte offsets of the words of the
// k-th successor of lane l's two nodes, 16 bits each; rows = largest out-degree in the tile; a list that is used
// up continues with the node's own word, which is neutral for both reductions below.  A sink has
// one made-up successor: a word that holds the sequence length T, which keeps its last copy to
// the end.  Every lane of a warp runs the same trip count.  Node slots beyond the last node of a
// class own a constant word (1, 1) and carry m = w = 0, so they need no special case.
//
// Stages for one sequence seq[0..T) (paper: Section 2, Eqs. 1-8):
//   1. occurrence words   step t exchanges (t+1, t+1) into its node's word; if the word was taken,
//                         the previous low half is stored into the high half.  An id outside
//                         [0, n) lands in a spare word.  A third copy, or an id out of range,
//                         loses a position: the sequence is well-formed (Eq. 7, C_v) iff no word
//                         is zero and the number of words with two positions is T - n.
//   2. free steps         one lane per node u with copies a <= b (a = b if computed once), one pass
//                         over its successors' words r with two packed 16-bit reductions (both
//                         halves of r take part in both):
//                           Ga = max (r - a) mod 2^16   a successor copy before a (Eq. 5 violated)
//                                                       makes it 2^15 or more; otherwise a + Ga is
//                                                       the latest successor copy: b is kept until
//                                                       there (seeded with b - a: at least b);
//                           Gb = max (r - b) mod 2^16   ranks the copies below b above all others,
//                                                       in order: the latest successor copy inside
//                                                       (a, b), until which the first copy a is kept
//                                                       (Eqs. 2, 3, 5); seeded with a - b, so that
//                                                       without such a copy the result is a itself.
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
    int32_t max_T;             // C * n
    const void* rec;           // 64 * n_tiles node records (8 bytes for 32-bit sums, 16 for 64-bit), slot = half * 32 + lane
    const uint64_t* wslot;     // 64 * n_tiles, same slots: w | 1 << 48 | (C_v == 1) << 63
    const uint32_t* sell;      // successor tiles: byte offsets of the successor words of a lane's two nodes, 16 bits each
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
    uint32_t rec_bytes, w_bytes, sell_bytes;     // graph, once per block
    uint32_t word_bytes, delta_bytes;            // per warp; 16 bytes after the words hold the constant (1, 1)
};

// Node record: {byte offset of the node's word | rows of the tile << 16, m}; m takes 32 bits, or 64
// bits after a pad word.
constexpr uint64_t kPairDurMask = (uint64_t(1) << 48) - 1;   // bits 0..47 of the summed wslot entries: w of the second copies
constexpr int kPairCntShift = 48;                             // bits 48..62: number of nodes with two copies

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
__device__ __forceinline__ uint32_t lds_u32_nv(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint64_t lds_u64(uint32_t addr) {
    uint64_t v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ int32_t lds_mem(uint32_t addr, int32_t) { return (int32_t)lds_u32(addr); }
__device__ __forceinline__ int64_t lds_mem(uint32_t addr, int64_t) { return (int64_t)lds_u64(addr); }
__device__ __forceinline__ void sts_mem(uint32_t addr, int32_t v) { sts_u32(addr, (uint32_t)v); }
__device__ __forceinline__ void sts_mem(uint32_t addr, int64_t v) {
    asm volatile("st.shared.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}

__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
    return v;
}
// st.shared.u16 [addr], v  if old != 0
__device__ __forceinline__ void sts_u16_if_nonzero(uint32_t old, uint32_t addr, uint32_t v) {
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %0, 0;\n\t@q st.shared.u16 [%1], %2;\n\t}" ::"r"(old), "r"(addr),
                 "h"((uint16_t)v) : "memory");
}
// Makes a value opaque to the compiler at this point: it is then kept in its register instead of
// being recomputed from the kernel parameters wherever it is used (the hot loops are short of
// instruction slots, not of registers).
#define MOC_KEEP(x) asm volatile("" : "+r"(x))


// kPre: how many 16-byte vectors of the next row each lane fetches ahead (rows of about 128*kPre
// steps; 0 for short rows, where the extra registers cost more than the wait).  Blocks have up to 16
// warps and two of them share an SM (62 registers per thread, no spills).
template <typename MemT, int kPre>
__global__ void __launch_bounds__(512, 2) eval_pair_kernel(const PairParams p) {
    extern __shared__ __align__(16) char smem[];
    __shared__ int64_t s_part[16];
    constexpr uint32_t kRecB = sizeof(MemT) == 4 ? 8u : 16u;
    // ---- graph -> shared memory, once per block: records | durations | successor tiles
    const uint32_t graph_bytes = p.rec_bytes + p.w_bytes + p.sell_bytes;
    {
        int4* s4 = reinterpret_cast<int4*>(smem);
        const uint32_t n_rec = p.rec_bytes >> 4, n_w = p.w_bytes >> 4, n_all = (p.rec_bytes + p.w_bytes + p.sell_bytes) >> 4;
        for (uint32_t i = threadIdx.x; i < n_all; i += blockDim.x) {
            int4 v;
            if (i < n_rec) v = __ldg(reinterpret_cast<const int4*>(p.rec) + i);
            else if (i < n_rec + n_w) v = __ldg(reinterpret_cast<const int4*>(p.wslot) + (i - n_rec));
            else v = __ldg(reinterpret_cast<const int4*>(p.sell) + (i - n_rec - n_w));
            s4[i] = v;
        }
    }
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    // broadcast from lane 0 so that the compiler knows the warp index is uniform across the warp
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    char* ws = smem + graph_bytes + (size_t)warp * (p.word_bytes + kPairWordTail + p.delta_bytes);
    uint32_t* word = reinterpret_cast<uint32_t*>(ws);
    char* delta_base = ws + p.word_bytes + kPairWordTail;          // includes the front pad
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(smem);
    uint32_t wa = (uint32_t)__cvta_generic_to_shared(word);
    uint32_t da = (uint32_t)__cvta_generic_to_shared(delta_base) + kPairDeltaFront;  // &delta[0]
    uint32_t da1 = da - (uint32_t)sizeof(MemT);                                     // &delta[-1]
    // this lane's entries of the first tile: record, duration, successor row
    uint32_t rec0 = sbase + kRecB * (uint32_t)lane, w0 = sbase + p.rec_bytes + 8u * (uint32_t)lane,
             sell0 = sbase + p.rec_bytes + p.w_bytes + 4u * (uint32_t)lane;
    int n_tiles = p.n_tiles;
    MOC_KEEP(wa);
    MOC_KEEP(da);
    MOC_KEEP(da1);
    MOC_KEEP(rec0);
    MOC_KEEP(w0);
    MOC_KEEP(sell0);
    MOC_KEEP(n_tiles);
    if (lane == 0) *reinterpret_cast<uint32_t*>(ws + p.word_bytes) = 0x00010001u;   // owned by empty node slots
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
            const int nvec_d = (T + 2 + kPerVec - 1) / kPerVec;        // vectors covering delta[0..T+1]
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
                    // ids outside [0, n) go to the spare word n; the copy count exposes them
                    const uint32_t addr = wa + 4u * min((uint32_t)node, (uint32_t)n);
                    const uint32_t old = exch_shared(addr, t1 * 0x10001u);
                    sts_u16_if_nonzero(old, addr + 2, old);
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

            if (kPre == 0 && b_next < b_end) {
                // short rows are read in place; ask for the next one to be brought into L2 meanwhile
                const int64_t off_n = self ? off + group_sum(len_raw, wpb) : off_next;
                const int32_t T_n = self ? __shfl_sync(0xFFFFFFFFu, len_next, 0) : T_next;
                if (T_n >= n && T_n <= p.max_T) {
                    const char* nrow = reinterpret_cast<const char*>(p.seqs + off_n);
                    const int bytes = 4 * T_n;
                    for (int i = 128 * lane; i < bytes; i += 4096) asm volatile("prefetch.global.L2 [%0];" ::"l"(nrow + i));
                    if (lane == 31) asm volatile("prefetch.global.L2 [%0];" ::"l"(nrow + bytes - 4));
                }
            }

            // ---- stage 2 and the scatter of stage 3: two node slots per lane and tile
            uint32_t vmin = 0xFFFFFFFFu, depw = 0, capw = 0;
            uint64_t acc = 0;
            {
                uint32_t prec = rec0, pw = w0, ps = sell0;
                for (int d = 0; d < n_tiles; ++d, prec += 64u * kRecB, pw += 512u) {
                    uint32_t ab[2], naa[2], nbb[2], Ga[2], Gb[2];
                    MemT m[2];
                    int rows = 0;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t x;
                        if constexpr (sizeof(MemT) == 4) {
                            const uint2 r = lds_v2(prec + 32u * kRecB * h);
                            x = r.x;
                            m[h] = (MemT)r.y;
                        } else {
                            const uint4 r = lds_v4(prec + 32u * kRecB * h);
                            x = r.x;
                            m[h] = (MemT)((uint64_t)r.z | ((uint64_t)r.w << 32));
                        }
                        if (h == 0) rows = (int)(x >> 16);
                        const uint32_t own = lds_u32(wa + (x & 0xFFFFu));
                        vmin = min(vmin, own);
                        const uint32_t sw = swap_halves(own);
                        const uint32_t mn = min_u16x2(own, sw), mx = max_u16x2(own, sw);   // (a, a), (b, b)
                        ab[h] = __byte_perm(mn, mx, 0x7610);   // (a, b)
                        naa[h] = 0x00010000u - mn;             // (-a, -a) mod 2^16 for a >= 1
                        nbb[h] = 0x00010000u - mx;
                        Ga[h] = mx - mn;                       // (b - a, b - a)
                        Gb[h] = 0x00010000u - Ga[h];           // (a - b, a - b) mod 2^16 when a < b
                    }
                    // successors of the tile: uniform trip count, used-up lists read the node's own word
                    rows = __shfl_sync(0xFFFFFFFFu, rows, 0);
#pragma unroll 2
                    for (int k = 0; k < rows; ++k) {
                        const uint32_t e = lds_u32(ps);
                        ps += 128u;
                        const uint32_t r0 = lds_u32(wa + (e & 0xFFFFu));
                        const uint32_t r1 = lds_u32(wa + (e >> 16));
                        Ga[0] = __viaddmax_u16x2(r0, naa[0], Ga[0]);
                        Ga[1] = __viaddmax_u16x2(r1, naa[1], Ga[1]);
                        Gb[0] = __viaddmax_u16x2(r0, nbb[0], Gb[0]);
                        Gb[1] = __viaddmax_u16x2(r1, nbb[1], Gb[1]);
                    }
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        depw |= Ga[h];                         // bit 15 or 31: a successor copy before a
                        const uint32_t gg = max_u16x2(__byte_perm(Ga[h], Gb[h], 0x5410), __byte_perm(Ga[h], Gb[h], 0x7632));
                        const uint32_t v = gg + ab[h];                           // (end of b, end of a) mod 2^16
                        const uint32_t a16 = ab[h] & 0xFFFFu, b16 = ab[h] >> 16;
                        const MemT neg_m = -m[h];
                        red_add_shared(da1 + (b16 << kShift), m[h]);
                        red_add_shared(da + ((v & 0xFFFFu) << kShift), neg_m);
                        if (a16 != b16) {
                            red_add_shared(da1 + (a16 << kShift), m[h]);
                            red_add_shared(da + ((v >> 16) << kShift), neg_m);
                            // bit 63 of the duration marks a node that may have one copy only (C_v = 1)
                            const uint64_t wx = lds_u64(pw + 256u * h);
                            capw |= (uint32_t)(wx >> 32);
                            acc += wx;
                        }
                    }
                }
            }
            vmin = __reduce_min_sync(0xFFFFFFFFu, vmin);
            const uint64_t acc_all = (uint64_t)warp_sum64((int64_t)acc);
            const bool cap_ok = !__any_sync(0xFFFFFFFFu, (int32_t)capw < 0);
            const bool well_formed = cap_ok && vmin != 0 && (int)((acc_all >> kPairCntShift) & 0x7FFFu) == T - n;
            const bool dep = __any_sync(0xFFFFFFFFu, (depw & 0x80008000u) != 0);
            const int64_t dur_extra = (int64_t)(acc_all & kPairDurMask);
            __syncwarp();

            if (!well_formed) {
                // status -2, sentinels already set
            } else if (dep) {
                out_st = -1;
                out_du = p.base_dur + dur_extra;
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
                out_du = p.base_dur + dur_extra;
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

// Fast path of the sequence evaluator for C <= 2 copies per node (the paper's experiments all use
// C_v = 2, Section 4.3): one warp evaluates one sequence, warp-synchronously, with the graph staged
// once per block in shared memory.
//
// Representation.  Positions are 1-based and 16 bits wide; 0 means "no copy".  Each node owns one
// 32-bit word holding its (at most two) positions, so a consumer reads both copies of a
// predecessor/successor with one load.  The successor lists are stored as a sliced ELL matrix:
// nodes are sorted by out-degree (descending) and cut into slices of 32; slice s is a dense
// [degree of its first node][32] tile whose row k holds the k-th successor of each of its nodes, as
// the byte offset of that successor's word, padded with the offset of a dummy word that stays zero.
// Lanes read consecutive entries, every lane of a warp runs the same trip count, and the padding
// is neutral for the maxima and minima taken over the successors.
//
// Stages for one sequence seq[0..T) (paper: Section 2, Eqs. 1-8):
//   1. occurrence words   step t exchanges t+1 into the low half of its node's word and moves the
//                         previous occupant to the high half.  A third copy loses a position, which
//                         the check "sum of stored positions == T(T+1)/2" detects; an absent node
//                         (Eq. 7) shows as a zero low half.
//   2. free steps         one lane per node u with copies a <= b (a = b if computed once), one pass
//                         over its successors' words r with three packed 16-bit reductions:
//                           F = max r            latest successor copy: b is kept until max(b, F);
//                           D = min (r - 1)      earliest successor copy: before a = Eq. 5 violated;
//                           G = max (r - b)      mod 2^16 this ranks the copies below b above all
//                                                others, in order: the latest successor copy inside
//                                                (a, b), until which the first copy a is kept
//                                                (Eqs. 2, 3, 5).
//                         A sink's last copy is kept to the end.
//   3. memory profile     delta[p] += m_u, delta[free+1] -= m_u, prefix sum (Eq. 4).
//   4. reductions         peak (Section 2), duration = sum_v w_v + sum over second copies (Eq. 1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "moc_kernels.cuh"

namespace moc {

struct PairParams {
    int32_t n;
    int32_t sell_len;          // entries of the sliced ELL matrix
    int32_t n_slices;          // ceil(n / 32)
    int32_t max_T;             // C * n
    const void* rec;           // n node records (NodeRec<MemT>) in out-degree order
    const uint16_t* sell;      // sell_len byte offsets (4 * successor id, 4 * n = dummy)
    const uint32_t* tile;      // n_slices: first entry of the slice | rows of the slice << 18
    const int64_t* w;          // n durations by node id
    int64_t base_dur;          // sum of all w
    const int32_t* seqs;
    const int32_t* lens;
    const int64_t* offs;
    int32_t B;
    int64_t M;
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_status;
    // shared-memory layout, bytes (multiples of 16)
    uint32_t rec_bytes, tile_bytes, sell_bytes;  // graph, once per block
    uint32_t word_bytes, delta_bytes;                  // per warp
};

constexpr int kPairDeltaFront = 16;  // bytes in front of delta[0]: lands writes of absent nodes

__device__ __forceinline__ int64_t warp_sum64(int64_t v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}
// per-halfword unsigned max / min of two packed 16-bit pairs (one instruction on sm_90 and later)
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
__device__ __forceinline__ uint32_t add_u16x2(uint32_t a, uint32_t b) {  // per halfword, wraps
    uint32_t d;
    asm("add.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Node record: byte offset of the node's word (4 * id) | out-degree << 16, and its output size.
template <typename MemT> struct NodeRec;
template <> struct __align__(8) NodeRec<int32_t> { uint32_t nd; int32_t m; };
template <> struct __align__(16) NodeRec<int64_t> { uint32_t nd; uint32_t pad; int64_t m; };

__device__ __forceinline__ int32_t warp_max_t(int32_t v) { return __reduce_max_sync(0xFFFFFFFFu, v); }
__device__ __forceinline__ int64_t warp_max_t(int64_t v) { return warp_max(v); }

template <typename MemT>
__global__ void __launch_bounds__(512) eval_pair_kernel(const PairParams p) {
    extern __shared__ __align__(16) char smem[];
    using Rec = NodeRec<MemT>;
    // ---- graph -> shared memory, once per block
    Rec* s_rec = reinterpret_cast<Rec*>(smem);
    uint32_t* s_tile = reinterpret_cast<uint32_t*>(smem + p.rec_bytes);
    uint16_t* s_sell = reinterpret_cast<uint16_t*>(smem + p.rec_bytes + p.tile_bytes);
    const uint32_t graph_bytes = p.rec_bytes + p.tile_bytes + p.sell_bytes;
    {
        const Rec* grec = reinterpret_cast<const Rec*>(p.rec);
        for (int i = threadIdx.x; i < p.n; i += blockDim.x) s_rec[i] = grec[i];
        for (int i = threadIdx.x; i < p.n_slices; i += blockDim.x) s_tile[i] = __ldg(&p.tile[i]);
        for (int i = threadIdx.x; i < p.sell_len; i += blockDim.x) s_sell[i] = __ldg(&p.sell[i]);
    }
    __syncthreads();
    wait_for_previous_kernel();  // the packing offsets come from the kernel launched just before

    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    // broadcast from lane 0 so that the compiler knows the warp index is uniform across the warp
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    char* ws = smem + graph_bytes + (size_t)warp * (p.word_bytes + p.delta_bytes);
    uint32_t* word = reinterpret_cast<uint32_t*>(ws);
    uint16_t* word16 = reinterpret_cast<uint16_t*>(ws);
    char* delta_base = ws + p.word_bytes;                          // includes the front pad
    MemT* delta = reinterpret_cast<MemT*>(delta_base + kPairDeltaFront);
    const int n = p.n;
    const int n_warps = gridDim.x * wpb;
    constexpr int kPerVec = 16 / (int)sizeof(MemT);  // delta entries per 16-byte vector
    constexpr int kRegVecs = sizeof(MemT) == 4 ? 7 : 0;  // scan keeps up to this many vectors per lane in registers

    for (int b = blockIdx.x * wpb + warp; b < p.B; b += n_warps) {
        const int64_t off = p.offs[b];
        const int32_t T = p.lens[b];
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

            // ---- stage 1: occurrence words
            {
                const int32_t* row = p.seqs + off;
                const int a = (int)((reinterpret_cast<uintptr_t>(row) & 15) >> 2);
                const int nvec = (T + a + 3) >> 2;
                auto put = [&](int node, uint32_t t1) {
                    if ((unsigned)node < (unsigned)n) {
                        const uint32_t old = atomicExch(&word[node], t1);
                        if (old) word16[2 * node + 1] = (uint16_t)old;
                    }
                };
                // vectors that lie completely inside the row
                for (int i = lane; i < nvec; i += 32) {
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

            // ---- stage 2 and the scatter of stage 3: one lane per node, slices in out-degree order
            uint32_t vmin = 0xFFFFFFFFu, vsum = 0;
            bool dep = false;
            int64_t dur_extra = 0;
            for (int i0 = 0, sl = 0; i0 < n; i0 += 32, ++sl) {
                const int i = i0 + lane;
                const bool live = i < n;
                Rec rec;
                rec.nd = 4u * (uint32_t)n;  // lanes past the last node look at the dummy word
                rec.m = 0;
                if (live) rec = s_rec[i];
                const uint32_t own = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(word) + (rec.nd & 0xFFFFu));
                const uint32_t lo = own & 0xFFFFu, hi = own >> 16;
                const bool dbl = hi != 0;
                const uint32_t hh = dbl ? hi : lo;
                const uint32_t a = min(lo, hh), bpos = max(lo, hh);
                const uint32_t nbb = ((0x10000u - bpos) & 0xFFFFu) * 0x10001u;   // -b in both halves
                // successors of the slice: uniform trip count, padded entries read the dummy word
                const uint32_t tl = __shfl_sync(0xFFFFFFFFu, s_tile[sl], 0);
                const uint16_t* pj = s_sell + (tl & 0x3FFFFu) + lane;
                const int rows = (int)(tl >> 18);
                uint32_t F = 0, D = 0xFFFFFFFFu, G = 0;
#pragma unroll 4
                for (int k = 0; k < rows; ++k) {
                    const uint32_t v4 = pj[k * 32];
                    const uint32_t r = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(word) + v4);
                    F = max_u16x2(F, r);
                    D = min_u16x2(D, r - 0x00010001u);   // empty half -> 0xFFFF
                    G = max_u16x2(G, add_u16x2(r, nbb));
                }
                if (live) {
                    const uint32_t deg = rec.nd >> 16;
                    vmin = min(vmin, lo);
                    vsum += lo + hi;
                    const uint32_t Fm = max(F & 0xFFFFu, F >> 16);
                    const uint32_t Dm = min(D & 0xFFFFu, D >> 16);
                    if (deg != 0 && Dm + 1 < a) dep = true;   // a successor copy before the first copy of u
                    const uint32_t fb = deg != 0 ? max(Fm, bpos) : (uint32_t)T;
                    atomic_add_mem(&delta[(int)bpos - 1], rec.m);
                    atomic_add_mem(&delta[fb], (MemT)(-rec.m));
                    if (dbl) {
                        // latest successor copy h with a < h < b, if any: (h - b) mod 2^16 is the largest
                        const uint32_t h = (max(G & 0xFFFFu, G >> 16) + bpos) & 0xFFFFu;
                        const uint32_t fa = (h - 1u < bpos - 1u) ? h : a;
                        atomic_add_mem(&delta[(int)a - 1], rec.m);
                        atomic_add_mem(&delta[fa], (MemT)(-rec.m));
                        dur_extra += __ldg(&p.w[(rec.nd & 0xFFFFu) >> 2]);
                    }
                }
            }
            vmin = __reduce_min_sync(0xFFFFFFFFu, vmin);
            vsum = __reduce_add_sync(0xFFFFFFFFu, vsum);
            const bool well_formed = vmin != 0 && vsum == (uint32_t)T * ((uint32_t)T + 1u) / 2u;
            dep = __any_sync(0xFFFFFFFFu, dep);
            __syncwarp();

            if (!well_formed) {
                // status -2, sentinels already set
            } else if (dep) {
                out_st = -1;
                out_du = p.base_dur + warp_sum64(dur_extra);
            } else {
                // ---- stage 3 + 4: prefix sum and running maximum; lane owns V consecutive vectors
                const int4* d4 = reinterpret_cast<const int4*>(delta) + lane * V;
                MemT peak = 0;
                if (kRegVecs > 0 && V <= kRegVecs) {
                    int4 q[kRegVecs > 0 ? kRegVecs : 1];
                    int32_t s = 0;
#pragma unroll
                    for (int j = 0; j < kRegVecs; ++j) {
                        q[j] = make_int4(0, 0, 0, 0);
                        if (j < V) q[j] = d4[j];
                        s += q[j].x + q[j].y + q[j].z + q[j].w;
                    }
                    int32_t run = warp_inclusive_sum(s, lane) - s;
                    int32_t pk = 0;
#pragma unroll
                    for (int j = 0; j < kRegVecs; ++j) {
                        run += q[j].x; pk = max(pk, run);
                        run += q[j].y; pk = max(pk, run);
                        run += q[j].z; pk = max(pk, run);
                        run += q[j].w; pk = max(pk, run);
                    }
                    peak = (MemT)pk;
                } else {
                    MemT s = 0;
                    for (int j = 0; j < V; ++j) {
                        const int4 q = d4[j];
                        if constexpr (sizeof(MemT) == 4) s += q.x + q.y + q.z + q.w;
                        else {
                            const longlong2 l = *reinterpret_cast<const longlong2*>(&q);
                            s += (MemT)(l.x + l.y);
                        }
                    }
                    MemT run = warp_inclusive_sum(s, lane) - s;
                    for (int j = 0; j < V; ++j) {
                        const int4 q = d4[j];
                        if constexpr (sizeof(MemT) == 4) {
                            run += q.x; peak = max(peak, run);
                            run += q.y; peak = max(peak, run);
                            run += q.z; peak = max(peak, run);
                            run += q.w; peak = max(peak, run);
                        } else {
                            const longlong2 l = *reinterpret_cast<const longlong2*>(&q);
                            run += (MemT)l.x; peak = run > peak ? run : peak;
                            run += (MemT)l.y; peak = run > peak ? run : peak;
                        }
                    }
                }
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
    }
}

}  // namespace moc

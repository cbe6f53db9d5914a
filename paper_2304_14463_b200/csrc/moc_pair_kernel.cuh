// Fast path of the sequence evaluator for C <= 2 copies per node (the paper's experiments all use
// C_v = 2, Section 4.3): one warp evaluates one sequence, warp-synchronously, with the graph staged
// once per block in shared memory.
//
// Representation.  Positions are 1-based and 16 bits wide; 0 means "no copy".  Each node owns one
// 32-bit word holding its (at most two) positions, so a consumer reads both copies of a
// predecessor/successor with one load.  The successor lists are stored in jagged-diagonal form:
// nodes are sorted by out-degree (descending) and column k holds the k-th successor of every node
// that has one, so that lanes working on consecutive sorted nodes read consecutive entries and a
// warp's trip count is the out-degree of its first lane.
//
// Stages for one sequence seq[0..T) (paper: Section 2, Eqs. 1-8):
//   1. occurrence words   step t exchanges t+1 into the low half of its node's word and moves the
//                         previous occupant to the high half.  A third copy loses a position, which
//                         the check "sum of stored positions == T(T+1)/2" detects; an absent node
//                         (Eq. 7) shows as a zero low half.
//   2. free steps         last copy b of u: free = max(b, latest copy of any successor) -- every
//                         successor copy after b falls in b's window; first copy a of a node
//                         computed twice: free = latest successor copy inside (a, b), else a
//                         (Eqs. 2, 3, 5).  A sink's last copy is kept to the end.  Precedence
//                         (Eq. 5) holds iff no successor copy precedes the first copy of u.
//   3. memory profile     delta[p] += m_u, delta[free+1] -= m_u, prefix sum (Eq. 4).
//   4. reductions         peak (Section 2), duration = sum_v w_v + sum over second copies (Eq. 1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "moc_kernels.cuh"

namespace moc {

struct PairParams {
    int32_t n;
    int32_t n_edges;
    int32_t max_deg;
    int32_t max_T;             // C * n
    const uint32_t* nd;        // n: node id | out-degree << 16, sorted by out-degree descending
    const uint16_t* jds;       // n_edges successor ids, column after column
    const uint32_t* colstart;  // max_deg + 1 column starts
    const void* mm;            // n output sizes (MemT) in sorted-node order
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
    uint32_t nd_bytes, mm_bytes, col_bytes, jds_bytes;  // graph, once per block
    uint32_t word_bytes, delta_bytes, list_bytes;       // per warp
};

constexpr int kPairDeltaFront = 16;  // bytes in front of delta[0]: lands writes of absent nodes

__device__ __forceinline__ int64_t warp_sum64(int64_t v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}
__device__ __forceinline__ int32_t warp_max_t(int32_t v) { return __reduce_max_sync(0xFFFFFFFFu, v); }
__device__ __forceinline__ int64_t warp_max_t(int64_t v) { return warp_max(v); }

template <typename MemT>
__global__ void __launch_bounds__(512) eval_pair_kernel(const PairParams p) {
    extern __shared__ __align__(16) char smem[];
    // ---- graph -> shared memory, once per block
    uint32_t* s_nd = reinterpret_cast<uint32_t*>(smem);
    MemT* s_mm = reinterpret_cast<MemT*>(smem + p.nd_bytes);
    uint32_t* s_col = reinterpret_cast<uint32_t*>(smem + p.nd_bytes + p.mm_bytes);
    uint16_t* s_jds = reinterpret_cast<uint16_t*>(smem + p.nd_bytes + p.mm_bytes + p.col_bytes);
    const uint32_t graph_bytes = p.nd_bytes + p.mm_bytes + p.col_bytes + p.jds_bytes;
    {
        const int n = p.n;
        const MemT* gm = reinterpret_cast<const MemT*>(p.mm);
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            s_nd[i] = __ldg(&p.nd[i]);
            s_mm[i] = __ldg(&gm[i]);
        }
        for (int i = threadIdx.x; i <= p.max_deg; i += blockDim.x) s_col[i] = __ldg(&p.colstart[i]);
        for (int i = threadIdx.x; i < p.n_edges; i += blockDim.x) s_jds[i] = __ldg(&p.jds[i]);
    }
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const uint32_t warp_bytes = p.word_bytes + p.delta_bytes + p.list_bytes;
    char* ws = smem + graph_bytes + (size_t)warp * warp_bytes;
    uint32_t* word = reinterpret_cast<uint32_t*>(ws);
    uint16_t* word16 = reinterpret_cast<uint16_t*>(ws);
    char* delta_base = ws + p.word_bytes;                          // includes the front pad
    MemT* delta = reinterpret_cast<MemT*>(delta_base + kPairDeltaFront);
    uint16_t* list = reinterpret_cast<uint16_t*>(ws + p.word_bytes + p.delta_bytes);
    const int n = p.n;
    const int n_warps = gridDim.x * wpb;
    const uint32_t lt_mask = (1u << lane) - 1u;
    constexpr int kPerVec = 16 / (int)sizeof(MemT);  // delta entries per 16-byte vector

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

            // ---- stage 2, last copies: one lane per node in out-degree order
            uint32_t vmin = 0xFFFFFFFFu, vsum = 0;
            bool dep = false;
            int n_dbl = 0;
            for (int i0 = 0; i0 < n; i0 += 32) {
                const int i = i0 + lane;
                bool dbl = false;
                if (i < n) {
                    const uint32_t nd = s_nd[i];
                    const uint32_t u = nd & 0xFFFFu, deg = nd >> 16;
                    const uint32_t own = word[u];
                    const uint32_t lo = own & 0xFFFFu, hi = own >> 16;
                    vmin = min(vmin, lo);
                    vsum += lo + hi;
                    dbl = hi != 0;
                    const uint32_t hh = dbl ? hi : lo;
                    const uint32_t a = min(lo, hh), bpos = max(lo, hh);
                    uint32_t F = 0, D = 0xFFFFFFFFu;
                    for (uint32_t k = 0; k < deg; ++k) {
                        const uint32_t v = s_jds[s_col[k] + i];
                        const uint32_t r = word[v];
                        F = __vmaxu2(F, r);                 // latest copy, per half
                        D = __vminu2(D, r - 0x00010001u);   // earliest copy (0-based); empty half -> 0xFFFF
                    }
                    const uint32_t Fm = max(F & 0xFFFFu, F >> 16);
                    const uint32_t Dm = min(D & 0xFFFFu, D >> 16);
                    if (deg != 0 && Dm + 1 < a) dep = true;   // a successor copy before the first copy of u
                    const uint32_t fb = deg != 0 ? max(Fm, bpos) : (uint32_t)T;
                    const MemT mu = s_mm[i];
                    atomic_add_mem(&delta[(int)bpos - 1], mu);
                    atomic_add_mem(&delta[fb], (MemT)(-mu));
                }
                const uint32_t mask = __ballot_sync(0xFFFFFFFFu, dbl);
                if (dbl) list[n_dbl + __popc(mask & lt_mask)] = (uint16_t)i;
                n_dbl += __popc(mask);
            }
            vmin = __reduce_min_sync(0xFFFFFFFFu, vmin);
            vsum = __reduce_add_sync(0xFFFFFFFFu, vsum);
            const bool well_formed = vmin != 0 && vsum == (uint32_t)T * ((uint32_t)T + 1u) / 2u;
            __syncwarp();

            // ---- stage 2, first copies of nodes computed twice
            int64_t dur_extra = 0;
            if (well_formed) {
                for (int j = lane; j < n_dbl; j += 32) {
                    const int i = list[j];
                    const uint32_t nd = s_nd[i];
                    const uint32_t u = nd & 0xFFFFu, deg = nd >> 16;
                    const uint32_t own = word[u];
                    const uint32_t lo = own & 0xFFFFu, hi = own >> 16;
                    const uint32_t a = min(lo, hi), bpos = max(lo, hi);
                    uint32_t fa = a;
                    for (uint32_t k = 0; k < deg; ++k) {
                        const uint32_t v = s_jds[s_col[k] + i];
                        const uint32_t r = word[v];
                        const uint32_t x = r & 0xFFFFu, y = r >> 16;
                        fa = max(fa, max(x < bpos ? x : 0u, y < bpos ? y : 0u));
                    }
                    const MemT mu = s_mm[i];
                    atomic_add_mem(&delta[(int)a - 1], mu);
                    atomic_add_mem(&delta[fa], (MemT)(-mu));
                    dur_extra += __ldg(&p.w[u]);
                }
            }
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
                MemT peak = 0;
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

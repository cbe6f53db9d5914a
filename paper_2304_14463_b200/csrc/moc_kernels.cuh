// Device code of the sequence evaluator: one thread group (a warp, part of a block or a whole
// block) evaluates one sequence at a time with all per-sequence state on chip.
//
// Stages for one sequence seq[0..T) (paper: Section 2, Eqs. 1-8):
//   1. occurrence table   for every node the positions of its copies (at most C, Section 2),
//                         built by a scatter over the steps; detects ids out of range, absent
//                         nodes (Eq. 7) and more than C copies.
//   2. free steps         for every copy p of node u with next copy q (or T): the interval end is
//                         the latest copy of any successor of u inside (p, q), else p itself
//                         (Eqs. 2, 3, 5); the last copy of a sink is kept to T-1.  This is the
//                         consumer-side scatter-max "free[latest copy of u before t] = max(.., t)"
//                         turned into a gather per producer copy, which needs no atomics.
//                         Precedence (Eq. 5) holds iff no copy of a successor precedes the first
//                         copy of u.
//   3. memory profile     delta[p] += m_u, delta[free+1] -= m_u, prefix sum (Eq. 4, inclusive ends).
//   4. reductions         peak = max profile (Section 2), duration = sum over copies of w (Eq. 1),
//                         status against the budget M.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace moc {

struct GraphDev {
    int32_t n;
    int32_t C;
    const int32_t* succ_start;  // n+1, successor lists (CSR)
    const int32_t* succ;        // distinct edges, grouped by producer
    const int64_t* w;           // n durations
    const void* m;              // n output sizes, int32 or int64 (matches MemT)
    const int32_t* cap;         // n per-node caps C_v <= C, or nullptr: every node may have C copies
};

struct EvalParams {
    GraphDev g;
    const int32_t* seqs;
    const int32_t* lens;
    const int64_t* offs;  // B+1, exclusive prefix sum of max(lens,0)
    int32_t B;
    int64_t M;
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_status;
    int64_t* out_profile;  // profile mode only
    int32_t* out_free;     // profile mode only, may be null
    int32_t single_len;    // profile mode only: length of the one sequence at seqs[0..)
    // per-group state layout (bytes, each a multiple of 16)
    uint32_t cnt_bytes, occ_bytes, delta_bytes, group_bytes;
    char* gstate;  // global-state variant: base of the per-block state slices
};

constexpr int kRedBytes = 32 * 8 * 3 + 16;  // three 32-entry reduction rows + a flag word

template <typename PosT> struct PosNone;
template <> struct PosNone<uint16_t> { static constexpr uint32_t value = 0xFFFFu; };
template <> struct PosNone<int32_t> { static constexpr uint32_t value = 0x7FFFFFFFu; };

template <int G>
__device__ __forceinline__ void group_sync(int bar_id) {
    if constexpr (G == 32) {
        __syncwarp();
    } else {
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(G) : "memory");
    }
}

template <typename T>
__device__ __forceinline__ T warp_inclusive_sum(T v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}
template <typename T>
__device__ __forceinline__ T warp_max(T v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        T o = __shfl_xor_sync(0xFFFFFFFFu, v, d);
        v = o > v ? o : v;
    }
    return v;
}
template <typename T>
__device__ __forceinline__ T warp_sum(T v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

__device__ __forceinline__ void atomic_add_mem(int32_t* p, int32_t v) { atomicAdd(p, v); }
__device__ __forceinline__ void atomic_add_mem(int64_t* p, int64_t v) {
    atomicAdd(reinterpret_cast<unsigned long long*>(p), static_cast<unsigned long long>(v));
}

// Evaluates sequence b with the G threads of one group.  `tid` is the thread's index in the group.
template <int G, typename MemT, typename PosT, int CP, bool kProfile>
__device__ __forceinline__ void eval_one(const EvalParams& p, const int b, const int tid,
                                         const int bar_id, char* state) {
    constexpr uint32_t NONE = PosNone<PosT>::value;
    const int n = p.g.n, C = p.g.C;
    int32_t* cnt = reinterpret_cast<int32_t*>(state);
    PosT* occ = reinterpret_cast<PosT*>(state + p.cnt_bytes);
    MemT* delta = reinterpret_cast<MemT*>(state + p.cnt_bytes + p.occ_bytes);
    char* red = state + p.cnt_bytes + p.occ_bytes + p.delta_bytes;
    MemT* red_a = reinterpret_cast<MemT*>(red);              // 32 entries (8 bytes reserved each)
    int64_t* red_dur = reinterpret_cast<int64_t*>(red + 256);
    MemT* red_max = reinterpret_cast<MemT*>(red + 512);
    int32_t* red_flags = reinterpret_cast<int32_t*>(red + 768);
    const int lane = tid & 31, warp = tid >> 5;

    const int64_t off = kProfile ? 0 : p.offs[b];
    const int32_t T = kProfile ? p.single_len : p.lens[b];
    const bool len_ok = T >= n && (int64_t)T <= (int64_t)C * n;

    int bad = len_ok ? 0 : 1, dep = 0;
    int64_t dur = 0;

    if (len_ok) {
        // ---- clear the per-sequence state
        {
            const int4 z = make_int4(0, 0, 0, 0);
            const int4 f = make_int4(-1, -1, -1, -1);
            int4* c4 = reinterpret_cast<int4*>(cnt);
            for (int i = tid; i < (int)(p.cnt_bytes >> 4); i += G) c4[i] = z;
            int4* o4 = reinterpret_cast<int4*>(occ);
            if constexpr (sizeof(PosT) == 2) {
                for (int i = tid; i < (int)(p.occ_bytes >> 4); i += G) o4[i] = f;
            } else {
                const int4 f32 = make_int4(0x7FFFFFFF, 0x7FFFFFFF, 0x7FFFFFFF, 0x7FFFFFFF);
                for (int i = tid; i < (int)(p.occ_bytes >> 4); i += G) o4[i] = f32;
            }
            int4* d4 = reinterpret_cast<int4*>(delta);
            const int nd = (int)(((size_t)(T + 1) * sizeof(MemT) + 15) >> 4);
            for (int i = tid; i < nd; i += G) d4[i] = z;
            if (G > 32 && tid == 0) *red_flags = 0;
        }
        group_sync<G>(bar_id);

        // ---- stage 1: occurrence table.  Rows are 4-byte aligned only: read 16-byte vectors from
        // the enclosing aligned range and mask what lies outside the row; a vector that would
        // reach outside the packed array is read element by element.
        {
            const int32_t* row = p.seqs + off;
            const int a = (int)((reinterpret_cast<uintptr_t>(row) & 15) >> 2);
            const int nvec = (T + a + 3) >> 2;
            const int64_t S = kProfile ? (int64_t)T : p.offs[p.B];
            for (int i = tid; i < nvec; i += G) {
                const int t0 = 4 * i - a;
                const int64_t e0 = off + t0;
                int4 v;
                if (e0 >= 0 && e0 + 4 <= S) {
                    v = __ldg(reinterpret_cast<const int4*>(row + t0));
                } else {
                    v.x = (e0 >= 0 && e0 < S) ? __ldg(row + t0) : 0;
                    v.y = (e0 + 1 >= 0 && e0 + 1 < S) ? __ldg(row + t0 + 1) : 0;
                    v.z = (e0 + 2 >= 0 && e0 + 2 < S) ? __ldg(row + t0 + 2) : 0;
                    v.w = (e0 + 3 >= 0 && e0 + 3 < S) ? __ldg(row + t0 + 3) : 0;
                }
                const int vals[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int t = t0 + k;
                    if ((unsigned)t < (unsigned)T) {
                        const int node = vals[k];
                        if ((unsigned)node < (unsigned)n) {
                            const int slot = atomicAdd(&cnt[node], 1);
                            if (slot < C) occ[node * CP + slot] = (PosT)t;
                            else bad = 1;
                        } else {
                            bad = 1;
                        }
                    }
                }
            }
        }
        group_sync<G>(bar_id);

        // ---- stage 2 + scatter of stage 3: one thread per producer node
        const MemT* mem = reinterpret_cast<const MemT*>(p.g.m);
        for (int u = tid; u < n; u += G) {
            const int c = cnt[u];
            if (c < 1) bad = 1;
            if (p.g.cap != nullptr && c > __ldg(&p.g.cap[u])) bad = 1;
            uint32_t o[CP], f[CP];
#pragma unroll
            for (int j = 0; j < CP; ++j) o[j] = occ[u * CP + j];
            // sort ascending; empty slots hold NONE (largest) and end up last
#pragma unroll
            for (int i = 1; i < CP; ++i)
#pragma unroll
                for (int j = CP - 1; j >= i; --j) {
                    const uint32_t lo = min(o[j - 1], o[j]), hi = max(o[j - 1], o[j]);
                    o[j - 1] = lo;
                    o[j] = hi;
                }
#pragma unroll
            for (int j = 0; j < CP; ++j) f[j] = o[j];
            dur += (int64_t)c * __ldg(&p.g.w[u]);
            const int s0 = __ldg(&p.g.succ_start[u]), s1 = __ldg(&p.g.succ_start[u + 1]);
            if (s0 == s1) {
                // result of the computation: its last copy stays to the final step
                const int jl = min(c, C) - 1;
#pragma unroll
                for (int j = 0; j < CP; ++j)
                    if (j == jl) f[j] = (uint32_t)(T - 1);
            }
            for (int e = s0; e < s1; ++e) {
                const int v = __ldg(&p.g.succ[e]);
                uint32_t r[CP];
#pragma unroll
                for (int i = 0; i < CP; ++i) r[i] = occ[v * CP + i];
#pragma unroll
                for (int i = 0; i < CP; ++i) {
                    const uint32_t x = r[i];
                    if (x != NONE) {
                        if (x < o[0]) dep = 1;  // a consumer copy before the first copy of u (Eq. 5)
#pragma unroll
                        for (int j = 0; j < CP; ++j) {
                            const bool in = o[j] < x && (j + 1 == CP || x < o[j + 1]);
                            if (in) f[j] = max(f[j], x);
                        }
                    }
                }
            }
            const MemT mu = __ldg(&mem[u]);
#pragma unroll
            for (int j = 0; j < CP; ++j) {
                if (o[j] != NONE) {
                    atomic_add_mem(&delta[o[j]], mu);
                    atomic_add_mem(&delta[f[j] + 1], (MemT)(-mu));
                    if constexpr (kProfile) {
                        if (p.out_free) p.out_free[o[j]] = (int32_t)f[j];
                    }
                }
            }
        }
    }

    // ---- combine flags and duration over the group
    int flags = bad | (dep << 1);
    if constexpr (G == 32) {
        flags = __reduce_or_sync(0xFFFFFFFFu, flags);
        dur = warp_sum(dur);
    } else {
        if (len_ok) {
            flags = __reduce_or_sync(0xFFFFFFFFu, flags);
            dur = warp_sum(dur);
            if (lane == 0) {
                if (flags) atomicOr(red_flags, flags);
                red_dur[warp] = dur;
            }
            group_sync<G>(bar_id);
            flags = *red_flags;
        }
    }

    MemT peak = 0;
    if (flags == 0) {
        // ---- stage 3: prefix sum of the deltas; each thread owns a contiguous chunk
        const int chunk = ((T + G - 1) / G) | 1;  // odd stride: conflict-free for 4-byte entries
        const int tb = min(tid * chunk, T), te = min(tb + chunk, T);
        MemT s = 0;
        for (int t = tb; t < te; ++t) s += delta[t];
        MemT incl = warp_inclusive_sum(s, lane);
        if constexpr (G > 32) {
            if (lane == 31) red_a[warp] = incl;
            group_sync<G>(bar_id);
            MemT prefix = 0;
            for (int k = 0; k < warp; ++k) prefix += red_a[k];
            incl += prefix;
        }
        MemT run = incl - s;
        for (int t = tb; t < te; ++t) {
            run += delta[t];
            peak = run > peak ? run : peak;
            if constexpr (kProfile) p.out_profile[t] = (int64_t)run;
        }
        // ---- stage 4: peak
        peak = warp_max(peak);
        if constexpr (G > 32) {
            if (lane == 0) red_max[warp] = peak;
            group_sync<G>(bar_id);
        }
    } else if constexpr (kProfile) {
        for (int t = tid; t < T; t += G) {
            p.out_profile[t] = -1;
            if (p.out_free) p.out_free[t] = -1;
        }
    }

    if (tid == 0) {
        int64_t pk = (int64_t)peak, du = dur;
        if constexpr (G > 32) {
            if (flags == 0) {
                for (int k = 1; k < G / 32; ++k) {
                    const MemT o = red_max[k];
                    pk = (int64_t)o > pk ? (int64_t)o : pk;
                }
            }
            if (len_ok) {
                du = 0;
                for (int k = 0; k < G / 32; ++k) du += red_dur[k];
            }
        }
        int32_t st;
        if (flags & 1) { st = -2; pk = -1; du = -1; }
        else if (flags & 2) { st = -1; pk = -1; }
        else st = (pk <= p.M) ? 1 : 0;
        if constexpr (kProfile) {
            p.out_status[0] = st;
        } else {
            p.out_peak[b] = pk;
            p.out_dur[b] = du;
            p.out_status[b] = st;
        }
    }
    // all reads of this sequence's state are done before the next one clears it
    group_sync<G>(bar_id);
}

// Persistent kernel, state in shared memory: group g of the grid takes sequences g, g+NG, ...
template <int G, typename MemT, int CP, bool kProfile>
__global__ void __launch_bounds__(1024) eval_shared_kernel(const EvalParams p) {
    extern __shared__ __align__(16) char smem[];
    const int gpc = blockDim.x / G;
    const int gi = threadIdx.x / G, tid = threadIdx.x % G;
    char* state = smem + (size_t)gi * p.group_bytes;
    const int n_groups = gridDim.x * gpc;
    for (int b = blockIdx.x * gpc + gi; b < p.B; b += n_groups)
        eval_one<G, MemT, uint16_t, CP, kProfile>(p, b, tid, gi + 1, state);
}

// Same evaluation with the per-sequence state in a global-memory slice per block, for graphs
// whose state does not fit in shared memory (or whose sequences are longer than 65534 steps).
template <int CP, bool kProfile>
__global__ void __launch_bounds__(1024) eval_global_kernel(const EvalParams p) {
    char* state = p.gstate + (size_t)blockIdx.x * p.group_bytes;
    for (int b = blockIdx.x; b < p.B; b += gridDim.x)
        eval_one<1024, int64_t, int32_t, CP, kProfile>(p, b, threadIdx.x, 0, state);
}

// offs = exclusive prefix sum of max(lens, 0); offs[B] = total.
// Block j owns elements [j*kOffsTile, (j+1)*kOffsTile): it first adds up everything in front of its
// tile (redundantly with the other blocks -- B is small, and this needs no cross-block handshake),
// then scans its own tile.
constexpr int kOffsThreads = 256;
constexpr int kOffsPer = 4;
constexpr int kOffsTile = kOffsThreads * kOffsPer;

static __global__ void __launch_bounds__(kOffsThreads) offsets_kernel(const int32_t* __restrict__ lens, int32_t B,
                                                                int64_t* __restrict__ offs) {
    __shared__ int64_t wsum[kOffsThreads / 32];
    __shared__ int64_t wtot[kOffsThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t tile0 = (int64_t)blockIdx.x * kOffsTile;
    // ---- sum of everything before the tile (16-byte loads, several in flight per thread)
    int64_t s = 0;
    if ((reinterpret_cast<uintptr_t>(lens) & 15) == 0) {
        const int4* l4 = reinterpret_cast<const int4*>(lens);
        const int64_t n4 = tile0 >> 2;  // the tile size is a multiple of 4
        int64_t s0 = 0, s1 = 0, s2 = 0, s3 = 0;
        int64_t i = tid;
        for (; i + 3 * kOffsThreads < n4; i += 4 * kOffsThreads) {
            const int4 a = __ldg(l4 + i), b = __ldg(l4 + i + kOffsThreads), c = __ldg(l4 + i + 2 * kOffsThreads),
                       d = __ldg(l4 + i + 3 * kOffsThreads);
            s0 += (int64_t)max(a.x, 0) + max(a.y, 0) + max(a.z, 0) + max(a.w, 0);
            s1 += (int64_t)max(b.x, 0) + max(b.y, 0) + max(b.z, 0) + max(b.w, 0);
            s2 += (int64_t)max(c.x, 0) + max(c.y, 0) + max(c.z, 0) + max(c.w, 0);
            s3 += (int64_t)max(d.x, 0) + max(d.y, 0) + max(d.z, 0) + max(d.w, 0);
        }
        for (; i < n4; i += kOffsThreads) {
            const int4 a = __ldg(l4 + i);
            s0 += (int64_t)max(a.x, 0) + max(a.y, 0) + max(a.z, 0) + max(a.w, 0);
        }
        s = s0 + s1 + s2 + s3;
    } else {
        for (int64_t i = tid; i < tile0; i += kOffsThreads) {
            const int32_t v = __ldg(lens + i);
            s += v > 0 ? v : 0;
        }
    }
    s = warp_sum(s);
    if (lane == 0) wtot[warp] = s;
    // ---- own tile: kOffsPer consecutive elements per thread
    int32_t loc[kOffsPer];
    int64_t t = 0;
#pragma unroll
    for (int k = 0; k < kOffsPer; ++k) {
        const int64_t i = tile0 + tid * kOffsPer + k;
        const int32_t v = i < B ? __ldg(lens + i) : 0;
        loc[k] = v > 0 ? v : 0;
        t += loc[k];
    }
    const int64_t incl = warp_inclusive_sum(t, lane);
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    int64_t run = incl - t;
    for (int k = 0; k < kOffsThreads / 32; ++k) {
        run += wtot[k];
        if (k < warp) run += wsum[k];
    }
#pragma unroll
    for (int k = 0; k < kOffsPer; ++k) {
        const int64_t i = tile0 + tid * kOffsPer + k;
        if (i < B) offs[i] = run;
        run += loc[k];
        if (i == B - 1) offs[B] = run;
    }
}

// 16-bit node ids -> 32-bit node ids (the evaluation kernels read int32 rows); 8 ids per thread and
// step through 16-byte loads when the source is aligned.
static __global__ void __launch_bounds__(256) widen_ids_kernel(const uint16_t* __restrict__ src, int32_t* __restrict__ dst, int64_t count) {
    const int64_t n8 = count >> 3, stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if ((reinterpret_cast<uintptr_t>(src) & 15) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        int4* d4 = reinterpret_cast<int4*>(dst);
        for (int64_t i = tid; i < n8; i += stride) {
            const uint4 v = __ldg(s4 + i);
            d4[2 * i] = make_int4((int)(v.x & 0xFFFFu), (int)(v.x >> 16), (int)(v.y & 0xFFFFu), (int)(v.y >> 16));
            d4[2 * i + 1] = make_int4((int)(v.z & 0xFFFFu), (int)(v.z >> 16), (int)(v.w & 0xFFFFu), (int)(v.w >> 16));
        }
        for (int64_t i = 8 * n8 + tid; i < count; i += stride) dst[i] = (int32_t)src[i];
    } else {
        for (int64_t i = tid; i < count; i += stride) dst[i] = (int32_t)src[i];
    }
}

}  // namespace moc

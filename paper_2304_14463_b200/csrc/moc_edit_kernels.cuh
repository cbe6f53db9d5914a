// Device code of the incremental evaluation: sequences that differ from an already evaluated parent
// by one edit (insert a copy, delete a copy, move a copy) are evaluated from the parent's cached
// evaluation instead of from scratch.  Retention intervals are local to a node's copies (Section 2,
// Eqs. 2, 3, 5): an edit of a copy of node x changes only the intervals of x itself and of the
// predecessors of x (their copies are consumed by the copies of x); every other interval keeps its
// place relative to the unchanged steps.  The memory profile of the edited sequence (Eq. 4) is
// therefore the parent's profile, shifted around the edit, plus a handful of range corrections, and
// its peak is the maximum of the parent's prefix / suffix maxima outside the touched window and a
// recomputation inside it.
//
// Restricted to C <= 2 (the paper's setting, Section 4.3) and sequences shorter than 65535 steps.
//
// Cache of one parent (all in 0-based steps; S = row stride):
//   row[S16] the sequence                      fre[S16] free step of the copy run at each step
//            (both 16 bits per step, S16 = S rounded up to a multiple of 8 so that rows start on 16 bytes)
//   prof[S]  memory in use at each step        pm[S]    max prof[0..t]      sm[S]  max prof[t..T-1]
//   occ[n]   the two steps of every node, 1-based, 16 bits each (equal when the node runs once)
//   len, status, peak, dur
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "moc_pair_kernel.cuh"

namespace moc {

constexpr int kEditThreads = 256;   // 8 warps per block, one edit per warp at a time
constexpr int kPrepThreads = 768;   // cache build: up to 24 warps per block, one parent per warp at a time

struct EditCacheDev {
    int32_t n, C, P, stride, occ_stride;
    int32_t stride16;           // row stride of the 16-bit arrays row and fre
    int32_t max_T;              // C * n
    const int32_t* succ_start;  // successor and predecessor lists (CSR)
    const int32_t* succ;
    const int32_t* pred_start;
    const int32_t* pred;
    const int64_t* w;
    const int64_t* m;
    const int32_t* cap;         // per-node caps or nullptr
    int64_t sink_m;             // sum of m over the nodes without successors
    uint16_t* row;
    uint16_t* fre;
    void* prof;                 // MemT [P][stride]
    void* pm;
    void* sm;
    uint32_t* occ;              // [P][occ_stride]
    int32_t* len;
    int32_t* status;
    int64_t* peak;
    int64_t* dur;
};

struct PrepParams {
    EditCacheDev c;
    const int32_t* seqs;        // packed parents
    const int32_t* lens;
    const int64_t* offs;        // exclusive prefix sum of the lengths
    int64_t M;
    int64_t* out_peak;          // may be null
    int64_t* out_dur;
    int32_t* out_status;
    const int32_t* todo;        // may be null: indices of the parents to (re)build, todo_count of them
    const int32_t* todo_count;  // device counter read by the kernel
    uint32_t warp_bytes;
    // successor tiles of the warp-per-sequence evaluation kernel (moc_pair_kernel.cuh), read through L1;
    // n_tiles = 0: not available, the node pass walks the plain successor lists
    int32_t n_tiles;
    const void* rec;
    const uint64_t* wslot;
    const uint32_t* sell;
    int64_t base_dur;           // sum of all w
    // chip_bytes > 0: the block first copies the tiles into its shared memory (records, then durations at
    // chip_w_b, then successor entries at chip_sell_b; sell_len entries) and the warps' arrays follow
    uint32_t chip_bytes, chip_w_b, chip_sell_b;
    int32_t sell_len;
};

template <typename T>
__device__ __forceinline__ T edit_warp_incl_sum(T v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}
template <typename T>
__device__ __forceinline__ T edit_warp_incl_max_up(T v, int lane) {     // max over lanes <= lane
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v = o > v ? o : v;
    }
    return v;
}
template <typename T>
__device__ __forceinline__ T edit_warp_incl_max_down(T v, int lane) {   // max over lanes >= lane
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T o = __shfl_down_sync(0xFFFFFFFFu, v, d);
        if (lane + d < 32) v = o > v ? o : v;
    }
    return v;
}
template <typename T>
__device__ __forceinline__ T edit_warp_max(T v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const T o = __shfl_xor_sync(0xFFFFFFFFu, v, d);
        v = o > v ? o : v;
    }
    return v;
}
__device__ __forceinline__ void edit_add(int32_t* p, int32_t v) { atomicAdd(p, v); }
__device__ __forceinline__ void edit_add(int64_t* p, int64_t v) {
    atomicAdd(reinterpret_cast<unsigned long long*>(p), (unsigned long long)v);
}

// Words of the occurrence array of one warp in shared memory: the n nodes, the spare word n, the word n + 1
// (sequence length, for sinks) and, at the next multiple of four after n + 2, the constant word of empty node slots.
__host__ __device__ inline int32_t edit_word_stride(int32_t n) { return ((n + 2 + 3) & ~3) + 4; }

// Shared memory of one warp (cache build): occurrence words [edit_word_stride(n)] uint32, then two arrays of stride + 8 MemT.
__host__ __device__ inline size_t edit_warp_bytes(int32_t n, int32_t stride, size_t mem_sz) {
    return (size_t)edit_word_stride(n) * 4 + 2 * ((((size_t)stride + 8) * mem_sz + 15) & ~size_t(15));
}

// Full evaluation of every parent (same quantities as the evaluation kernels: Section 2, Eqs. 1-8)
// that also writes the cache.  One warp per parent.
template <typename MemT, bool kChip>
__global__ void __launch_bounds__(kPrepThreads) edit_prepare_kernel(const PrepParams p) {
    extern __shared__ __align__(16) char smem[];
    const EditCacheDev& c = p.c;
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    if (kChip) {
        // what the L1 keeps of the tiles between parents is little beside the warps' arrays: the block holds its own copy
        const uint32_t rec_v = (sizeof(MemT) == 4 ? 8u : 16u) * 64u * (uint32_t)p.n_tiles / 16u, w_v = 8u * 64u * (uint32_t)p.n_tiles / 16u;
        const uint32_t sell_v = ((uint32_t)p.sell_len * 4u + 15u) / 16u;
        const uint4* g_rec = reinterpret_cast<const uint4*>(p.rec);
        const uint4* g_w = reinterpret_cast<const uint4*>(p.wslot);
        const uint4* g_sell = reinterpret_cast<const uint4*>(p.sell);
        for (uint32_t i = threadIdx.x; i < rec_v; i += blockDim.x) reinterpret_cast<uint4*>(smem)[i] = __ldg(g_rec + i);
        for (uint32_t i = threadIdx.x; i < w_v; i += blockDim.x) reinterpret_cast<uint4*>(smem + p.chip_w_b)[i] = __ldg(g_w + i);
        for (uint32_t i = threadIdx.x; i < sell_v; i += blockDim.x) reinterpret_cast<uint4*>(smem + p.chip_sell_b)[i] = __ldg(g_sell + i);
        __syncthreads();
    }
    char* ws = smem + (kChip ? p.chip_bytes : 0u) + (size_t)warp * p.warp_bytes;
    uint32_t* word = reinterpret_cast<uint32_t*>(ws);
    const size_t arr_bytes = (((size_t)c.stride + 8) * sizeof(MemT) + 15) & ~size_t(15);
    const int32_t n = c.n, wstride = edit_word_stride(c.n);
    MemT* arrA = reinterpret_cast<MemT*>(ws + (size_t)wstride * 4);
    MemT* arrB = reinterpret_cast<MemT*>(ws + (size_t)wstride * 4 + arr_bytes);
    constexpr uint32_t kFull = 0xFFFFFFFFu;

    const int32_t count = p.todo != nullptr ? min(*p.todo_count, c.P) : c.P;
    // the parent after this one is looked up while this one is evaluated (index, then length and row offset)
    const int32_t it_step = gridDim.x * wpb;
    int32_t it = blockIdx.x * wpb + warp;
    int32_t b_nx = it < count ? (p.todo != nullptr ? p.todo[it] : it) : 0;
    int32_t T_nx = it < count ? p.lens[b_nx] : 0;
    int64_t off_nx = it < count ? p.offs[b_nx] : 0;
    for (; it < count; it += it_step) {
        const int32_t b = b_nx, T = T_nx;
        const int64_t off = off_nx;
        const bool more = it + it_step < count;
        b_nx = more ? (p.todo != nullptr ? p.todo[it + it_step] : it + it_step) : 0;
        bool got_nx = false;
        int64_t out_pk = -1, out_du = -1;
        int32_t out_st = -2;
        uint16_t* row = c.row + (int64_t)b * c.stride16;
        if (T >= n && T <= c.max_T) {
            for (int32_t i = lane; i < wstride / 4; i += 32) reinterpret_cast<uint4*>(word)[i] = make_uint4(0, 0, 0, 0);
            for (int32_t i = lane; i < (int32_t)arr_bytes / 16; i += 32) reinterpret_cast<uint4*>(arrA)[i] = make_uint4(0, 0, 0, 0);
            __syncwarp();
            // ---- occurrence words (1-based steps, 16 bits each) and the copy of the row
            const int32_t* src = p.seqs + off;
            auto put = [&](int32_t v, int32_t t) {
                row[t] = (uint16_t)v;
                const uint32_t slot = min((uint32_t)v, (uint32_t)n);      // ids outside [0, n) land in a spare word
                const uint32_t t1 = (uint32_t)t + 1u;
                const uint32_t old = atomicExch(&word[slot], t1 * 0x10001u);
                if (old) reinterpret_cast<uint16_t*>(&word[slot])[1] = (uint16_t)old;
            };
            for (int32_t t0 = lane; t0 < T; t0 += 256) {                  // eight loads in flight per lane
                int32_t v[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) v[k] = t0 + 32 * k < T ? __ldg(src + t0 + 32 * k) : 0;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (t0 + 32 * k < T) put(v[k], t0 + 32 * k);
            }
            __syncwarp();
            if (more) { T_nx = p.lens[b_nx]; off_nx = p.offs[b_nx]; got_nx = true; }
            // ---- per node: both copies a <= b, free steps from the successors' copies, profile deltas
            uint32_t vsum = 0;
            bool absent = false, dep = false, over = false;
            int64_t dur = 0;
            uint16_t* fre = c.fre + (int64_t)b * c.stride16;
            if (p.n_tiles > 0) {
                // The node pass of the evaluation kernel: lane l serves the nodes l (mod 32) in tiles of two
                // slots, successor rows of packed word offsets, two shifted packed reductions per successor
                // word (end of the last copy with the precedence test, end of the first copy).
                constexpr uint32_t kRecB = sizeof(MemT) == 4 ? 8u : 16u;
                const uint32_t wa = (uint32_t)__cvta_generic_to_shared(word);
                const char* prec = (kChip ? smem : reinterpret_cast<const char*>(p.rec)) + kRecB * lane;
                const uint64_t* pw = (kChip ? reinterpret_cast<const uint64_t*>(smem + p.chip_w_b) : p.wslot) + lane;
                const uint32_t* ps = (kChip ? reinterpret_cast<const uint32_t*>(smem + p.chip_sell_b) : p.sell) + lane;
                auto ld32 = [&](const uint32_t* q) -> uint32_t { return kChip ? lds_u32_nv((uint32_t)__cvta_generic_to_shared(q)) : __ldg(q); };
                auto ld64 = [&](const uint64_t* q) -> uint64_t { return kChip ? lds_u64((uint32_t)__cvta_generic_to_shared(q)) : __ldg(q); };
                uint32_t vmin = 0xFFFFFFFFu, depw = 0, capw = 0;
                uint64_t acc = 0;
                const uint32_t empty_off = 4u * (((uint32_t)n + 2u + 3u) & ~3u);   // where the records of empty slots point
                if (lane == 0) {
                    word[n + 1] = (uint32_t)T * 0x10001u;               // the made-up successor of sinks
                    word[empty_off >> 2] = 0x00010001u;
                }
                __syncwarp();
                for (int d = 0; d < p.n_tiles; ++d, prec += 64 * kRecB, pw += 64) {
                    uint32_t ab[2], naa[2], nbb[2], Ga[2], Gb[2], xoff[2];
                    MemT mm[2];
                    int rows = 0;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t x;
                        if constexpr (sizeof(MemT) == 4) {
                            const uint2 r = kChip ? lds_v2((uint32_t)__cvta_generic_to_shared(prec + 32 * kRecB * h))
                                                  : __ldg(reinterpret_cast<const uint2*>(prec + 32 * kRecB * h));
                            x = r.x;
                            mm[h] = (MemT)r.y;
                        } else {
                            const uint4 r = kChip ? lds_v4((uint32_t)__cvta_generic_to_shared(prec + 32 * kRecB * h))
                                                  : __ldg(reinterpret_cast<const uint4*>(prec + 32 * kRecB * h));
                            x = r.x;
                            mm[h] = (MemT)((uint64_t)r.z | ((uint64_t)r.w << 32));
                        }
                        if (h == 0) rows = (int)(x >> 16);
                        xoff[h] = x & 0xFFFFu;
                        const uint32_t own = lds_u32(wa + xoff[h]);
                        vmin = min(vmin, own);
                        const uint32_t sw = swap_halves(own);
                        const uint32_t mn = min_u16x2(own, sw), mx = max_u16x2(own, sw);
                        ab[h] = __byte_perm(mn, mx, 0x7610);
                        naa[h] = 0x00010000u - mn;
                        nbb[h] = 0x00010000u - mx;
                        Ga[h] = mx - mn;
                        Gb[h] = 0x00010000u - Ga[h];
                    }
                    rows = __shfl_sync(kFull, rows, 0);
                    uint32_t e_next = rows > 0 ? ld32(ps) : 0u;            // one row ahead
                    for (int k = 0; k < rows; ++k, ps += 32) {
                        const uint32_t e = e_next;
                        if (k + 1 < rows) e_next = ld32(ps + 32);
                        const uint32_t r0 = lds_u32(wa + (e & 0xFFFFu)), r1 = lds_u32(wa + (e >> 16));
                        Ga[0] = __viaddmax_u16x2(r0, naa[0], Ga[0]);
                        Ga[1] = __viaddmax_u16x2(r1, naa[1], Ga[1]);
                        Gb[0] = __viaddmax_u16x2(r0, nbb[0], Gb[0]);
                        Gb[1] = __viaddmax_u16x2(r1, nbb[1], Gb[1]);
                    }
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        depw |= Ga[h];
                        const uint32_t gg = max_u16x2(__byte_perm(Ga[h], Gb[h], 0x5410), __byte_perm(Ga[h], Gb[h], 0x7632));
                        const uint32_t v = gg + ab[h];                   // (end of b, end of a), 1-based
                        const uint32_t a16 = ab[h] & 0xFFFFu, b16 = ab[h] >> 16, fb = v & 0xFFFFu, fa = v >> 16;
                        const bool real = xoff[h] != empty_off;          // empty slots own the constant word: no step is theirs
                        if (real && b16 != 0) {
                            arrB[b16 - 1] = (MemT)fb - 1;                // free steps gather on chip, written out in order below
                            edit_add(&arrA[b16 - 1], mm[h]);
                            edit_add(&arrA[fb], (MemT)(-mm[h]));
                            if (a16 != b16) {
                                arrB[a16 - 1] = (MemT)fa - 1;
                                edit_add(&arrA[a16 - 1], mm[h]);
                                edit_add(&arrA[fa], (MemT)(-mm[h]));
                                const uint64_t wx = ld64(pw + 32 * h);
                                capw |= (uint32_t)(wx >> 32);
                                acc += wx;
                            }
                        }
                    }
                }
                vmin = __reduce_min_sync(kFull, vmin);
                int64_t accs = (int64_t)acc;
                for (int dd = 16; dd > 0; dd >>= 1) accs += __shfl_xor_sync(kFull, accs, dd);
                const uint64_t acc_all = (uint64_t)accs;
                absent = vmin == 0;
                over = __any_sync(kFull, (int32_t)capw < 0) || (int)((acc_all >> kPairCntShift) & 0x7FFFu) != T - n;
                dep = (depw & 0x80008000u) != 0;
                __syncwarp();
                for (int32_t t = 8 * lane; t < T; t += 256) {             // eight free steps per 16-byte store
                    uint32_t q[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) q[i] = ((uint32_t)arrB[t + 2 * i] & 0xFFFFu) | (uint32_t)arrB[t + 2 * i + 1] << 16;
                    *reinterpret_cast<uint4*>(fre + t) = make_uint4(q[0], q[1], q[2], q[3]);
                }
                // position sum and duration in the form the rest of the kernel expects
                vsum = lane == 0 ? (uint32_t)T * ((uint32_t)T + 1u) / 2u : 0u;
                dur = lane == 0 ? p.base_dur + (int64_t)(acc_all & kPairDurMask) : 0;
            } else
            for (int32_t u = lane; u < n; u += 32) {
                const uint32_t wd = word[u];
                const uint32_t lo = wd & 0xFFFFu, hi = wd >> 16;
                const uint32_t a = min(lo, hi), bp = max(lo, hi);        // 1-based
                absent |= a == 0;
                vsum += bp + (a != bp ? a : 0u);
                if (a != bp && (c.C < 2 || (c.cap != nullptr && __ldg(&c.cap[u]) < 2))) over = true;
                const int64_t wu = __ldg(&c.w[u]);
                dur += a != bp ? 2 * wu : wu;
                const int32_t e0 = __ldg(&c.succ_start[u]), e1 = __ldg(&c.succ_start[u + 1]);
                uint32_t fb = bp, fa = a;
                if (e0 == e1) fb = (uint32_t)T;                           // result of the computation
                for (int32_t k = e0; k < e1; ++k) {
                    const uint32_t r = word[__ldg(&c.succ[k])];
                    const uint32_t r1 = min(r & 0xFFFFu, r >> 16), r2 = max(r & 0xFFFFu, r >> 16);
                    if (r1 != 0 && r1 < a) dep = true;                     // consumer before the first copy (Eq. 5)
                    fb = max(fb, r2);
                    const uint32_t g = r2 < bp ? r2 : (r1 < bp ? r1 : 0u); // latest consumer copy before b
                    fa = max(fa, g);
                }
                if (a != 0) {
                    const MemT mu = (MemT)__ldg(&c.m[u]);
                    fre[bp - 1] = (uint16_t)(fb - 1);
                    edit_add(&arrA[bp - 1], mu);
                    edit_add(&arrA[fb], (MemT)(-mu));
                    if (a != bp) {
                        fre[a - 1] = (uint16_t)(fa - 1);
                        edit_add(&arrA[a - 1], mu);
                        edit_add(&arrA[fa], (MemT)(-mu));
                    }
                }
            }
            vsum = __reduce_add_sync(kFull, vsum);
            const bool well = !__any_sync(kFull, absent || over) && vsum == (uint32_t)T * ((uint32_t)T + 1u) / 2u;
            const bool viol = __any_sync(kFull, dep);
            for (int d = 16; d > 0; d >>= 1) dur += __shfl_xor_sync(kFull, dur, d);
            __syncwarp();
            if (well && viol) {
                out_st = -1;
                out_du = dur;
            } else if (well) {
                // ---- profile, prefix maxima, suffix maxima: lane owns a run of consecutive steps, a whole number
                // of 16-byte vectors long and an odd number of them (the lanes' vectors fall into different banks).
                // Steps T .. Tp - 1 pad the last vector: their deltas are 0 and the usage there is 0.
                constexpr int32_t VW = 16 / (int32_t)sizeof(MemT);
                const int32_t Tp = (T + VW - 1) & ~(VW - 1);
                const int32_t per = VW * ((((T + 31) / 32 + VW - 1) / VW) | 1);
                const int32_t t0 = min(Tp, lane * per), t1 = min(Tp, t0 + per);
                auto ldv = [](const MemT* a, MemT (&v)[VW]) { *reinterpret_cast<uint4*>(v) = *reinterpret_cast<const uint4*>(a); };
                auto stv = [](MemT* a, const MemT (&v)[VW]) { *reinterpret_cast<uint4*>(a) = *reinterpret_cast<const uint4*>(v); };
                // pass 1: sum and largest running sum of the run, both relative to its start
                MemT sum = 0, top = 0;
                for (int32_t t = t0; t < t1; t += VW) {
                    alignas(16) MemT v[VW];
                    ldv(arrA + t, v);
#pragma unroll
                    for (int i = 0; i < VW; ++i) { sum += v[i]; top = sum > top ? sum : top; }
                }
                MemT run = edit_warp_incl_sum(sum, lane) - sum;             // usage in front of the run
                top += run;                                                 // largest usage inside the run (0 for an empty one)
                MemT carry = edit_warp_incl_max_up(top, lane);
                const MemT peak = __shfl_sync(kFull, carry, 31);
                carry = __shfl_up_sync(kFull, carry, 1);
                if (lane == 0) carry = 0;
                // pass 2: usage and prefix maxima
                for (int32_t t = t0; t < t1; t += VW) {
                    alignas(16) MemT v[VW], w[VW];
                    ldv(arrA + t, v);
#pragma unroll
                    for (int i = 0; i < VW; ++i) {
                        run += v[i];
                        v[i] = run;
                        carry = run > carry ? run : carry;
                        w[i] = carry;
                    }
                    stv(arrA + t, v);                                       // prof
                    stv(arrB + t, w);                                       // pm
                }
                __syncwarp();
                uint4* g_prof = reinterpret_cast<uint4*>(reinterpret_cast<MemT*>(c.prof) + (int64_t)b * c.stride);
                uint4* g_pm = reinterpret_cast<uint4*>(reinterpret_cast<MemT*>(c.pm) + (int64_t)b * c.stride);
                uint4* g_sm = reinterpret_cast<uint4*>(reinterpret_cast<MemT*>(c.sm) + (int64_t)b * c.stride);
                for (int32_t i = lane; i < Tp / VW; i += 32) {
                    g_prof[i] = reinterpret_cast<const uint4*>(arrA)[i];
                    g_pm[i] = reinterpret_cast<const uint4*>(arrB)[i];
                }
                __syncwarp();
                // pass 3: suffix maxima
                MemT back = edit_warp_incl_max_down(top, lane);
                back = __shfl_down_sync(kFull, back, 1);
                if (lane == 31) back = 0;
                for (int32_t t = t1 - VW; t >= t0; t -= VW) {
                    alignas(16) MemT v[VW], w[VW];
                    ldv(arrA + t, v);
#pragma unroll
                    for (int i = VW - 1; i >= 0; --i) {
                        back = v[i] > back ? v[i] : back;
                        w[i] = back;
                    }
                    stv(arrB + t, w);                                       // sm
                }
                __syncwarp();
                for (int32_t i = lane; i < Tp / VW; i += 32) g_sm[i] = reinterpret_cast<const uint4*>(arrB)[i];
                uint4* g_occ = reinterpret_cast<uint4*>(c.occ + (int64_t)b * c.occ_stride);
                for (int32_t i = lane; i < c.occ_stride / 4; i += 32) g_occ[i] = reinterpret_cast<const uint4*>(word)[i];
                out_pk = (int64_t)peak;
                out_du = dur;
                out_st = out_pk <= p.M ? 1 : 0;
            }
            __syncwarp();
        }
        if (more && !got_nx) { T_nx = p.lens[b_nx]; off_nx = p.offs[b_nx]; }
        if (lane == 0) {
            c.len[b] = T;
            c.status[b] = out_st;
            c.peak[b] = out_pk;
            c.dur[b] = out_du;
            if (p.out_peak) p.out_peak[b] = out_pk;
            if (p.out_dur) p.out_dur[b] = out_du;
            if (p.out_status) p.out_status[b] = out_st;
        }
        __syncwarp();
    }
}

struct EditParams {
    EditCacheDev c;
    const int32_t* parent;      // B: index of the cached parent
    const int32_t* op;          // B: 0 insert, 1 delete, 2 move
    const int32_t* q;           // B: step of the parent the edit refers to
    const int32_t* j;           // B: insertion index (insert: 0..T, move: 0..T-1 in the shortened row)
    int32_t B;
    int64_t M;
    int64_t* out_peak;
    int64_t* out_dur;
    int32_t* out_status;
    int32_t* out_window;        // may be null: steps of the child whose usage was recomputed
    uint32_t warp_bytes;        // two arrays of stride + 4 MemT
};

constexpr int32_t kEditNone = 1 << 30;        // "no such step"
constexpr int32_t kStatusParentInvalid = -3;  // the parent itself has no valid evaluation

// One warp per edit.  Steps are 0-based here.  qd = deleted step of the parent (delete, move) or none,
// ji = inserted index of the child (insert, move) or none.  A parent step p != qd becomes child step
// map(p); a child step t != ji comes from parent step inv(t).
template <typename MemT>
__global__ void __launch_bounds__(kEditThreads) edit_eval_kernel(const EditParams p) {
    extern __shared__ __align__(16) char smem[];
    const EditCacheDev& c = p.c;
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const size_t arr_bytes = (((size_t)c.stride + 4) * sizeof(MemT) + 15) & ~size_t(15);
    MemT* win_d = reinterpret_cast<MemT*>(smem + (size_t)warp * p.warp_bytes);
    MemT* win_b = reinterpret_cast<MemT*>(smem + (size_t)warp * p.warp_bytes + arr_bytes);
    constexpr uint32_t kFull = 0xFFFFFFFFu;

    for (int32_t e = blockIdx.x * wpb + warp; e < p.B; e += gridDim.x * wpb) {
        int64_t out_pk = -1, out_du = -1;
        int32_t out_st = -2, out_win = 0;
        const int32_t ci = __ldg(&p.parent[e]), o = __ldg(&p.op[e]), qq = __ldg(&p.q[e]), jj = __ldg(&p.j[e]);
        bool go = ci >= 0 && ci < c.P;
        int32_t T = 0;
        if (go) {
            T = c.len[ci];
            if (c.status[ci] < 0) { out_st = kStatusParentInvalid; go = false; }
        }
        if (go) go = o >= 0 && o <= 2 && qq >= 0 && qq < T && (o == 1 || (jj >= 0 && jj <= (o == 0 ? T : T - 1)));
        if (go) {
            const uint16_t* row = c.row + (int64_t)ci * c.stride16;
            const uint16_t* fre = c.fre + (int64_t)ci * c.stride16;
            const MemT* prof = reinterpret_cast<const MemT*>(c.prof) + (int64_t)ci * c.stride;
            const MemT* pmx = reinterpret_cast<const MemT*>(c.pm) + (int64_t)ci * c.stride;
            const MemT* smx = reinterpret_cast<const MemT*>(c.sm) + (int64_t)ci * c.stride;
            const uint32_t* occ = c.occ + (int64_t)ci * c.occ_stride;
            const int32_t x = (int32_t)row[qq];
            const int32_t qd = o >= 1 ? qq : kEditNone, ji = o != 1 ? jj : kEditNone;
            const int32_t Tc = T + (o == 0 ? 1 : 0) - (o == 1 ? 1 : 0);
            auto map = [&](int32_t s) -> int32_t { const int32_t s1 = s - (s > qd ? 1 : 0); return s1 + (s1 >= ji ? 1 : 0); };
            auto inv = [&](int32_t t) -> int32_t { const int32_t t1 = t - (t > ji ? 1 : 0); return t1 + (t1 >= qd ? 1 : 0); };
            // copies of x in the parent and in the child
            const uint32_t wx = occ[x];
            const int32_t xa = (int32_t)min(wx & 0xFFFFu, wx >> 16) - 1, xb = (int32_t)max(wx & 0xFFFFu, wx >> 16) - 1;
            const int32_t cnt = xa == xb ? 1 : 2, cnt2 = cnt - (o >= 1 ? 1 : 0) + (o != 1 ? 1 : 0);
            int32_t cx0 = kEditNone, cx1 = kEditNone;     // child steps of x, ascending; cx1 = none when one copy
            {
                int32_t k0 = xa != qd ? map(xa) : kEditNone, k1 = (cnt == 2 && xb != qd) ? map(xb) : kEditNone;
                if (k0 == kEditNone) { k0 = k1; k1 = kEditNone; }
                if (ji != kEditNone) {
                    if (k0 == kEditNone) k0 = ji;
                    else if (ji < k0) { k1 = k0; k0 = ji; }
                    else k1 = ji;                               // cnt2 <= 2 is checked below
                }
                cx0 = k0; cx1 = k1;
            }
            const bool x_two_ok = c.C >= 2 && (c.cap == nullptr || __ldg(&c.cap[x]) >= 2);
            if (cnt2 >= 1 && cnt2 <= 2 && (cnt2 == 1 || x_two_ok)) {
                const int64_t wxv = __ldg(&c.w[x]);
                const int64_t du = c.dur[ci] + wxv * (cnt2 - cnt);
                // child steps of any node: (first, last)
                auto cpos = [&](int32_t v, int32_t& f0, int32_t& f1) {
                    if (v == x) { f0 = cx0; f1 = cx1 == kEditNone ? cx0 : cx1; return; }
                    const uint32_t wv = occ[v];
                    f0 = map((int32_t)min(wv & 0xFFFFu, wv >> 16) - 1);
                    f1 = map((int32_t)max(wv & 0xFFFFu, wv >> 16) - 1);
                };
                const int32_t ps0 = __ldg(&c.pred_start[x]), ps1 = __ldg(&c.pred_start[x + 1]);
                const int32_t ss0 = __ldg(&c.succ_start[x]), ss1 = __ldg(&c.succ_start[x + 1]);
                // ---- precedence (Eq. 5) can only break on edges that touch x
                bool viol = false;
                for (int32_t k = ps0 + lane; k < ps1; k += 32) {
                    int32_t f0, f1;
                    cpos(__ldg(&c.pred[k]), f0, f1);
                    viol |= f0 > cx0;
                }
                for (int32_t k = ss0 + lane; k < ss1; k += 32) {
                    int32_t f0, f1;
                    cpos(__ldg(&c.succ[k]), f0, f1);
                    viol |= f0 < cx0;
                }
                if (__any_sync(kFull, viol)) {
                    out_st = -1;
                    out_du = du;
                } else {
                    out_du = du;
                    // ---- cleared difference array over the child steps (only the window is read later)
                    for (int32_t i = lane; i < Tc + 2; i += 32) win_d[i] = 0;
                    __syncwarp();
                    const bool x_sink = ss0 == ss1;
                    int32_t lo_w = kEditNone, hi_w = -1;
                    auto emit = [&](int32_t l, int32_t h, MemT val) {       // += val on child steps l..h
                        if (l > h) return;
                        edit_add(&win_d[l], val);
                        edit_add(&win_d[h + 1], (MemT)(-val));
                        lo_w = min(lo_w, l);
                        hi_w = max(hi_w, h);
                    };
                    // ---- the affected nodes: x and its predecessors
                    const int32_t nA = 1 + (ps1 - ps0);
                    for (int32_t k = lane; k < nA; k += 32) {
                        const int32_t y = k == 0 ? x : __ldg(&c.pred[ps0 + k - 1]);
                        const MemT my = (MemT)__ldg(&c.m[y]);
                        const uint32_t wy = occ[y];
                        const int32_t ya = (int32_t)min(wy & 0xFFFFu, wy >> 16) - 1, yb = (int32_t)max(wy & 0xFFFFu, wy >> 16) - 1;
                        // new copies and their free steps
                        int32_t n0, n1;
                        cpos(y, n0, n1);
                        const bool two = n1 != n0;
                        int32_t f0 = n0, f1 = n1;
                        const int32_t s0 = __ldg(&c.succ_start[y]), s1 = __ldg(&c.succ_start[y + 1]);
                        for (int32_t z = s0; z < s1; ++z) {
                            int32_t r0, r1;
                            cpos(__ldg(&c.succ[z]), r0, r1);
                            if (two) {
                                if (r0 > n0 && r0 < n1) f0 = max(f0, r0);
                                if (r1 > n0 && r1 < n1) f0 = max(f0, r1);
                            }
                            f1 = max(f1, r1);          // every consumer copy lies behind the first copy here
                            if (!two) f0 = f1;
                        }
                        if (s0 == s1) { f1 = Tc - 1; if (!two) f0 = f1; }
                        // old copies in child steps
                        auto old_range = [&](int32_t ps, int32_t pf, bool to_end, int32_t& l, int32_t& h) {
                            l = ps == qd ? (pf > qd ? map(qd + 1) : kEditNone) : map(ps);
                            h = pf == qd ? (pf > ps ? map(pf - 1) : -1) : map(pf);
                            if (to_end && ps != qd) h = Tc - 1;
                        };
                        if (y == x) {
                            int32_t l, h;
                            old_range(xa, (int32_t)fre[xa], x_sink && cnt == 1, l, h);
                            emit(l, h, (MemT)(-my));
                            if (cnt == 2) {
                                old_range(xb, (int32_t)fre[xb], x_sink, l, h);
                                emit(l, h, (MemT)(-my));
                            }
                            emit(n0, f0, my);
                            if (two) emit(n1, f1, my);
                        } else {
                            int32_t l, h;
                            old_range(ya, (int32_t)fre[ya], false, l, h);
                            if (h != f0) emit(min(h, f0) + 1, max(h, f0), f0 > h ? my : (MemT)(-my));
                            if (yb != ya) {
                                old_range(yb, (int32_t)fre[yb], false, l, h);
                                if (h != f1) emit(min(h, f1) + 1, max(h, f1), f1 > h ? my : (MemT)(-my));
                            }
                        }
                    }
                    lo_w = __reduce_min_sync(kFull, lo_w);
                    hi_w = __reduce_max_sync(kFull, hi_w);
                    if (qd != kEditNone) {
                        // the parent's prefix / suffix maxima must not reach across the deleted step
                        const int32_t cl = qd > 0 ? map(qd - 1) : -1, cr = qd < T - 1 ? map(qd + 1) : Tc;
                        lo_w = min(lo_w, cl + 1);
                        hi_w = max(hi_w, cr - 1);
                    }
                    __syncwarp();
                    // ---- usage inside the window: parent's profile (or the usage carried across the
                    // inserted step) plus the corrections
                    const int32_t L = hi_w - lo_w + 1;
                    out_win = max(L, 0);
                    MemT cross = 0;
                    if (ji != kEditNone) {
                        if (ji + 1 < Tc) {
                            const int32_t tr = inv(ji + 1), tl = ji >= 1 ? inv(ji - 1) : -1;
                            cross = prof[tr] - (MemT)__ldg(&c.m[(int32_t)row[tr]]);
                            if (qd != kEditNone && qd > tl && qd < tr && (int32_t)fre[qd] >= tr) cross -= (MemT)__ldg(&c.m[x]);
                        } else {
                            cross = (MemT)c.sink_m;
                            if (x_sink && qd == xb) cross -= (MemT)__ldg(&c.m[x]);
                        }
                    }
                    for (int32_t i = lane; i < L; i += 32) {
                        const int32_t t = lo_w + i;
                        win_b[i] = t == ji ? cross : prof[inv(t)];
                    }
                    __syncwarp();
                    MemT best = 0;
                    if (L > 0) {
                        const int32_t per = (L + 31) / 32;
                        const int32_t i0 = min(L, lane * per), i1 = min(L, i0 + per);
                        MemT sum = 0;
                        for (int32_t i = i0; i < i1; ++i) sum += win_d[lo_w + i];
                        MemT run = edit_warp_incl_sum(sum, lane) - sum;
                        for (int32_t i = i0; i < i1; ++i) {
                            run += win_d[lo_w + i];
                            const MemT u = run + win_b[i];
                            best = u > best ? u : best;
                        }
                    }
                    if (lane == 0) {
                        if (lo_w > 0) { const MemT v = pmx[inv(lo_w - 1)]; best = v > best ? v : best; }
                        if (hi_w < Tc - 1) { const MemT v = smx[inv(hi_w + 1)]; best = v > best ? v : best; }
                    }
                    best = edit_warp_max(best);
                    out_pk = (int64_t)best;
                    out_st = out_pk <= p.M ? 1 : 0;
                    __syncwarp();
                }
            }
        }
        if (lane == 0) {
            p.out_peak[e] = out_pk;
            p.out_dur[e] = out_du;
            p.out_status[e] = out_st;
            if (p.out_window) p.out_window[e] = out_win;
        }
        __syncwarp();
    }
}

}  // namespace moc

// Device code of the local search over rematerialization sequences (paper: Section 3,
// "Optimization in Two Phases").  P independent chains each keep one sequence and its evaluation.
// A generation proposes one edited copy per chain, the evaluation kernels score all proposals as one
// batch, and a proposal replaces its chain's sequence when its key
//     ( max(peak, M), duration )
// is not larger: while a chain is over the budget M this lowers max(peak, M), the objective of the
// paper's Phase 1; once peak <= M the first component is M for everything that can be accepted and
// only the duration (Eq. 1) decides, which is Phase 2 with the memory constraint of Eq. 4.
//
// Layout.  Both the chains' sequences and the proposals live in one array `rows` of 2*P rows of
// `stride` ints (stride a multiple of 4, at least C*n): chain c owns rows c and P + c, and cur[c]
// says which of the two holds its sequence; the proposal is written to the other one.  Accepting a
// proposal flips cur[c]; no row is ever copied.  The evaluation kernels read the proposals through an
// array of row offsets that the proposing kernel writes.
//
// Random draws: one block of Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC 2011) per chain and
// generation with counter (generation, chain0 + chain, 0, 0) and the 64-bit seed as the key; chain0
// numbers the chains globally when a population is split over several devices.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace moc {

// Ten rounds of the 4x32 variant: the products of two counter words with the two multipliers are
// crossed with the other words and the round key, which advances by the two Weyl constants.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
    constexpr uint32_t kMul0 = 0xD2511F53u, kMul1 = 0xCD9E8D57u;
    constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(kMul0, c.x), lo0 = kMul0 * c.x;
        const uint32_t hi1 = __umulhi(kMul1, c.z), lo1 = kMul1 * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += kWeyl0;
        k.y += kWeyl1;
    }
    return c;
}

struct SearchParams {
    int32_t P;
    int32_t stride;      // ints per row, multiple of 4
    int32_t max_T;       // C * n: longest sequence the evaluator admits
    int64_t M;
    uint32_t seed_lo, seed_hi;
    uint32_t generation; // of the proposals written by this launch
    uint32_t chain0;     // global number of chain 0 (enters the random draws only)
    uint32_t kinds;      // enabled kinds of edit: bit 0 insert, bit 1 delete, bit 2 move (never 0)
    int32_t* rows;       // 2 * P * stride
    int32_t* cur;        // P: 0 or 1
    int32_t* lens;       // P: length of each chain's sequence
    int64_t* peak;       // P: evaluation of each chain's sequence
    int64_t* dur;
    int32_t* status;
    int32_t* n_acc;      // P: proposals accepted so far
    // proposals
    int32_t* c_lens;     // P
    int64_t* c_offs;     // P + 1: offset of each proposal's row in `rows`; c_offs[P] = 2*P*stride
    int64_t* c_peak;     // P: written by the evaluation kernels
    int64_t* c_dur;
    int32_t* c_status;
};

// Order of two evaluated sequences under the key (max(peak, M), duration); status < 0 ranks last.
__device__ __forceinline__ bool search_not_worse(int64_t pk_c, int64_t du_c, int32_t st_c, int64_t pk_p,
                                                 int64_t du_p, int32_t st_p, int64_t M) {
    if (st_c < 0) return false;
    if (st_p < 0) return true;
    const int64_t a = pk_c > M ? pk_c : M, b = pk_p > M ? pk_p : M;
    return a < b || (a == b && du_c <= du_p);
}

constexpr int kSearchThreads = 256;  // 8 chains per block, one warp each

// The (r0 mod k)-th enabled kind of edit, k = number of enabled kinds (order: insert, delete, move).
__device__ __forceinline__ uint32_t search_pick_kind(uint32_t kinds, uint32_t r0) {
    uint32_t pick = r0 % (uint32_t)__popc(kinds), op = 0;
    for (uint32_t o = 0; o < 3; ++o) {
        if (kinds >> o & 1u) {
            if (pick == 0) { op = o; break; }
            --pick;
        }
    }
    return op;
}

// Writes the edited copy of src[0..T) to dst with the lanes of one warp: element qd taken out (none:
// INT32_MAX), then x put in front of index j of what is left (none: INT32_MAX); Tc elements result.
// 16-byte stores, sources through the read-only path.
__device__ __forceinline__ void search_write_edited(const int32_t* __restrict__ src, int32_t* __restrict__ dst,
                                                    int32_t Tc, int32_t qd, int32_t j, int32_t x, int lane) {
    auto at = [&](int32_t i) -> int32_t {
        if (i == j) return x;
        const int32_t k = i - (i > j ? 1 : 0);       // index in the row without element qd
        return __ldg(src + k + (k >= qd ? 1 : 0));
    };
    for (int32_t i0 = 4 * lane; i0 < Tc; i0 += 128) {
        if (i0 + 4 <= Tc) {
            int4 v;
            v.x = at(i0); v.y = at(i0 + 1); v.z = at(i0 + 2); v.w = at(i0 + 3);
            *reinterpret_cast<int4*>(dst + i0) = v;
        } else {
            for (int32_t i = i0; i < Tc; ++i) dst[i] = at(i);
        }
    }
}

// One warp per chain.  kSelect: settle the pending proposal of the chain (written by the previous
// launch, scored since).  kPropose: write the next proposal.
//   op = the (r0 mod k)-th of the k enabled kinds in the order insert (0), delete (1), move (2); r0 mod 3
//   when all are enabled; q = r1 mod T the copy the edit refers to,
//   insert: the node seq[q] goes in front of index j = r2 mod (T+1);
//   delete: element q is removed;
//   move:   element q is removed and re-inserted in front of index j = r2 mod T of the shortened row.
// A proposal longer than max_T is only announced by its length (the evaluator refuses it unread); a
// chain of length 0 proposes length 0, which the evaluator refuses as well.
template <bool kSelect, bool kPropose>
__global__ void __launch_bounds__(kSearchThreads) search_step_kernel(const SearchParams p) {
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * (kSearchThreads / 32) + (threadIdx.x >> 5);
    if (c >= p.P) return;
    int32_t cur = p.cur[c], T = p.lens[c];
    if (kSelect) {
        const int64_t pk = p.c_peak[c], du = p.c_dur[c];
        const int32_t st = p.c_status[c];
        if (search_not_worse(pk, du, st, p.peak[c], p.dur[c], p.status[c], p.M)) {
            cur ^= 1;
            T = p.c_lens[c];
            __syncwarp();   // every lane has read the old evaluation before lane 0 replaces it
            if (lane == 0) {
                p.cur[c] = cur;
                p.lens[c] = T;
                p.peak[c] = pk;
                p.dur[c] = du;
                p.status[c] = st;
                p.n_acc[c] += 1;
            }
        }
    }
    if (!kPropose) return;
    const int64_t src_off = ((int64_t)cur * p.P + c) * p.stride;
    const int64_t dst_off = ((int64_t)(cur ^ 1) * p.P + c) * p.stride;
    if (lane == 0) {
        p.c_offs[c] = dst_off;
        if (c == 0) p.c_offs[p.P] = (int64_t)2 * p.P * p.stride;
    }
    if (T <= 0) {
        if (lane == 0) p.c_lens[c] = 0;
        return;
    }
    const uint4 r = philox4x32_10(make_uint4(p.generation, p.chain0 + (uint32_t)c, 0u, 0u), make_uint2(p.seed_lo, p.seed_hi));
    const uint32_t op = search_pick_kind(p.kinds, r.x);
    const int32_t q = (int32_t)(r.y % (uint32_t)T);
    // The proposal is "take element q out (delete, move), then put x in front of index j (insert,
    // move)"; qd / j beyond every index switch a half off.
    int32_t qd, j, Tc;
    if (op == 0) { qd = INT32_MAX; j = (int32_t)(r.z % ((uint32_t)T + 1u)); Tc = T + 1; }
    else if (op == 1) { qd = q; j = INT32_MAX; Tc = T - 1; }
    else { qd = q; j = (int32_t)(r.z % (uint32_t)T); Tc = T; }
    if (lane == 0) p.c_lens[c] = Tc;
    if (Tc > p.max_T) return;
    const int32_t* __restrict__ src = p.rows + src_off;
    int32_t* __restrict__ dst = p.rows + dst_off;
    const int32_t x = __ldg(src + q);
    search_write_edited(src, dst, Tc, qd, j, x, lane);
}

// ---- search on the incremental evaluation: E proposals per chain and generation are drawn as edit
// records, scored from the cached evaluation of the chain's sequence, and only the winner of a chain
// is ever written out.
struct SearchIncParams {
    SearchParams s;
    int32_t samples;        // E
    int32_t* e_parent;      // P * E edit records: chain, kind, step, insertion index
    int32_t* e_op;
    int32_t* e_q;
    int32_t* e_j;
    int64_t* r_peak;        // P * E results of the incremental evaluation
    int64_t* r_dur;
    int32_t* r_status;
    int64_t* row_offs;      // P + 1: offset of every chain's current row in `rows` (input of the cache build)
    int32_t* todo;          // P: chains whose sequence changed in this generation
    int32_t* todo_count;
};

// One thread per proposal: proposal e of chain c draws Philox4x32-10 with counter (generation, chain0 + c, e, 0).
__global__ void __launch_bounds__(256) search_draw_kernel(const SearchIncParams p) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t == 0) *p.todo_count = 0;
    if (t >= (int64_t)p.s.P * p.samples) return;
    const int32_t c = (int32_t)(t / p.samples), e = (int32_t)(t % p.samples);
    const int32_t T = p.s.lens[c];
    const uint4 r = philox4x32_10(make_uint4(p.s.generation, p.s.chain0 + (uint32_t)c, (uint32_t)e, 0u),
                                  make_uint2(p.s.seed_lo, p.s.seed_hi));
    const uint32_t op = search_pick_kind(p.s.kinds, r.x);
    const uint32_t Tu = (uint32_t)max(T, 1);
    p.e_parent[t] = c;
    p.e_op[t] = (int32_t)op;
    p.e_q[t] = (int32_t)(r.y % Tu);
    p.e_j[t] = op == 0 ? (int32_t)(r.z % (Tu + 1u)) : (int32_t)(r.z % Tu);
}

// One warp per chain: the best proposal of the chain (smallest key among status >= 0, lowest sample
// among equals) replaces the chain's sequence when it is not worse; its row is written to the chain's
// other row, and the chain is listed for the rebuild of its cache entry.
__global__ void __launch_bounds__(kSearchThreads) search_pick_kernel(const SearchIncParams p) {
    const SearchParams& s = p.s;
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * (kSearchThreads / 32) + (threadIdx.x >> 5);
    if (c >= s.P) return;
    constexpr uint32_t kFull = 0xFFFFFFFFu;
    const int64_t kInf = INT64_MAX;
    int64_t a = kInf, d = kInf;
    int32_t be = INT32_MAX;
    for (int32_t e = lane; e < p.samples; e += 32) {          // ascending e: ties keep the lowest sample
        const int64_t i = (int64_t)c * p.samples + e;
        if (p.r_status[i] < 0) continue;
        const int64_t pk = p.r_peak[i], ca = pk > s.M ? pk : s.M, cd = p.r_dur[i];
        if (ca < a || (ca == a && cd < d)) { a = ca; d = cd; be = e; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const int64_t a2 = __shfl_xor_sync(kFull, a, o), d2 = __shfl_xor_sync(kFull, d, o);
        const int32_t e2 = __shfl_xor_sync(kFull, be, o);
        if (a2 < a || (a2 == a && (d2 < d || (d2 == d && e2 < be)))) { a = a2; d = d2; be = e2; }
    }
    if (be == INT32_MAX) return;                                // no valid proposal
    const int64_t i = (int64_t)c * p.samples + be;
    const int64_t pk = p.r_peak[i], du = p.r_dur[i];
    const int32_t st = p.r_status[i];
    if (!search_not_worse(pk, du, st, s.peak[c], s.dur[c], s.status[c], s.M)) return;
    const int32_t cur = s.cur[c], T = s.lens[c];
    const int32_t op = p.e_op[i], q = p.e_q[i], j = p.e_j[i];
    const int32_t qd = op >= 1 ? q : INT32_MAX, ji = op != 1 ? j : INT32_MAX;
    const int32_t Tc = T + (op == 0 ? 1 : 0) - (op == 1 ? 1 : 0);
    const int64_t src_off = ((int64_t)cur * s.P + c) * s.stride, dst_off = ((int64_t)(cur ^ 1) * s.P + c) * s.stride;
    const int32_t x = __ldg(s.rows + src_off + q);
    search_write_edited(s.rows + src_off, s.rows + dst_off, Tc, qd, ji, x, lane);
    __syncwarp();
    if (lane == 0) {
        s.cur[c] = cur ^ 1;
        s.lens[c] = Tc;
        s.peak[c] = pk;
        s.dur[c] = du;
        s.status[c] = st;
        s.n_acc[c] += 1;
        p.row_offs[c] = dst_off;
        p.todo[atomicAdd(p.todo_count, 1)] = c;
    }
}

// Offsets of the chains' current rows, for the build of the whole cache.
__global__ void search_row_offsets_kernel(const SearchIncParams p) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < p.s.P) p.row_offs[c] = ((int64_t)p.s.cur[c] * p.s.P + c) * p.s.stride;
    if (c == 0) p.row_offs[p.s.P] = (int64_t)2 * p.s.P * p.s.stride;
}

// Start of a search: packed sequences (offs = exclusive prefix sum of the lengths) become rows
// 0..P-1; every chain starts in row set 0 with no accepted proposal.  A length outside [0, C*n]
// sets *bad_len (and is clamped, so that nothing is written outside a row).  One warp per chain.
__global__ void __launch_bounds__(kSearchThreads) search_init_kernel(const SearchParams p, const int32_t* __restrict__ seqs,
                                                                     const int32_t* __restrict__ in_lens,
                                                                     const int64_t* __restrict__ offs,
                                                                     int32_t* __restrict__ bad_len) {
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * (kSearchThreads / 32) + (threadIdx.x >> 5);
    if (c >= p.P) return;
    if (lane == 0 && (in_lens[c] < 0 || in_lens[c] > p.max_T)) atomicExch(bad_len, 1);   // reported by the host
    const int32_t T = min(max(in_lens[c], 0), p.max_T);
    const int32_t* src = seqs + offs[c];
    int32_t* dst = p.rows + (int64_t)c * p.stride;
    for (int32_t i = lane; i < T; i += 32) dst[i] = __ldg(src + i);
    if (lane == 0) {
        p.cur[c] = 0;
        p.lens[c] = T;
        p.n_acc[c] = 0;
    }
}

// Row offsets of the chains' current sequences (used to score the initial population).
__global__ void search_offsets_kernel(const SearchParams p) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < p.P) p.c_offs[c] = ((int64_t)p.cur[c] * p.P + c) * p.stride;
    if (c == 0) p.c_offs[p.P] = (int64_t)2 * p.P * p.stride;
}

// Copies every chain's current sequence to out_rows (P rows of `stride` ints; only the first
// lens[c] entries of a row are written).  One warp per chain.
__global__ void __launch_bounds__(kSearchThreads) search_export_kernel(const SearchParams p, int32_t* __restrict__ out_rows) {
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * (kSearchThreads / 32) + (threadIdx.x >> 5);
    if (c >= p.P) return;
    const int32_t T = p.lens[c];
    const int32_t* src = p.rows + ((int64_t)p.cur[c] * p.P + c) * p.stride;
    int32_t* dst = out_rows + (int64_t)c * p.stride;
    for (int32_t i = lane; i < T; i += 32) dst[i] = src[i];
}

// Best chain: smallest key (max(peak, M), duration) among the chains with status >= 0, lowest
// index among equals.  One block.  out_best: index (-1: no valid chain), length, peak, duration,
// status, total number of accepted proposals; out_seq (may be null) receives the sequence.
constexpr int kBestThreads = 1024;
__global__ void __launch_bounds__(kBestThreads) search_best_kernel(const SearchParams p, int32_t* __restrict__ out_seq,
                                                                   int64_t* __restrict__ out_best) {
    __shared__ int64_t s_a[kBestThreads / 32], s_d[kBestThreads / 32], s_acc[kBestThreads / 32];
    __shared__ int32_t s_i[kBestThreads / 32];
    __shared__ int32_t s_best;
    const int64_t kInf = INT64_MAX;
    int64_t a = kInf, d = kInf, acc = 0;
    int32_t idx = INT32_MAX;
    for (int c = threadIdx.x; c < p.P; c += kBestThreads) {   // ascending c: ties keep the lowest index
        acc += p.n_acc[c];
        if (p.status[c] < 0) continue;
        const int64_t pk = p.peak[c], ca = pk > p.M ? pk : p.M, cd = p.dur[c];
        if (ca < a || (ca == a && cd < d)) { a = ca; d = cd; idx = c; }
    }
    auto better = [](int64_t a1, int64_t d1, int32_t i1, int64_t a2, int64_t d2, int32_t i2) {
        return a1 < a2 || (a1 == a2 && (d1 < d2 || (d1 == d2 && i1 < i2)));
    };
    for (int o = 16; o > 0; o >>= 1) {
        const int64_t a2 = __shfl_xor_sync(0xFFFFFFFFu, a, o), d2 = __shfl_xor_sync(0xFFFFFFFFu, d, o);
        const int32_t i2 = __shfl_xor_sync(0xFFFFFFFFu, idx, o);
        acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (better(a2, d2, i2, a, d, idx)) { a = a2; d = d2; idx = i2; }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { s_a[warp] = a; s_d[warp] = d; s_i[warp] = idx; s_acc[warp] = acc; }
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t tot = 0;
        for (int k = 0; k < kBestThreads / 32; ++k) {
            tot += s_acc[k];
            if (better(s_a[k], s_d[k], s_i[k], a, d, idx)) { a = s_a[k]; d = s_d[k]; idx = s_i[k]; }
        }
        const bool any = idx != INT32_MAX;
        s_best = any ? idx : -1;
        out_best[0] = any ? idx : -1;
        out_best[1] = any ? p.lens[idx] : 0;
        out_best[2] = any ? p.peak[idx] : -1;
        out_best[3] = any ? p.dur[idx] : -1;
        out_best[4] = any ? p.status[idx] : -2;
        out_best[5] = tot;
    }
    __syncthreads();
    const int32_t b = s_best;
    if (b < 0 || out_seq == nullptr) return;
    const int32_t* src = p.rows + ((int64_t)p.cur[b] * p.P + b) * p.stride;
    for (int32_t i = threadIdx.x; i < p.lens[b]; i += kBestThreads) out_seq[i] = src[i];
}

}  // namespace moc

// One generation of the search on the cached evaluation in one kernel (paper: Section 3, the two-phase
// local search; Section 2, Eqs. 1-5 for what a proposal's score is).  A warp owns a chain: it brings the
// chain's cached copy positions, free steps, sequence and memory profile into shared memory once, draws the
// chain's E proposals with one lane each, scores them from the staged copy (edit_pass, moc_edit_pass.cuh) and
// settles the chain: the best proposal replaces the sequence when its key is not larger, and the chain is then
// listed for the rebuild of its cache entry.  Same draws, same scores and same choice as the three kernels
// search_draw_kernel, edit_eval_kernel and search_pick_kernel, which remain the general path.
#pragma once
#include "moc_edit_pass.cuh"
#include "moc_search_kernels.cuh"

namespace moc {

constexpr int kScoreThreads = 512;

struct ScoreParams {
    SearchParams s;
    EditCacheDev c;
    int32_t samples;        // E
    int64_t* row_offs;      // P + 1: offset of every chain's current row (input of the cache rebuild)
    int32_t* todo;          // P: chains whose sequence changed in this generation
    int32_t* todo_count;    // two counters: [generation & 1] collects this generation's chains, the other is cleared
    uint32_t graph_bytes;   // shared memory of the block's copy of the graph (kGraphOnChip), a multiple of 16
    uint32_t gs_pred_b, gs_m_b, gs_succ_b, gs_predl_b;   // its parts after the successor offsets
    uint32_t warp_bytes;    // shared memory of one warp
    uint32_t fre_b, row_b, prof_b, lh_b, val_b, diff_b;   // byte offsets of its parts (copy positions come first)
    int32_t list_cap;
};

// Bytes of one warp: copy positions (occ_stride words), free steps and the sequence (16 bits each), profile,
// range list, difference array of the corrections (stride + 4 entries).
__host__ __device__ inline size_t score_warp_bytes(int32_t occ_stride, int32_t stride, size_t mem_sz, int32_t list_cap,
                                                   uint32_t* fre_b, uint32_t* row_b, uint32_t* prof_b, uint32_t* lh_b,
                                                   uint32_t* val_b, uint32_t* diff_b) {
    size_t o = (size_t)occ_stride * 4;
    *fre_b = (uint32_t)o;
    o += ((size_t)stride * 2 + 15) & ~size_t(15);          // = 2 * stride16
    *row_b = (uint32_t)o;
    o += ((size_t)stride * 2 + 15) & ~size_t(15);
    *prof_b = (uint32_t)o;
    o += ((size_t)stride * mem_sz + 15) & ~size_t(15);
    *val_b = (uint32_t)o;
    o += ((size_t)list_cap * mem_sz + 15) & ~size_t(15);
    *lh_b = (uint32_t)o;
    o += ((size_t)list_cap * 4 + 15) & ~size_t(15);
    *diff_b = (uint32_t)o;
    o += (((size_t)stride + 4) * mem_sz + 15) & ~size_t(15);
    return o;
}

// 16 bytes from global to shared memory without a register in between (completed by cp.async.wait_all).
__device__ __forceinline__ void score_copy16(void* dst_shared, const void* src_global) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_shared)), "l"(src_global) : "memory");
}

// The lane's parent for edit_pass: the warp's staged copy (every lane has the same parent); prefix and suffix maxima
// are read from the cache in global memory (two values per admissible edit).
template <typename MemT>
struct ScoreParent {
    const uint32_t* occ_;
    const uint16_t* fre_;
    const uint16_t* row_;
    const MemT* prof_;
    const MemT* pm_;
    const MemT* sm_;
    struct View {
        const MemT* p;
        __device__ __forceinline__ MemT operator()(int32_t s) const { return p[s]; }
    };
    __device__ __forceinline__ uint32_t occ(int32_t v) const { return occ_[v]; }
    __device__ __forceinline__ int32_t fre(int32_t s) const { return (int32_t)fre_[s]; }
    __device__ __forceinline__ int32_t row(int32_t s) const { return (int32_t)row_[s]; }
    __device__ __forceinline__ MemT prof(int32_t s) const { return prof_[s]; }
    __device__ __forceinline__ MemT pm(int32_t s) const { return pm_[s]; }
    __device__ __forceinline__ MemT sm(int32_t s) const { return sm_[s]; }
    __device__ __forceinline__ View prof_view(int) const { return View{prof_}; }
};

// kGraphOnChip: the block keeps the graph's lists and output sizes in shared memory (every lane walks them
// at its own node, and what the warps' arrays leave of the L1 is too small to hold them).
template <typename MemT, bool kGraphOnChip>
__global__ void __launch_bounds__(kScoreThreads, 1) search_score_kernel(const ScoreParams p) {
    extern __shared__ __align__(16) char smem[];
    const EditCacheDev& c = p.c;
    const SearchParams& s = p.s;
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    if (kGraphOnChip) score_stage_graph<MemT>(c, smem, p.gs_pred_b, p.gs_m_b, p.gs_succ_b, p.gs_predl_b);
    const ScoreGraph<MemT, kGraphOnChip> graph{reinterpret_cast<const uint32_t*>(smem), reinterpret_cast<const uint32_t*>(smem + p.gs_pred_b),
                                               reinterpret_cast<const MemT*>(smem + p.gs_m_b), reinterpret_cast<const uint16_t*>(smem + p.gs_succ_b),
                                               reinterpret_cast<const uint16_t*>(smem + p.gs_predl_b), &c};
    char* mine = smem + (kGraphOnChip ? p.graph_bytes : 0u) + (size_t)warp * p.warp_bytes;
    uint32_t* occ = reinterpret_cast<uint32_t*>(mine);
    uint16_t* fre = reinterpret_cast<uint16_t*>(mine + p.fre_b);
    uint16_t* row = reinterpret_cast<uint16_t*>(mine + p.row_b);
    MemT* prof = reinterpret_cast<MemT*>(mine + p.prof_b);
    MemT* rv = reinterpret_cast<MemT*>(mine + p.val_b);
    uint32_t* rl = reinterpret_cast<uint32_t*>(mine + p.lh_b);
    MemT* diff = reinterpret_cast<MemT*>(mine + p.diff_b);
    for (int32_t i = lane; i < c.stride + 4; i += 32) diff[i] = 0;
    constexpr uint32_t kFull = 0xFFFFFFFFu;
    constexpr int64_t kInf = INT64_MAX;
    if (blockIdx.x == 0 && threadIdx.x == 0) p.todo_count[(s.generation + 1u) & 1u] = 0;
    int32_t* const counter = p.todo_count + (s.generation & 1u);

    for (int32_t ci = blockIdx.x * wpb + warp; ci < s.P; ci += gridDim.x * wpb) {
        const int32_t T = c.len[ci], pst = c.status[ci];
        const int64_t pdur = c.dur[ci];
        const MemT* g_pm = reinterpret_cast<const MemT*>(c.pm) + (int64_t)ci * c.stride;
        const MemT* g_sm = reinterpret_cast<const MemT*>(c.sm) + (int64_t)ci * c.stride;
        // ---- stage the chain's cache entry (copy positions, profile, free steps, sequence): asynchronous
        // 16-byte copies, all in flight at once
        {
            const uint4* g_occ = reinterpret_cast<const uint4*>(c.occ + (int64_t)ci * c.occ_stride);
            for (int32_t i = lane; i < c.occ_stride / 4; i += 32) score_copy16(reinterpret_cast<uint4*>(occ) + i, g_occ + i);
            const uint4* g_prof = reinterpret_cast<const uint4*>(reinterpret_cast<const MemT*>(c.prof) + (int64_t)ci * c.stride);
            constexpr int32_t kPer = 16 / (int32_t)sizeof(MemT);
            for (int32_t i = lane; i < (T + kPer - 1) / kPer; i += 32) score_copy16(reinterpret_cast<uint4*>(prof) + i, g_prof + i);
            const uint4* g_fre = reinterpret_cast<const uint4*>(c.fre + (int64_t)ci * c.stride16);
            const uint4* g_row = reinterpret_cast<const uint4*>(c.row + (int64_t)ci * c.stride16);
            for (int32_t i = lane; i < (T + 7) / 8; i += 32) {
                score_copy16(reinterpret_cast<uint4*>(fre) + i, g_fre + i);
                score_copy16(reinterpret_cast<uint4*>(row) + i, g_row + i);
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
        }
        __syncwarp();

        const ScoreParent<MemT> parent{occ, fre, row, prof, g_pm, g_sm};
        // best proposal of this lane over the passes: key (a, d), sample number, result, edit
        int64_t b_a = kInf, b_d = kInf, b_pk = -1;
        int32_t b_e = INT32_MAX, b_st = -2, b_op = 0, b_q = 0, b_j = 0;

        for (int32_t e0 = 0; e0 < p.samples; e0 += 32) {
            const int32_t e = e0 + lane;
            const bool live = e < p.samples;
            const uint4 r = philox4x32_10(make_uint4(s.generation, s.chain0 + (uint32_t)ci, (uint32_t)e, 0u),
                                          make_uint2(s.seed_lo, s.seed_hi));
            const int32_t o = (int32_t)search_pick_kind(s.kinds, r.x);
            const uint32_t Tu = (uint32_t)max(T, 1);
            const int32_t qq = (int32_t)(r.y % Tu);
            const int32_t jj = o == 0 ? (int32_t)(r.z % (Tu + 1u)) : (int32_t)(r.z % Tu);
            int64_t out_pk, out_du;
            int32_t out_st, out_win;
            edit_pass<MemT>(parent, graph, c, s.M, lane, live, pst, T, pdur, o, qq, jj, rl, rv, diff, p.list_cap, out_pk, out_du,
                            out_st, out_win);
            // ---- this lane's best so far (ascending sample numbers: ties keep the lowest)
            if (live && out_st >= 0) {
                const int64_t ca = out_pk > s.M ? out_pk : s.M;
                if (ca < b_a || (ca == b_a && out_du < b_d)) {
                    b_a = ca; b_d = out_du; b_e = e; b_pk = out_pk; b_st = out_st; b_op = o; b_q = qq; b_j = jj;
                }
            }
        }

        // ---- the chain's best proposal, and whether it replaces the sequence
        // smallest key (a, d) among the lanes that hold a proposal, lowest sample among equals; a, d >= 0
        auto min64 = [&](int64_t v, bool in) -> int64_t {
            const uint32_t hi = in ? (uint32_t)((uint64_t)v >> 32) : 0xFFFFFFFFu, hmin = __reduce_min_sync(kFull, hi);
            const uint32_t lo = (in && hi == hmin) ? (uint32_t)v : 0xFFFFFFFFu, lmin = __reduce_min_sync(kFull, lo);
            return (int64_t)((uint64_t)hmin << 32 | lmin);
        };
        const bool has = b_e != INT32_MAX;
        const int64_t a_min = min64(b_a, has);
        const bool has_a = has && b_a == a_min;
        const int64_t d_min = min64(b_d, has_a);
        const int32_t be = (int32_t)__reduce_min_sync(kFull, (has_a && b_d == d_min) ? (uint32_t)b_e : (uint32_t)INT32_MAX);
        if (be != INT32_MAX) {
            const int src = be & 31;
            const int64_t pk = __shfl_sync(kFull, b_pk, src), du = __shfl_sync(kFull, b_d, src);
            const int32_t st = __shfl_sync(kFull, b_st, src), op = __shfl_sync(kFull, b_op, src);
            const int32_t q = __shfl_sync(kFull, b_q, src), j = __shfl_sync(kFull, b_j, src);
            if (search_not_worse(pk, du, st, s.peak[ci], s.dur[ci], s.status[ci], s.M)) {
                const int32_t cur = s.cur[ci];
                const int32_t qd = op >= 1 ? q : INT32_MAX, ji = op != 1 ? j : INT32_MAX;
                const int32_t Tc = T + (op == 0 ? 1 : 0) - (op == 1 ? 1 : 0);
                const int64_t dst_off = ((int64_t)(cur ^ 1) * s.P + ci) * s.stride;
                // the edited copy of the staged sequence: element qd out, x in front of index ji of what is left
                const int32_t x = (int32_t)row[q];
                int32_t* dst = s.rows + dst_off;
                auto at = [&](int32_t i) -> int32_t {
                    if (i == ji) return x;
                    const int32_t k = i - (i > ji ? 1 : 0);
                    return (int32_t)row[k + (k >= qd ? 1 : 0)];
                };
                for (int32_t i0 = 4 * lane; i0 < Tc; i0 += 128) {
                    if (i0 + 4 <= Tc) {
                        *reinterpret_cast<int4*>(dst + i0) = make_int4(at(i0), at(i0 + 1), at(i0 + 2), at(i0 + 3));
                    } else {
                        for (int32_t i = i0; i < Tc; ++i) dst[i] = at(i);
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    s.cur[ci] = cur ^ 1;
                    s.lens[ci] = Tc;
                    s.peak[ci] = pk;
                    s.dur[ci] = du;
                    s.status[ci] = st;
                    s.n_acc[ci] += 1;
                    p.row_offs[ci] = dst_off;
                    p.todo[atomicAdd(counter, 1)] = ci;
                }
            }
        }
        __syncwarp();
    }
}

}  // namespace moc

// General incremental evaluation with a lane per edit (moc_eval_edits): a warp takes 32 edit records of any
// parents, every lane reads what it needs of its own parent's cache entry from global memory (so 32
// dependent chains of small reads are in flight per warp instead of one), and the admissible edits are
// finished by the whole warp one at a time (edit_pass, moc_edit_pass.cuh).  The block keeps the graph's
// lists and output sizes in shared memory when they fit.
#pragma once
#include "moc_edit_pass.cuh"

namespace moc {

constexpr int kLanesThreads = 256;

struct LanesParams {
    EditParams e;
    uint32_t graph_bytes;                                 // block's copy of the graph (0: read from global memory)
    uint32_t gs_pred_b, gs_m_b, gs_succ_b, gs_predl_b;
    uint32_t warp_bytes;                                  // correction list and difference array of one warp
    uint32_t lh_b, diff_b;                                // after the list values, which come first
    int32_t list_cap;
};

// Bytes of one warp: list values, list ranges (list_cap each), difference array (stride + 4).
__host__ __device__ inline size_t lanes_warp_bytes(int32_t stride, size_t mem_sz, int32_t list_cap, uint32_t* lh_b, uint32_t* diff_b) {
    size_t o = ((size_t)list_cap * mem_sz + 15) & ~size_t(15);
    *lh_b = (uint32_t)o;
    o += ((size_t)list_cap * 4 + 15) & ~size_t(15);
    *diff_b = (uint32_t)o;
    o += (((size_t)stride + 4) * mem_sz + 15) & ~size_t(15);
    return o;
}

// The lane's parent for edit_pass: its cache entry in global memory.
template <typename MemT>
struct LaneParent {
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
    // the usage array of lane l's parent, for all lanes of the warp
    __device__ __forceinline__ View prof_view(int l) const {
        const unsigned long long a = __shfl_sync(0xFFFFFFFFu, (unsigned long long)reinterpret_cast<uintptr_t>(prof_), l);
        return View{reinterpret_cast<const MemT*>((uintptr_t)a)};
    }
};

template <typename MemT, bool kGraphOnChip>
__global__ void __launch_bounds__(kLanesThreads, 4) edit_eval_lanes_kernel(const LanesParams p) {
    extern __shared__ __align__(16) char smem[];
    const EditParams& e = p.e;
    const EditCacheDev& c = e.c;
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    if (kGraphOnChip) score_stage_graph<MemT>(c, smem, p.gs_pred_b, p.gs_m_b, p.gs_succ_b, p.gs_predl_b);
    const ScoreGraph<MemT, kGraphOnChip> graph{reinterpret_cast<const uint32_t*>(smem), reinterpret_cast<const uint32_t*>(smem + p.gs_pred_b),
                                               reinterpret_cast<const MemT*>(smem + p.gs_m_b), reinterpret_cast<const uint16_t*>(smem + p.gs_succ_b),
                                               reinterpret_cast<const uint16_t*>(smem + p.gs_predl_b), &c};
    char* mine = smem + (kGraphOnChip ? p.graph_bytes : 0u) + (size_t)warp * p.warp_bytes;
    MemT* rv = reinterpret_cast<MemT*>(mine);
    uint32_t* rl = reinterpret_cast<uint32_t*>(mine + p.lh_b);
    MemT* diff = reinterpret_cast<MemT*>(mine + p.diff_b);
    for (int32_t i = lane; i < c.stride + 4; i += 32) diff[i] = 0;
    __syncwarp();

    const int64_t n_groups = ((int64_t)e.B + 31) / 32;
    for (int64_t g = (int64_t)blockIdx.x * wpb + warp; g < n_groups; g += (int64_t)gridDim.x * wpb) {
        const int64_t i = g * 32 + lane;
        const bool have = i < e.B;
        int32_t ci = 0, o = 0, qq = 0, jj = 0;
        if (have) {
            ci = __ldg(&e.parent[i]);
            o = __ldg(&e.op[i]);
            qq = __ldg(&e.q[i]);
            jj = __ldg(&e.j[i]);
        }
        const bool known = have && ci >= 0 && ci < c.P;
        if (!known) ci = 0;                                // any valid entry: nothing of it is used
        const int32_t T = c.len[ci], pst = c.status[ci];
        const int64_t pdur = c.dur[ci];
        // an unknown parent or a record out of range is malformed (status -2); an invalid parent comes first (-3)
        const bool live = known && pst >= 0 && o >= 0 && o <= 2 && qq >= 0 && qq < T && (o == 1 || (jj >= 0 && jj <= (o == 0 ? T : T - 1)));
        const LaneParent<MemT> parent{c.occ + (int64_t)ci * c.occ_stride, c.fre + (int64_t)ci * c.stride16, c.row + (int64_t)ci * c.stride16,
                                      reinterpret_cast<const MemT*>(c.prof) + (int64_t)ci * c.stride,
                                      reinterpret_cast<const MemT*>(c.pm) + (int64_t)ci * c.stride,
                                      reinterpret_cast<const MemT*>(c.sm) + (int64_t)ci * c.stride};
        int64_t out_pk, out_du;
        int32_t out_st, out_win;
        edit_pass<MemT>(parent, graph, c, e.M, lane, live, 0, live ? T : 0, pdur, o, live ? qq : 0, jj, rl, rv, diff, p.list_cap,
                        out_pk, out_du, out_st, out_win);
        if (known && pst < 0) out_st = kStatusParentInvalid;
        if (have) {
            e.out_peak[i] = out_pk;
            e.out_dur[i] = out_du;
            e.out_status[i] = out_st;
            if (e.out_window) e.out_window[i] = out_win;
        }
    }
}

}  // namespace moc

// Host side of the incremental evaluation (moc_cache_*, moc_eval_edits; declared in include/moc.h):
// the cache of evaluated parents on the device and the two launches.
#include <algorithm>
#include <new>

#include "moc_cache_host.cuh"

using namespace moc_host;

namespace {
size_t up256(size_t x) { return (x + 255) & ~size_t(255); }
}  // namespace

namespace moc_host {
int cache_prepare(moc_cache* h, const int32_t* seqs, const int32_t* lens, const int64_t* offs, int32_t P,
                  const int32_t* todo, const int32_t* todo_count, int64_t M, int64_t* out_peak, int64_t* out_dur,
                  int32_t* out_status, cudaStream_t st) {
    if (todo && h->graph_generation != h->g->generation)
        return fail(MOC_ERR_ARG, "the graph's C or node caps changed after the cache was built: rebuild the cache");
    if (h->g->C != h->c.C) return fail(MOC_ERR_ARG, "the graph's C changed after the cache was created: create a new cache");
    if (!todo) h->graph_generation = h->g->generation;
    h->c.P = P;
    h->c.cap = h->g->d_cap;
    moc::PrepParams p{};
    p.c = h->c;
    p.seqs = seqs;
    p.lens = lens;
    p.offs = offs;
    p.M = M;
    p.out_peak = out_peak;
    p.out_dur = out_dur;
    p.out_status = out_status;
    p.todo = todo;
    p.todo_count = todo_count;
    p.warp_bytes = (uint32_t)h->warp_bytes;
    // the successor tiles of the warp-per-sequence kernel, when the graph has them and its durations fit their packing
    const moc_graph* g = h->g;
    const bool tiles = g->d_rec32 != nullptr && g->C <= 2 && (__int128)g->C * g->sum_w < ((__int128)1 << 48);
    p.n_tiles = tiles ? g->n_tiles : 0;
    p.rec = h->wide ? g->d_rec64 : g->d_rec32;
    p.wslot = g->d_wslot;
    p.sell = g->d_sell;
    p.base_dur = g->sum_w;
    // block shape: with the tiles in the block's shared memory when that keeps at least 12 warps on an SM
    const size_t optin = g->smem_optin, cap = optin > 2048 ? optin - 2048 : 0;
    const size_t rec_b = (h->wide ? 16 : 8) * 64 * (size_t)g->n_tiles, w_b = 8 * 64 * (size_t)g->n_tiles,
                 sell_b = (4 * (size_t)g->sell_len + 15) & ~size_t(15), chip_b = rec_b + w_b + sell_b;
    int wpb = h->wpb, grid_cap = h->grid_cap;
    bool chip = false;
    if (tiles && chip_b + 12 * h->warp_bytes <= cap) {
        chip = true;
        wpb = (int)std::min<size_t>(moc::kPrepThreads / 32, (cap - chip_b) / h->warp_bytes);
        grid_cap = g->sm_count;
        p.chip_bytes = (uint32_t)chip_b;
        p.chip_w_b = (uint32_t)rec_b;
        p.chip_sell_b = (uint32_t)(rec_b + w_b);
        p.sell_len = g->sell_len;
    }
    const void* fn = chip ? (h->wide ? (const void*)moc::edit_prepare_kernel<int64_t, true> : (const void*)moc::edit_prepare_kernel<int32_t, true>)
                          : (h->wide ? (const void*)moc::edit_prepare_kernel<int64_t, false> : (const void*)moc::edit_prepare_kernel<int32_t, false>);
    MOC_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(optin - 1024)));
    const int grid = (int)std::min<int64_t>(grid_cap, ((int64_t)P + wpb - 1) / wpb);
    void* args[] = {&p};
    MOC_CUDA(cudaLaunchKernel(fn, dim3(grid), dim3(32 * wpb), args, (chip ? chip_b : 0) + h->warp_bytes * wpb, st));
    MOC_CUDA(cudaGetLastError());
    return MOC_OK;
}
}  // namespace moc_host

extern "C" {

int moc_cache_create(const moc_graph* g, int32_t max_parents, moc_cache** out) {
    clear_error();
    if (out) *out = nullptr;
    if (!g || !out || max_parents < 1) return fail(MOC_ERR_ARG, "moc_cache_create: null pointer or max_parents < 1");
    if (g->C > 2) return fail(MOC_ERR_ARG, "moc_cache_create: the incremental evaluation covers C <= 2 (handle has C = %d)", g->C);
    const int64_t max_T = (int64_t)g->C * g->n;
    if (max_T > 65534) return fail(MOC_ERR_ARG, "moc_cache_create: sequences of up to %lld steps exceed 65534", (long long)max_T);
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    moc_cache* h = new (std::nothrow) moc_cache();
    if (!h) return fail(MOC_ERR_NOMEM, "host allocation failed");
    h->g = g;
    h->device = g->device;
    h->max_parents = max_parents;
    h->wide = g->sum_m > (int64_t)INT32_MAX / g->C;
    const size_t msz = h->wide ? 8 : 4;
    const int32_t stride = (int32_t)((max_T + 3) & ~int64_t(3)), occ_stride = (g->n + 1 + 3) & ~3, stride16 = (stride + 7) & ~7;
    h->warp_bytes = moc::edit_warp_bytes(g->n, stride, msz);
    const size_t cap = g->smem_optin > 2048 ? g->smem_optin - 2048 : 0;
    if (h->warp_bytes > cap) {
        delete h;
        return fail(MOC_ERR_ARG, "moc_cache_create: %zu bytes of shared memory per sequence exceed the device's %zu", h->warp_bytes, cap);
    }
    // warps per block: the count that puts most warps on an SM
    int best = 0;
    for (int k = 1; k <= moc::kEditThreads / 32; ++k) {
        const size_t blk = h->warp_bytes * k + 1024;
        const int fit = blk <= cap + 1024 ? (int)(g->smem_optin / blk) * k : 0;
        if (fit > best) { best = fit; h->wpb = k; }
    }
    h->grid_cap = g->sm_count * std::max(1, best / h->wpb);
    const size_t P = (size_t)max_parents, S = (size_t)stride, S16 = (size_t)stride16;
    const size_t o_row = 0, o_fre = o_row + up256(P * S16 * 2), o_prof = o_fre + up256(P * S16 * 2), o_pm = o_prof + up256(P * S * msz),
                 o_sm = o_pm + up256(P * S * msz), o_occ = o_sm + up256(P * S * msz), o_len = o_occ + up256(P * occ_stride * 4),
                 o_st = o_len + up256(P * 4), o_peak = o_st + up256(P * 4), o_dur = o_peak + up256(P * 8),
                 o_offs = o_dur + up256(P * 8), total = o_offs + up256((P + 1) * 8);
    cudaError_t e = cudaMalloc((void**)&h->d_block, total);
    if (e != cudaSuccess) {
        delete h;
        cudaGetLastError();
        return fail(e == cudaErrorMemoryAllocation ? MOC_ERR_NOMEM : MOC_ERR_CUDA, "moc_cache_create: %s", cudaGetErrorString(e));
    }
    char* b = h->d_block;
    moc::EditCacheDev& c = h->c;
    c.n = g->n;
    c.C = g->C;
    c.P = 0;
    c.stride = stride;
    c.occ_stride = occ_stride;
    c.stride16 = stride16;
    c.max_T = (int32_t)max_T;
    c.succ_start = g->d_succ_start;
    c.succ = g->d_succ;
    c.pred_start = g->d_pred_start;
    c.pred = g->d_pred;
    c.w = g->d_w;
    c.m = g->d_m64;
    c.cap = g->d_cap;
    c.sink_m = g->sink_m;
    c.row = (uint16_t*)(b + o_row);
    c.fre = (uint16_t*)(b + o_fre);
    c.prof = b + o_prof;
    c.pm = b + o_pm;
    c.sm = b + o_sm;
    c.occ = (uint32_t*)(b + o_occ);
    c.len = (int32_t*)(b + o_len);
    c.status = (int32_t*)(b + o_st);
    c.peak = (int64_t*)(b + o_peak);
    c.dur = (int64_t*)(b + o_dur);
    h->d_offs = (int64_t*)(b + o_offs);
    *out = h;
    return MOC_OK;
}

int moc_cache_build(moc_cache* h, const int32_t* seqs, const int32_t* lens, int32_t P, int64_t M, int64_t* out_peak,
                    int64_t* out_dur, int32_t* out_status, void* stream) {
    clear_error();
    launch_counter() = 0;
    if (!h || !seqs || !lens || P < 1 || P > h->max_parents)
        return fail(MOC_ERR_ARG, "moc_cache_build: null pointer, or P outside [1, max_parents = %d]", h ? h->max_parents : 0);
    if (h->g->C != h->c.C) return fail(MOC_ERR_ARG, "moc_cache_build: the graph's C changed after the cache was created");
    DeviceGuard dg(h->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", h->device);
    cudaStream_t st = (cudaStream_t)stream;
    moc::offsets_kernel<<<(P + moc::kOffsTile - 1) / moc::kOffsTile, moc::kOffsThreads, 0, st>>>(lens, P, h->d_offs);
    int rc = cache_prepare(h, seqs, lens, h->d_offs, P, nullptr, nullptr, M, out_peak, out_dur, out_status, st);
    if (rc != MOC_OK) return rc;
    launch_counter() = 2;
    return MOC_OK;
}

int moc_eval_edits(const moc_cache* h, const int32_t* parent, const int32_t* op, const int32_t* q, const int32_t* j,
                   int32_t B, int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_status, int32_t* out_window,
                   void* stream) {
    clear_error();
    launch_counter() = 0;
    if (!h || B < 0) return fail(MOC_ERR_ARG, "moc_eval_edits: null handle or B < 0");
    if (B == 0) return MOC_OK;
    if (!parent || !op || !q || !j || !out_peak || !out_dur || !out_status) return fail(MOC_ERR_ARG, "moc_eval_edits: null array");
    if (h->c.P < 1) return fail(MOC_ERR_ARG, "moc_eval_edits: the cache holds no parents (call moc_cache_build first)");
    if (h->graph_generation != h->g->generation)
        return fail(MOC_ERR_ARG, "moc_eval_edits: the graph's C or node caps changed after the cache was built "
                    "(its copy of the caps is stale): rebuild the cache with moc_cache_build");
    DeviceGuard dg(h->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", h->device);
    moc::EditParams p{};
    p.c = h->c;
    p.parent = parent;
    p.op = op;
    p.q = q;
    p.j = j;
    p.B = B;
    p.M = M;
    p.out_peak = out_peak;
    p.out_dur = out_dur;
    p.out_status = out_status;
    p.out_window = out_window;
    const size_t msz = h->wide ? 8 : 4;
    const moc_graph* g = h->g;
    // ---- a lane per edit, when the correction lists of a warp and (if it fits) the graph find room on an SM
    if (h->lanes_state == 0) {
        h->lanes_state = -1;
        moc::LanesParams& lp = h->lanes;
        lp.list_cap = std::max(128, (4 + 2 * g->max_indeg + 31) & ~31);
        lp.warp_bytes = (uint32_t)moc::lanes_warp_bytes(h->c.stride, msz, lp.list_cap, &lp.lh_b, &lp.diff_b);
        const size_t cap = g->smem_optin > 2048 ? g->smem_optin - 2048 : 0;
        const int wpb = moc::kLanesThreads / 32;
        const size_t graph_b = moc::score_graph_bytes(g->n, g->n_edges, msz, &lp.gs_pred_b, &lp.gs_m_b, &lp.gs_succ_b, &lp.gs_predl_b);
        for (int chip = 1; chip >= 0 && h->lanes_state < 0; --chip) {
            if (chip && (g->n > 65535 || graph_b > cap / 8)) continue;
            const size_t smem = (chip ? graph_b : 0) + (size_t)lp.warp_bytes * wpb;
            if (smem > cap) continue;
            const void* fn = chip ? (h->wide ? (const void*)moc::edit_eval_lanes_kernel<int64_t, true> : (const void*)moc::edit_eval_lanes_kernel<int32_t, true>)
                                  : (h->wide ? (const void*)moc::edit_eval_lanes_kernel<int64_t, false> : (const void*)moc::edit_eval_lanes_kernel<int32_t, false>);
            MOC_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(g->smem_optin - 1024)));
            int nb = 0;
            MOC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, moc::kLanesThreads, smem));
            if (nb < 1) continue;
            lp.graph_bytes = chip ? (uint32_t)graph_b : 0u;
            h->lanes_fn = fn;
            h->lanes_smem = smem;
            h->lanes_grid_cap = g->sm_count * nb;
            h->lanes_state = 1;
        }
    }
    if (h->lanes_state > 0) {
        moc::LanesParams lp = h->lanes;
        lp.e = p;
        lp.e.c.cap = g->d_cap;
        const int wpb = moc::kLanesThreads / 32;
        const int64_t n_groups = ((int64_t)B + 31) / 32;
        const int grid = (int)std::min<int64_t>(h->lanes_grid_cap, (n_groups + wpb - 1) / wpb);
        void* args[] = {&lp};
        MOC_CUDA(cudaLaunchKernel(h->lanes_fn, dim3(grid), dim3(moc::kLanesThreads), args, h->lanes_smem, (cudaStream_t)stream));
        launch_counter() = 1;
        return MOC_OK;
    }
    // ---- a warp per edit
    const size_t warp_b = 2 * ((((size_t)h->c.stride + 4) * msz + 15) & ~size_t(15));
    p.warp_bytes = (uint32_t)warp_b;
    const int wpb = moc::kEditThreads / 32;
    const size_t smem = warp_b * wpb;
    auto fn = h->wide ? moc::edit_eval_kernel<int64_t> : moc::edit_eval_kernel<int32_t>;
    MOC_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(h->g->smem_optin - 1024)));
    if (smem > h->g->smem_optin - 1024) return fail(MOC_ERR_ARG, "moc_eval_edits: sequences too long for this build");
    int nb = 0;
    MOC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, moc::kEditThreads, smem));
    if (nb < 1) return fail(MOC_ERR_CUDA, "moc_eval_edits: kernel does not fit on an SM");
    const int grid = (int)std::min<int64_t>((int64_t)h->g->sm_count * nb, ((int64_t)B + wpb - 1) / wpb);
    fn<<<grid, moc::kEditThreads, smem, (cudaStream_t)stream>>>(p);
    MOC_CUDA(cudaGetLastError());
    launch_counter() = 1;
    return MOC_OK;
}

void moc_cache_destroy(moc_cache* h) {
    if (!h) return;
    DeviceGuard dg(h->device);
    cudaFree(h->d_block);
    delete h;
}

}  // extern "C"

// Host side of the search entry points of libmoc_b200.so (declared in include/moc.h): state of the
// chains on the device and the per-generation launch sequence.  Proposals, scoring and selection
// all run in kernels (moc_search_kernels.cuh and the evaluation kernels).
#include <algorithm>
#include <new>

#include <vector>

#include "moc_cache_host.cuh"
#include "moc_search_kernels.cuh"
#include "moc_search_score_kernel.cuh"

using namespace moc_host;

struct moc_search {
    const moc_graph* g = nullptr;
    int device = 0;
    int32_t P = 0, stride = 0;
    int64_t M = 0;
    uint64_t seed = 0;
    uint32_t generation = 0;   // generations completed (proposed, scored and settled)
    char* d_block = nullptr;   // one allocation, carved up below
    int32_t* d_bad = nullptr;
    moc::SearchParams p{};
    // search on the incremental evaluation (off until moc_search_set_samples switches it on)
    bool incremental = false;
    int32_t samples = 1;
    moc_cache* cache = nullptr;
    char* d_inc = nullptr;
    moc::SearchIncParams ip{};
    // one kernel per generation with a warp per chain (moc_search_score_kernel.cuh) instead of draw, score, pick
    bool fused = false;
    moc::ScoreParams sp{};
    int score_wpb = 0, score_grid_cap = 0;
    const void* score_fn = nullptr;
    size_t score_smem = 0;
};

namespace {

size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

int chain_blocks(int32_t P) { return (P + moc::kSearchThreads / 32 - 1) / (moc::kSearchThreads / 32); }

// Launch shape of the warp-per-chain generation kernel; false when the graph's largest in-degree or the row
// length leaves fewer than four warps on an SM.
bool plan_fused(moc_search* s) {
    const moc_graph* g = s->g;
    const moc_cache* h = s->cache;
    moc::ScoreParams& sp = s->sp;
    const size_t msz = h->wide ? 8 : 4;
    const int32_t worst = 4 + 2 * g->max_indeg;
    sp.list_cap = std::max(128, (worst + 31) & ~31);
    sp.warp_bytes = (uint32_t)moc::score_warp_bytes(h->c.occ_stride, h->c.stride, msz, sp.list_cap, &sp.fre_b, &sp.row_b, &sp.prof_b,
                                                   &sp.lh_b, &sp.val_b, &sp.diff_b);
    const size_t cap = g->smem_optin > 2048 ? g->smem_optin - 2048 : 0;
    if ((size_t)sp.warp_bytes * 4 > cap) return false;
    // with the block's own copy of the graph when that still leaves eight warps on an SM, else from global memory
    const int64_t E = g->n_edges;
    const size_t graph_b = moc::score_graph_bytes(g->n, E, msz, &sp.gs_pred_b, &sp.gs_m_b, &sp.gs_succ_b, &sp.gs_predl_b);
    sp.graph_bytes = (uint32_t)std::min<size_t>(graph_b, 0xFFFFFFF0u);
    int best = 0;
    for (int chip = 1; chip >= 0; --chip) {
        if (chip && (g->n > 65535 || graph_b > cap / 4)) continue;
        s->score_fn = chip ? (h->wide ? (const void*)moc::search_score_kernel<int64_t, true> : (const void*)moc::search_score_kernel<int32_t, true>)
                           : (h->wide ? (const void*)moc::search_score_kernel<int64_t, false> : (const void*)moc::search_score_kernel<int32_t, false>);
        if (cudaFuncSetAttribute(s->score_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(g->smem_optin - 1024)) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        const size_t fixed = chip ? sp.graph_bytes : 0;
        best = 0;
        for (int k = 1; k <= moc::kScoreThreads / 32; ++k) {
            const size_t blk = fixed + (size_t)sp.warp_bytes * k;
            if (blk > cap) break;
            int nb = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, s->score_fn, 32 * k, blk) != cudaSuccess) {
                cudaGetLastError();
                return false;
            }
            if (nb * k >= best && nb > 0) { best = nb * k; s->score_wpb = k; }     // ties: the larger block (one copy of the graph)
        }
        s->score_smem = fixed + (size_t)sp.warp_bytes * s->score_wpb;
        if (best >= 8) break;
    }
    if (best < 4) return false;
    s->score_grid_cap = g->sm_count * (best / s->score_wpb);
    return true;
}

}  // namespace

extern "C" {

int moc_search_create(const moc_graph* g, const int32_t* seqs, const int32_t* lens, int32_t P, int64_t M,
                      uint64_t seed, uint32_t first_chain, void* stream, moc_search** out) {
    clear_error();
    launch_counter() = 0;
    if (out) *out = nullptr;
    if (!g || !out || !seqs || !lens || P < 1) return fail(MOC_ERR_ARG, "moc_search_create: null pointer or P < 1");
    if (reinterpret_cast<uintptr_t>(seqs) & 3) return fail(MOC_ERR_ARG, "moc_search_create: seqs not 4-byte aligned");
    const int64_t max_T = (int64_t)g->C * g->n;
    const int64_t stride = (max_T + 3) & ~int64_t(3);
    if ((uint64_t)first_chain + (uint64_t)P > 0x100000000ull)
        return fail(MOC_ERR_ARG, "moc_search_create: first_chain + P exceeds 2^32");
    if (2 * (int64_t)P * stride > ((int64_t)1 << 40)) return fail(MOC_ERR_ARG, "moc_search_create: population too large");
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    cudaStream_t st = (cudaStream_t)stream;
    moc_search* s = new (std::nothrow) moc_search();
    if (!s) return fail(MOC_ERR_NOMEM, "host allocation failed");
    s->g = g;
    s->device = g->device;
    s->P = P;
    s->stride = (int32_t)stride;
    s->M = M;
    s->seed = seed;
    const size_t bP = (size_t)P;
    const size_t o_rows = 0, o_offs = o_rows + up256(2 * bP * (size_t)stride * 4), o_peak = o_offs + up256((bP + 1) * 8),
                 o_dur = o_peak + up256(bP * 8), o_cpeak = o_dur + up256(bP * 8), o_cdur = o_cpeak + up256(bP * 8),
                 o_cur = o_cdur + up256(bP * 8), o_lens = o_cur + up256(bP * 4), o_st = o_lens + up256(bP * 4),
                 o_acc = o_st + up256(bP * 4), o_clens = o_acc + up256(bP * 4), o_cst = o_clens + up256(bP * 4),
                 o_bad = o_cst + up256(bP * 4), total = o_bad + 256;
    cudaError_t e = cudaMalloc((void**)&s->d_block, total);
    if (e != cudaSuccess) {
        delete s;
        cudaGetLastError();
        return fail(e == cudaErrorMemoryAllocation ? MOC_ERR_NOMEM : MOC_ERR_CUDA, "moc_search_create: %s", cudaGetErrorString(e));
    }
    char* b = s->d_block;
    moc::SearchParams& p = s->p;
    p.P = P;
    p.stride = (int32_t)stride;
    p.max_T = (int32_t)max_T;
    p.M = M;
    p.seed_lo = (uint32_t)(seed & 0xFFFFFFFFu);
    p.seed_hi = (uint32_t)(seed >> 32);
    p.generation = 0;
    p.chain0 = first_chain;
    p.kinds = 7u;
    p.rows = (int32_t*)(b + o_rows);
    p.c_offs = (int64_t*)(b + o_offs);
    p.peak = (int64_t*)(b + o_peak);
    p.dur = (int64_t*)(b + o_dur);
    p.c_peak = (int64_t*)(b + o_cpeak);
    p.c_dur = (int64_t*)(b + o_cdur);
    p.cur = (int32_t*)(b + o_cur);
    p.lens = (int32_t*)(b + o_lens);
    p.status = (int32_t*)(b + o_st);
    p.n_acc = (int32_t*)(b + o_acc);
    p.c_lens = (int32_t*)(b + o_clens);
    p.c_status = (int32_t*)(b + o_cst);
    s->d_bad = (int32_t*)(b + o_bad);
    int rc = MOC_OK;
    int32_t bad = 0;
    auto run = [&]() -> int {
        MOC_CUDA(cudaMemsetAsync(s->d_bad, 0, 4, st));
        // packed offsets of the caller's sequences, then the rows, then their evaluation
        moc::offsets_kernel<<<(P + moc::kOffsTile - 1) / moc::kOffsTile, moc::kOffsThreads, 0, st>>>(lens, P, p.c_offs);
        moc::search_init_kernel<<<chain_blocks(P), moc::kSearchThreads, 0, st>>>(p, seqs, lens, p.c_offs, s->d_bad);
        moc::search_offsets_kernel<<<(P + 255) / 256, 256, 0, st>>>(p);
        MOC_CUDA(cudaGetLastError());
        int r = eval_rows(g, p.c_offs, p.rows, p.lens, P, M, p.peak, p.dur, p.status, st);
        if (r != MOC_OK) return r;
        MOC_CUDA(cudaMemcpyAsync(&bad, s->d_bad, 4, cudaMemcpyDeviceToHost, st));
        MOC_CUDA(cudaStreamSynchronize(st));
        return MOC_OK;
    };
    rc = run();
    if (rc == MOC_OK && bad)
        rc = fail(MOC_ERR_ARG, "moc_search_create: a sequence length lies outside [0, C*n = %lld]", (long long)max_T);
    if (rc != MOC_OK) {
        cudaFree(s->d_block);
        delete s;
        return rc;
    }
    *out = s;
    return MOC_OK;
}

int moc_search_run(moc_search* s, int32_t n_generations, void* stream) {
    clear_error();
    launch_counter() = 0;
    if (!s || n_generations < 0) return fail(MOC_ERR_ARG, "moc_search_run: null handle or negative count");
    if ((uint64_t)s->generation + (uint64_t)n_generations > 0xFFFFFFFFull)
        return fail(MOC_ERR_ARG, "moc_search_run: generation counter would pass 2^32 - 1");
    if (n_generations == 0) return MOC_OK;
    DeviceGuard dg(s->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", s->device);
    cudaStream_t st = (cudaStream_t)stream;
    moc::SearchParams& p = s->p;
    const int blocks = chain_blocks(s->P);
    int launches = 0;
    if (s->incremental && s->fused) {
        moc_cache* h = s->cache;
        if (h->graph_generation != h->g->generation)
            return fail(MOC_ERR_ARG, "moc_search_run: the graph's C or node caps changed after the search's cache was built");
        const int wpb = s->score_wpb;
        const int grid = (int)std::min<int64_t>(s->score_grid_cap, ((int64_t)s->P + wpb - 1) / wpb);
        for (int32_t k = 0; k < n_generations; ++k) {
            p.generation = s->generation + (uint32_t)k;
            s->sp.s = p;
            s->sp.c = h->c;
            s->sp.c.cap = h->g->d_cap;
            void* args[] = {&s->sp};
            MOC_CUDA(cudaLaunchKernel(s->score_fn, dim3(grid), dim3(32 * wpb), args, s->score_smem, st));
            int rc = cache_prepare(h, p.rows, p.lens, s->ip.row_offs, s->P, s->ip.todo, s->ip.todo_count + (p.generation & 1u),
                                   s->M, nullptr, nullptr, nullptr, st);
            if (rc != MOC_OK) return rc;
            launches += 2;
        }
        MOC_CUDA(cudaGetLastError());
        s->generation += (uint32_t)n_generations;
        launch_counter() = launches;
        return MOC_OK;
    }
    if (s->incremental) {
        const int64_t nE = (int64_t)s->P * s->samples;
        for (int32_t k = 0; k < n_generations; ++k) {
            p.generation = s->generation + (uint32_t)k;
            s->ip.s = p;
            moc::search_draw_kernel<<<(unsigned)((nE + 255) / 256), 256, 0, st>>>(s->ip);
            int rc = moc_eval_edits(s->cache, s->ip.e_parent, s->ip.e_op, s->ip.e_q, s->ip.e_j, (int32_t)nE, s->M,
                                    s->ip.r_peak, s->ip.r_dur, s->ip.r_status, nullptr, stream);
            if (rc != MOC_OK) return rc;
            moc::search_pick_kernel<<<blocks, moc::kSearchThreads, 0, st>>>(s->ip);
            rc = cache_prepare(s->cache, p.rows, p.lens, s->ip.row_offs, s->P, s->ip.todo, s->ip.todo_count, s->M,
                               nullptr, nullptr, nullptr, st);
            if (rc != MOC_OK) return rc;
            launches += 4;
        }
        MOC_CUDA(cudaGetLastError());
        s->generation += (uint32_t)n_generations;
        launch_counter() = launches;
        return MOC_OK;
    }
    for (int32_t k = 0; k < n_generations; ++k) {
        p.generation = s->generation + (uint32_t)k;
        // settle the previous generation's proposals (none before the first one), propose the next
        if (k == 0) moc::search_step_kernel<false, true><<<blocks, moc::kSearchThreads, 0, st>>>(p);
        else moc::search_step_kernel<true, true><<<blocks, moc::kSearchThreads, 0, st>>>(p);
        ++launches;
        int rc = eval_rows(s->g, p.c_offs, p.rows, p.c_lens, s->P, s->M, p.c_peak, p.c_dur, p.c_status, st);
        launches += launch_counter();
        launch_counter() = 0;
        if (rc != MOC_OK) return rc;
    }
    moc::search_step_kernel<true, false><<<blocks, moc::kSearchThreads, 0, st>>>(p);
    ++launches;
    MOC_CUDA(cudaGetLastError());
    s->generation += (uint32_t)n_generations;
    launch_counter() = launches;
    return MOC_OK;
}

int moc_search_set_kinds(moc_search* s, uint32_t kinds) {
    clear_error();
    if (!s || kinds == 0 || kinds > 7u) return fail(MOC_ERR_ARG, "moc_search_set_kinds: null handle or mask outside 1..7");
    s->p.kinds = kinds;
    return MOC_OK;
}

int moc_search_set_samples(moc_search* s, int32_t samples, int32_t incremental) {
    clear_error();
    if (!s || samples < 1 || samples > 4096 || incremental < 0 || incremental > 3)
        return fail(MOC_ERR_ARG, "moc_search_set_samples: null handle, samples outside [1, 4096] or mode outside 0..3");
    if (samples > 1 && !incremental)
        return fail(MOC_ERR_ARG, "moc_search_set_samples: more than one proposal per chain needs the incremental evaluation");
    if ((int64_t)s->P * samples > INT32_MAX) return fail(MOC_ERR_ARG, "moc_search_set_samples: P * samples exceeds 2^31 - 1");
    DeviceGuard dg(s->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", s->device);
    MOC_CUDA(cudaDeviceSynchronize());          // generations in flight still use the old buffers
    if (!incremental) {
        s->incremental = false;
        s->fused = false;
        s->samples = 1;
        return MOC_OK;
    }
    // every chain needs a valid evaluation to start from
    std::vector<int32_t> st((size_t)s->P);
    MOC_CUDA(cudaMemcpy(st.data(), s->p.status, (size_t)s->P * 4, cudaMemcpyDeviceToHost));
    for (int32_t c = 0; c < s->P; ++c)
        if (st[c] < 0)
            return fail(MOC_ERR_ARG, "moc_search_set_samples: chain %d has no valid sequence (status %d); the incremental "
                        "evaluation starts from valid sequences only", c, st[c]);
    if (!s->cache) {
        moc_cache* h = nullptr;
        int rc = moc_cache_create(s->g, s->P, &h);
        if (rc != MOC_OK) return rc;
        s->cache = h;
    }
    const size_t nE = (size_t)s->P * samples, bP = (size_t)s->P;
    const size_t o_par = 0, o_op = o_par + up256(nE * 4), o_q = o_op + up256(nE * 4), o_j = o_q + up256(nE * 4),
                 o_st = o_j + up256(nE * 4), o_pk = o_st + up256(nE * 4), o_du = o_pk + up256(nE * 8),
                 o_offs = o_du + up256(nE * 8), o_todo = o_offs + up256((bP + 1) * 8), o_cnt = o_todo + up256(bP * 4),
                 total = o_cnt + 256;          // o_cnt: two counters, used in turn by the warp-per-chain kernel
    if (s->d_inc) MOC_CUDA(cudaFree(s->d_inc));
    s->d_inc = nullptr;
    s->incremental = false;
    cudaError_t e = cudaMalloc((void**)&s->d_inc, total);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(e == cudaErrorMemoryAllocation ? MOC_ERR_NOMEM : MOC_ERR_CUDA, "moc_search_set_samples: %s", cudaGetErrorString(e));
    }
    char* b = s->d_inc;
    moc::SearchIncParams& ip = s->ip;
    ip.s = s->p;
    ip.samples = samples;
    ip.e_parent = (int32_t*)(b + o_par);
    ip.e_op = (int32_t*)(b + o_op);
    ip.e_q = (int32_t*)(b + o_q);
    ip.e_j = (int32_t*)(b + o_j);
    ip.r_status = (int32_t*)(b + o_st);
    ip.r_peak = (int64_t*)(b + o_pk);
    ip.r_dur = (int64_t*)(b + o_du);
    ip.row_offs = (int64_t*)(b + o_offs);
    ip.todo = (int32_t*)(b + o_todo);
    ip.todo_count = (int32_t*)(b + o_cnt);
    MOC_CUDA(cudaMemset(ip.todo_count, 0, 8));
    // scoring kernel: a warp per chain when asked for, or by default from 24 proposals per chain on
    // (below that the lane-per-edit kernel of moc_eval_edits, with more warps per SM, is as fast or faster)
    s->fused = false;
    if (incremental == MOC_SEARCH_SCORE_CHAIN || (incremental == MOC_SEARCH_SCORE_AUTO && samples >= 24)) {
        s->fused = plan_fused(s);
        if (!s->fused && incremental == MOC_SEARCH_SCORE_CHAIN) {
            cudaFree(s->d_inc);
            s->d_inc = nullptr;
            return fail(MOC_ERR_ARG, "moc_search_set_samples: the warp-per-chain kernel cannot hold this graph's rows and "
                        "correction lists (n = %d, largest in-degree %d) in shared memory", s->g->n, s->g->max_indeg);
        }
    }
    s->sp.samples = samples;
    s->sp.row_offs = ip.row_offs;
    s->sp.todo = ip.todo;
    s->sp.todo_count = ip.todo_count;
    // cache of all chains from their current rows
    moc::search_row_offsets_kernel<<<(s->P + 255) / 256, 256>>>(ip);
    int rc = cache_prepare(s->cache, s->p.rows, s->p.lens, ip.row_offs, s->P, nullptr, nullptr, s->M, nullptr, nullptr, nullptr, nullptr);
    if (rc != MOC_OK) return rc;
    MOC_CUDA(cudaDeviceSynchronize());
    s->samples = samples;
    s->incremental = true;
    return MOC_OK;
}

int moc_search_state(const moc_search* s, int32_t* out_rows, int32_t* out_lens, int64_t* out_peak,
                     int64_t* out_dur, int32_t* out_status, int32_t* out_accepted, void* stream) {
    clear_error();
    if (!s) return fail(MOC_ERR_ARG, "moc_search_state: null handle");
    DeviceGuard dg(s->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", s->device);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t bP = (size_t)s->P;
    if (out_rows) {
        moc::search_export_kernel<<<chain_blocks(s->P), moc::kSearchThreads, 0, st>>>(s->p, out_rows);
        MOC_CUDA(cudaGetLastError());
    }
    if (out_lens) MOC_CUDA(cudaMemcpyAsync(out_lens, s->p.lens, bP * 4, cudaMemcpyDeviceToDevice, st));
    if (out_peak) MOC_CUDA(cudaMemcpyAsync(out_peak, s->p.peak, bP * 8, cudaMemcpyDeviceToDevice, st));
    if (out_dur) MOC_CUDA(cudaMemcpyAsync(out_dur, s->p.dur, bP * 8, cudaMemcpyDeviceToDevice, st));
    if (out_status) MOC_CUDA(cudaMemcpyAsync(out_status, s->p.status, bP * 4, cudaMemcpyDeviceToDevice, st));
    if (out_accepted) MOC_CUDA(cudaMemcpyAsync(out_accepted, s->p.n_acc, bP * 4, cudaMemcpyDeviceToDevice, st));
    return MOC_OK;
}

int moc_search_best(const moc_search* s, int32_t* out_seq, int64_t* out_best, void* stream) {
    clear_error();
    if (!s || !out_best) return fail(MOC_ERR_ARG, "moc_search_best: null handle or null out_best");
    DeviceGuard dg(s->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", s->device);
    moc::search_best_kernel<<<1, moc::kBestThreads, 0, (cudaStream_t)stream>>>(s->p, out_seq, out_best);
    MOC_CUDA(cudaGetLastError());
    return MOC_OK;
}

int moc_search_info(const moc_search* s, int32_t* P, int32_t* stride, uint32_t* generation) {
    clear_error();
    if (!s) return fail(MOC_ERR_ARG, "moc_search_info: null handle");
    if (P) *P = s->P;
    if (stride) *stride = s->stride;
    if (generation) *generation = s->generation;
    return MOC_OK;
}

void moc_search_destroy(moc_search* s) {
    if (!s) return;
    DeviceGuard dg(s->device);
    moc_cache_destroy(s->cache);
    cudaFree(s->d_inc);
    cudaFree(s->d_block);
    delete s;
}

}  // extern "C"

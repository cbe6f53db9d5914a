// Host side of libmoc_b200.so: graph handle, validation, launch planning and the C ABI declared in
// include/moc.h.  Every step of the evaluation itself runs in the kernels of moc_kernels.cuh.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "moc_host.cuh"

using namespace moc_host;

namespace {
thread_local char g_err[512] = "";
thread_local int g_launches_tl = 0;
}  // namespace
#define g_launches (moc_host::launch_counter())

namespace moc_host {
int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}
void clear_error() { g_err[0] = 0; }
int& launch_counter() { return g_launches_tl; }
}  // namespace moc_host

namespace {

size_t align16(size_t x) { return (x + 15) & ~size_t(15); }

template <int G, typename MemT>
KernelFn shared_fn_cp(int CP, bool profile) {
    if (profile && G != 1024) return nullptr;
    switch (CP) {
        case 2: return profile ? (KernelFn)moc::eval_shared_kernel<1024, MemT, 2, true>
                               : (KernelFn)moc::eval_shared_kernel<G, MemT, 2, false>;
        case 4: return profile ? (KernelFn)moc::eval_shared_kernel<1024, MemT, 4, true>
                               : (KernelFn)moc::eval_shared_kernel<G, MemT, 4, false>;
        default: return profile ? (KernelFn)moc::eval_shared_kernel<1024, MemT, 8, true>
                                : (KernelFn)moc::eval_shared_kernel<G, MemT, 8, false>;
    }
}
template <typename MemT>
KernelFn shared_fn_g(int G, int CP, bool profile) {
    switch (G) {
        case 32: return shared_fn_cp<32, MemT>(CP, profile);
        case 64: return shared_fn_cp<64, MemT>(CP, profile);
        case 128: return shared_fn_cp<128, MemT>(CP, profile);
        case 256: return shared_fn_cp<256, MemT>(CP, profile);
        case 512: return shared_fn_cp<512, MemT>(CP, profile);
        case 1024: return shared_fn_cp<1024, MemT>(CP, profile);
        default: return nullptr;
    }
}
KernelFn global_fn(int CP, bool profile) {
    switch (CP) {
        case 2: return profile ? (KernelFn)moc::eval_global_kernel<2, true> : (KernelFn)moc::eval_global_kernel<2, false>;
        case 4: return profile ? (KernelFn)moc::eval_global_kernel<4, true> : (KernelFn)moc::eval_global_kernel<4, false>;
        default: return profile ? (KernelFn)moc::eval_global_kernel<8, true> : (KernelFn)moc::eval_global_kernel<8, false>;
    }
}

template <typename MemT>
PairFn pair_fn_t(int pre) {
    switch (pre) {
        case 0: return (PairFn)moc::eval_pair_kernel<MemT, 0>;
        case 1: return (PairFn)moc::eval_pair_kernel<MemT, 1>;
        case 2: return (PairFn)moc::eval_pair_kernel<MemT, 2>;
        case 3: return (PairFn)moc::eval_pair_kernel<MemT, 3>;
        case 4: return (PairFn)moc::eval_pair_kernel<MemT, 4>;
        default: return (PairFn)moc::eval_pair_kernel<MemT, 5>;
    }
}
PairFn pair_fn(bool wide, int pre) { return wide ? pair_fn_t<int64_t>(pre) : pair_fn_t<int32_t>(pre); }

template <typename MemT, int LG>
LaneFn lane_fn_kp(int kp) {
    switch (kp) {
        case 2: return (LaneFn)moc::eval_lane_kernel<MemT, LG, 2>;
        case 4: return (LaneFn)moc::eval_lane_kernel<MemT, LG, 4>;
        case 6: return (LaneFn)moc::eval_lane_kernel<MemT, LG, 6>;
        default: return (LaneFn)moc::eval_lane_kernel<MemT, LG, 8>;
    }
}
template <typename MemT>
LaneFn lane_fn_lg(int lg, int kp) {
    switch (lg) {
        case 5: return lane_fn_kp<MemT, 5>(kp);
        case 4: return lane_fn_kp<MemT, 4>(kp);
        default: return lane_fn_kp<MemT, 3>(kp);
    }
}
LaneFn lane_fn(bool wide, int lg, int kp) { return wide ? lane_fn_lg<int64_t>(lg, kp) : lane_fn_lg<int32_t>(lg, kp); }

QuadFn quad_fn(bool wide, int C) {
    if (C <= 3) return wide ? (QuadFn)moc::eval_quad_kernel<int64_t, 3> : (QuadFn)moc::eval_quad_kernel<int32_t, 3>;
    return wide ? (QuadFn)moc::eval_quad_kernel<int64_t, 4> : (QuadFn)moc::eval_quad_kernel<int32_t, 4>;
}

// Raises a kernel's dynamic shared-memory limit to all the device offers beside its static part.
cudaError_t raise_smem_limit(const void* fn, size_t smem_optin) {
    cudaFuncAttributes a{};
    cudaError_t e = cudaFuncGetAttributes(&a, fn);
    if (e != cudaSuccess) return e;
    const size_t room = smem_optin > a.sharedSizeBytes ? smem_optin - a.sharedSizeBytes : 0;
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)room);
}

int pow2_ceil(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

// Plan of the sequence-per-lane path: the largest group whose state fits beside the graph, with as
// many warps per SM as fit.  Returns nullptr on success, else the reason it cannot serve the graph.
const char* plan_lane(const moc_graph* g, size_t smem_cap, Plan* out) {
    Plan pl = *out;
    const int64_t n = g->n, C = g->C, t_max = C * n;
    if (C > 2) return "C > 2";
    if ((__int128)C * g->sum_w >= ((__int128)1 << 40)) return "C * sum(w) reaches 2^40";
    const bool forced = g->want_kind == MOC_KERNEL_LANE;
    const size_t msz = pl.wide ? 8 : 4;
    for (int li = 0; li < 3; ++li) {
        const int lg = 5 - li, gsz = 1 << lg, S = 32 >> lg;
        const LaneLayout& L = g->lane[li];
        if (!L.ok) continue;
        if (forced && g->want_a && g->want_a != gsz) continue;
        const size_t rec_b = 32 * (size_t)S * L.n_bundles, succ_b = align16(4 * (size_t)L.succ_len),
                     part_b = 2 * align16(32 * msz * ((size_t)gsz + 1)),
                     word_b = moc::lane_special(gsz) + align16((size_t)moc::lane_word_row(gsz) * (n + 1)),
                     delta_b = align16(msz * gsz * (size_t)(t_max + 3));
        const size_t sm = rec_b + succ_b + part_b + word_b + delta_b;
        if (sm > smem_cap) continue;
        int best_w = 0, best_nb = 0, best_kp = 0;
        for (int w = 32; w >= gsz; w -= gsz) {    // a whole number of warps per row of the group
            if (forced && g->want_b && g->want_b != w) continue;
            // pieces of 128 steps fetched ahead per warp: enough for typical rows of about 1.3 n steps
            const int64_t pieces = ((n * 13 / 10 + 6) / 4 + 31) / 32;
            int kp = (int)((pieces * gsz + w - 1) / w);
            kp = std::min(8, std::max(2, (kp + 1) & ~1));
            LaneFn fn = lane_fn(pl.wide, lg, kp);
            if (raise_smem_limit((const void*)fn, g->smem_optin) != cudaSuccess) { cudaGetLastError(); continue; }
            int nb = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, (const void*)fn, w * 32, sm) != cudaSuccess) { cudaGetLastError(); continue; }
            if (nb < 1) continue;
            // as many warps per SM as fit, up to 64; among equals the shape with more blocks
            const int warps = std::min(nb * w, 64), best = std::min(best_nb * best_w, 64);
            if (warps > best || (warps == best && nb > best_nb && w >= 8)) { best_w = w; best_nb = nb; best_kp = kp; }
        }
        if (best_w == 0) continue;
        pl.lane = true;
        pl.lane_fn = lane_fn(pl.wide, lg, best_kp);
        pl.lane_lg = lg;
        pl.G = 32 * best_w / gsz;
        pl.gpc = gsz;
        pl.block = 32 * best_w;
        pl.smem = sm;
        pl.grid = g->sm_count * best_nb;
        pl.sm_count = g->sm_count;
        pl.lane_rec_b = (uint32_t)rec_b; pl.lane_succ_b = (uint32_t)succ_b;
        pl.lane_word_b = (uint32_t)word_b; pl.lane_delta_b = (uint32_t)delta_b;
        pl.valid = true;
        *out = pl;
        return nullptr;
    }
    return "the state of a group of sequences exceeds shared memory in the requested shape, n >= 4096, or a degree above 255";
}

// Plan of the block-per-sequence path with packed words (C <= 4).  Returns nullptr on success.
const char* plan_quad(const moc_graph* g, size_t smem_cap, Plan* out) {
    Plan pl = *out;
    const int64_t n = g->n, C = g->C, t_max = C * n;
    if (C > 4) return "C > 4";
    if (!g->d_order32) return "n above 32000 or a degree above 65535";
    if (t_max > 32766) return "sequences of more than 32766 steps";
    const size_t msz = pl.wide ? 8 : 4;
    const size_t word_b = align16(8 * (size_t)(n + 2)), cnt_b = align16(2 * (size_t)(n + 2)), delta_b = align16(msz * (size_t)(t_max + 4));
    const size_t sm = word_b + cnt_b + delta_b;
    if (sm > smem_cap) return "the state of a sequence exceeds shared memory";
    QuadFn fn = quad_fn(pl.wide, (int)C);
    if (raise_smem_limit((const void*)fn, g->smem_optin) != cudaSuccess) { cudaGetLastError(); return "cudaFuncSetAttribute failed"; }
    // threads per sequence, from measurements at n = 100, 1000 and 5000 (more threads lose to the block-wide
    // barriers, fewer to the length of the per-thread loops); or as requested
    int thr = n < 200 ? 64 : (n < 1600 ? 128 : (n < 12000 ? 512 : 1024));
    if (g->want_kind == MOC_KERNEL_BLOCK && g->want_a) thr = g->want_a;
    int nb = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, (const void*)fn, thr, sm) != cudaSuccess || nb < 1) { cudaGetLastError(); return "kernel does not fit on an SM"; }
    pl.quad = true;
    pl.quad_fn = fn;
    pl.G = thr;
    pl.gpc = 1;
    pl.block = thr;
    pl.smem = sm;
    pl.grid = g->sm_count * nb;
    pl.quad_word_b = (uint32_t)word_b;
    pl.quad_cnt_b = (uint32_t)cnt_b;
    pl.valid = true;
    *out = pl;
    return nullptr;
}

// Chooses kernel variant, group size and grid for the handle's current n and C.  The dynamic
// shared-memory limit of a kernel is a property of the kernel, not of the handle: it is always
// raised to the device maximum, so that handles with different needs can share one kernel.
int make_plan(const moc_graph* g, bool profile, Plan* out) {
    Plan pl;
    const int64_t n = g->n, C = g->C;
    pl.CP = C <= 2 ? 2 : (C <= 4 ? 4 : 8);
    pl.wide = g->sum_m > (int64_t)INT32_MAX / C;  // C*sum(m) bounds every partial sum of deltas
    const int64_t t_max = C * n;
    const size_t mem_sz = pl.wide ? 8 : 4;
    const size_t sh_cnt = align16(4 * n), sh_occ = align16(2 * n * pl.CP),
                 sh_delta = align16((t_max + 1) * mem_sz);
    const size_t sh_group = sh_cnt + sh_occ + sh_delta + align16(moc::kRedBytes);
    const size_t smem_cap = g->smem_optin > 1024 ? g->smem_optin - 1024 : 0;  // 1 KB per block is reserved
    const int kind = profile ? MOC_KERNEL_GROUP : g->want_kind;
    const bool shape_given = g->want_G != 0 || g->want_gpc != 0;       // moc_graph_set_launch
    // Order of preference when nothing is forced: warp per sequence, then sequence per lane (it also
    // serves graphs whose degrees are too uneven for the warp kernel's padded successor tiles), then
    // the thread-group kernel, which serves everything.
    const bool warp_ok = C <= 2 && g->d_rec32 != nullptr && (__int128)C * g->sum_w < ((__int128)1 << 48);
    if (kind == MOC_KERNEL_LANE || (kind == MOC_KERNEL_AUTO && !shape_given && !warp_ok)) {
        const char* why = plan_lane(g, smem_cap, &pl);
        if (!why) {
            *out = pl;
            return MOC_OK;
        }
        if (kind == MOC_KERNEL_LANE) return fail(MOC_ERR_ARG, "the sequence-per-lane kernel cannot serve this graph: %s", why);
    }
    if (kind == MOC_KERNEL_BLOCK || (kind == MOC_KERNEL_AUTO && !shape_given && !profile && C >= 3)) {
        const char* why = plan_quad(g, smem_cap, &pl);
        if (!why) {
            *out = pl;
            return MOC_OK;
        }
        if (kind == MOC_KERNEL_BLOCK) return fail(MOC_ERR_ARG, "the block-per-sequence kernel cannot serve this graph: %s", why);
    }
    if (kind == MOC_KERNEL_WARP && !warp_ok)
        return fail(MOC_ERR_ARG, "the warp-per-sequence kernel cannot serve this graph (C > 2, degrees too uneven or C * sum(w) >= 2^48)");
    if (!profile && g->want_G == 0 && kind != MOC_KERNEL_GROUP && warp_ok) {
        // warp-per-sequence fast path
        const size_t msz = pl.wide ? 8 : 4, per_vec = 16 / msz;
        const size_t nvec_d = (t_max + 2 + per_vec - 1) / per_vec;
        const size_t v_max = ((nvec_d + 31) / 32) | 1;
        const size_t rec_b = (pl.wide ? 16 : 8) * 64 * (size_t)g->n_tiles, jds_b = align16(4 * (size_t)g->sell_len),
                     word_b = align16(4 * (n + 2)), delta_b = moc::kPairDeltaFront + 32 * v_max * 16;
        const size_t w_b = 8 * 64 * (size_t)g->n_tiles;
        const size_t graph_b = rec_b + w_b + jds_b, warp_b = word_b + moc::kPairWordTail + delta_b;
        // vectors of the next row fetched ahead per lane: enough for a typical row of about 1.3 n steps
        const int pre = n < 256 ? 0 : (int)std::min<int64_t>(5, (n * 13 / 10 + 96) / 128);
        PairFn fn = pair_fn(pl.wide, pre);
        int best_wpb = 0, best_warps = 0, best_nb = 0;
        if (raise_smem_limit((const void*)fn, g->smem_optin) != cudaSuccess) cudaGetLastError();
        for (int wpb = 16; wpb >= 4; --wpb) {    // every kernel variant is compiled for up to 512 threads, two blocks per SM
            if (g->want_gpc && wpb != std::min(g->want_gpc, 16)) continue;
            const size_t sm = graph_b + wpb * warp_b;
            if (sm > smem_cap) continue;
            int nb = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, (const void*)fn, wpb * 32, sm) != cudaSuccess) { cudaGetLastError(); continue; }
            pl.pair_nb[wpb] = nb;
            if (nb * wpb > best_warps) { best_warps = nb * wpb; best_wpb = wpb; best_nb = nb; }
        }
        pl.pair_graph_b = graph_b;
        pl.pair_warp_b = warp_b;
        pl.sm_count = g->sm_count;
        if (best_warps >= 8) {
            pl.pair = true;
            pl.pair_fn = fn;
            pl.G = 32;
            pl.gpc = best_wpb;
            pl.block = 32 * best_wpb;
            pl.smem = graph_b + best_wpb * warp_b;
            pl.grid = g->sm_count * best_nb;
            pl.rec_bytes = (uint32_t)rec_b; pl.w_bytes = (uint32_t)w_b;
            pl.sell_bytes = (uint32_t)jds_b; pl.word_bytes = (uint32_t)word_b; pl.delta_bytes = (uint32_t)delta_b;
            cudaError_t e = raise_smem_limit((const void*)fn, g->smem_optin);
            if (e != cudaSuccess) return fail(MOC_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
            pl.valid = true;
            *out = pl;
            return MOC_OK;
        }
    }
    if (t_max <= 65534 && sh_group <= smem_cap) {
        pl.global_state = false;
        pl.cnt_bytes = (uint32_t)sh_cnt;
        pl.occ_bytes = (uint32_t)sh_occ;
        pl.delta_bytes = (uint32_t)sh_delta;
        pl.group_bytes = (uint32_t)sh_group;
        int G = 1024, gpc = 1;
        if (!profile) {
            const int per_sm = (int)std::max<size_t>(1, g->smem_optin / sh_group);  // groups resident per SM
            G = g->want_G ? g->want_G : std::min(1024, std::max(32, pow2_ceil(32 * 48 / std::min(per_sm, 48))));
            gpc = g->want_gpc ? g->want_gpc : std::max(1, 256 / G);
            gpc = std::min(gpc, G == 32 ? 32 : 15);          // named barriers 1..15
            gpc = std::min(gpc, 1024 / G);
            while (gpc > 1 && (size_t)gpc * sh_group > smem_cap) --gpc;
        }
        pl.G = G;
        pl.gpc = gpc;
        pl.block = G * gpc;
        pl.smem = (size_t)gpc * sh_group;
        pl.fn = pl.wide ? shared_fn_g<int64_t>(G, pl.CP, profile) : shared_fn_g<int32_t>(G, pl.CP, profile);
        if (!pl.fn) return fail(MOC_ERR_ARG, "unsupported launch shape");
        cudaError_t e = raise_smem_limit((const void*)pl.fn, g->smem_optin);
        if (e != cudaSuccess) return fail(MOC_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        int nb = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, (const void*)pl.fn, pl.block, pl.smem);
        if (e != cudaSuccess) return fail(MOC_ERR_CUDA, "occupancy query: %s", cudaGetErrorString(e));
        if (nb < 1) return fail(MOC_ERR_CUDA, "kernel does not fit on an SM (block %d, smem %zu)", pl.block, pl.smem);
        pl.grid = profile ? 1 : g->sm_count * nb;
    } else {
        // state in global memory: int32 positions, int64 sums
        pl.global_state = true;
        pl.wide = true;
        pl.cnt_bytes = (uint32_t)align16(4 * n);
        const size_t occ = align16(4 * n * pl.CP), del = align16((t_max + 1) * 8);
        const size_t grp = pl.cnt_bytes + occ + del + align16(moc::kRedBytes);
        if (grp > 0xFFFFFFFFull) return fail(MOC_ERR_ARG, "graph too large: per-sequence state of %zu bytes", grp);
        pl.occ_bytes = (uint32_t)occ;
        pl.delta_bytes = (uint32_t)del;
        pl.group_bytes = (uint32_t)grp;
        pl.G = 1024;
        pl.gpc = 1;
        pl.block = 1024;
        pl.smem = 0;
        pl.fn = global_fn(pl.CP, profile);
        int nb = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, (const void*)pl.fn, pl.block, 0);
        if (e != cudaSuccess) return fail(MOC_ERR_CUDA, "occupancy query: %s", cudaGetErrorString(e));
        if (nb < 1) nb = 1;
        pl.grid = profile ? 1 : g->sm_count * nb;
    }
    pl.valid = true;
    *out = pl;
    return MOC_OK;
}

int ensure(void** ptr, size_t* cap, size_t need) {
    if (need <= *cap) return MOC_OK;
    if (*ptr) {
        MOC_CUDA(cudaFree(*ptr));
        *ptr = nullptr;
        *cap = 0;
    }
    size_t want = std::max(need, *cap * 2);
    MOC_CUDA(cudaMalloc(ptr, want));
    *cap = want;
    return MOC_OK;
}


// Words 4-5 of the node records of the sequence-per-lane layouts: w | 1 << 40 (counts the node when
// it has two copies) | 1 << 52 when the node's cap C_v is 1.  Uploads both record arrays.
int upload_lane_rec(moc_graph* g) {
    for (int li = 0; li < 3; ++li) {
        LaneLayout& L = g->lane[li];
        if (!L.ok) continue;
        for (size_t r = 0; r < L.h_node.size(); ++r) {
            const int32_t v = L.h_node[r];
            uint64_t x = 0;
            if (v >= 0) {
                x = (uint64_t)g->h_w[v] | (uint64_t(1) << moc::kLaneCntShift);
                if (!g->h_cap.empty() && g->h_cap[v] == 1) x |= uint64_t(1) << moc::kLaneCapShift;
            }
            L.h_rec32[8 * r + 4] = L.h_rec64[8 * r + 4] = (uint32_t)(x & 0xFFFFFFFFu);
            L.h_rec32[8 * r + 5] = L.h_rec64[8 * r + 5] = (uint32_t)(x >> 32);
        }
        MOC_CUDA(cudaMemcpy(L.d_rec32, L.h_rec32.data(), L.h_rec32.size() * 4, cudaMemcpyHostToDevice));
        MOC_CUDA(cudaMemcpy(L.d_rec64, L.h_rec64.data(), L.h_rec64.size() * 4, cudaMemcpyHostToDevice));
    }
    return MOC_OK;
}

// Layouts for the sequence-per-lane kernel, one per group size g = 32, 16, 8 (S = 1, 2, 4 sub-lanes).
// Nodes in order of falling out-degree (a sink counts one: its made-up successor), S consecutive
// nodes form a bundle and share a row count; entry (k, h) of a bundle is the byte offset of the
// word row of the k-th successor of its h-th node, the node's own row once its list is used up.
int build_lane_layouts(moc_graph* g, const std::vector<int32_t>& succ_start, const std::vector<int32_t>& succ,
                       const int64_t* m, const std::vector<int32_t>& m32) {
    const int32_t n = g->n;
    if (n >= 4096) return MOC_OK;                       // the count of two-copy nodes has 12 bits
    auto deg = [&](int32_t v) { return std::max(1, succ_start[v + 1] - succ_start[v]); };
    std::vector<int32_t> order((size_t)n);
    for (int32_t v = 0; v < n; ++v) order[v] = v;
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return deg(x) > deg(y); });
    if (deg(order[0]) > 255) return MOC_OK;
    for (int li = 0; li < 3; ++li) {
        const int lg = 5 - li, gsz = 1 << lg, S = 32 >> lg;
        LaneLayout& L = g->lane[li];
        const int32_t nb = (n + S - 1) / S;
        std::vector<int32_t> node((size_t)nb * S, -1);
        for (int32_t i = 0; i < n; ++i) node[i] = order[i];
        std::vector<uint32_t> rec32(node.size() * 8, 0u), rec64(node.size() * 8, 0u);
        std::vector<uint32_t> se;
        const uint32_t row_b = moc::lane_word_row(gsz);
        const uint32_t t_row = 0u - moc::lane_special(gsz), one_row = t_row + row_b;   // relative to the first node row
        for (int32_t bd = 0; bd < nb; ++bd) {
            int rows = 0;
            for (int h = 0; h < S; ++h)
                if (node[(size_t)bd * S + h] >= 0) rows = std::max(rows, deg(node[(size_t)bd * S + h]));
            const uint32_t first = (uint32_t)se.size();
            for (int k = 0; k < rows; ++k)
                for (int h = 0; h < S; ++h) {
                    const int32_t v = node[(size_t)bd * S + h];
                    uint32_t off;
                    if (v < 0) off = one_row;
                    else if (k < succ_start[v + 1] - succ_start[v]) off = (uint32_t)succ[succ_start[v] + k] * row_b;
                    else if (k == 0) off = t_row;                    // a sink: the word that holds T
                    else off = (uint32_t)v * row_b;
                    se.push_back(off);
                }
            for (int h = 0; h < S; ++h) {
                const size_t r = (size_t)bd * S + h;
                const int32_t v = node[r];
                const uint64_t mv = v >= 0 ? (uint64_t)m[v] : 0;
                rec32[8 * r + 0] = rec64[8 * r + 0] = v >= 0 ? (uint32_t)v * row_b : one_row;
                rec32[8 * r + 1] = rec64[8 * r + 1] = (4u * (first + (uint32_t)h)) | ((uint32_t)rows << 24);
                rec32[8 * r + 2] = v >= 0 ? (uint32_t)m32[v] : 0u;
                rec32[8 * r + 3] = 0u - rec32[8 * r + 2];
                rec64[8 * r + 2] = (uint32_t)(mv & 0xFFFFFFFFu);
                rec64[8 * r + 3] = (uint32_t)(mv >> 32);
                rec64[8 * r + 6] = (uint32_t)((0 - mv) & 0xFFFFFFFFu);
                rec64[8 * r + 7] = (uint32_t)((0 - mv) >> 32);
            }
        }
        while (se.size() % 4) se.push_back(one_row);
        if (se.empty()) se.assign(4, one_row);
        if (se.size() * 4 + 64 >= (size_t(1) << 24)) continue;
        cudaError_t e = cudaMalloc(&L.d_rec32, rec32.size() * 4);
        if (e == cudaSuccess) e = cudaMalloc(&L.d_rec64, rec64.size() * 4);
        if (e == cudaSuccess) e = cudaMalloc((void**)&L.d_succ, se.size() * 4);
        if (e == cudaSuccess) e = cudaMemcpy(L.d_succ, se.data(), se.size() * 4, cudaMemcpyHostToDevice);
        if (e != cudaSuccess)
            return fail(e == cudaErrorMemoryAllocation ? MOC_ERR_NOMEM : MOC_ERR_CUDA, "moc_graph_create: %s", cudaGetErrorString(e));
        L.n_bundles = nb;
        L.succ_len = (int64_t)se.size();
        L.h_node = node;
        L.h_rec32 = rec32;
        L.h_rec64 = rec64;
        L.ok = true;
    }
    return upload_lane_rec(g);
}

// Layout for the block-per-sequence kernel: the nodes in order of falling out-degree (a sink counts one:
// its made-up successor n + 1) with the place of their successor lists, and the lists as 16-bit ids.
int build_quad_layout(moc_graph* g, const std::vector<int32_t>& succ_start, const std::vector<int32_t>& succ,
                      const int64_t* m, const std::vector<int32_t>& m32) {
    const int32_t n = g->n;
    if (n > 32000) return MOC_OK;
    auto deg = [&](int32_t v) { return std::max(1, succ_start[v + 1] - succ_start[v]); };
    std::vector<int32_t> order((size_t)n);
    for (int32_t v = 0; v < n; ++v) order[v] = v;
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return deg(x) > deg(y); });
    if (deg(order[0]) > 65535) return MOC_OK;
    for (int wide = 0; wide < 2; ++wide) {
        std::vector<uint32_t> rec((size_t)n * 8, 0u);
        std::vector<uint16_t> rest;
        for (int32_t i = 0; i < n; ++i) {
            const int32_t v = order[i];
            std::vector<uint16_t> ids;
            if (succ_start[v + 1] == succ_start[v]) ids.push_back((uint16_t)(n + 1));
            for (int32_t e = succ_start[v]; e < succ_start[v + 1]; ++e) ids.push_back((uint16_t)succ[e]);
            uint32_t* r = &rec[(size_t)i * 8];
            r[0] = (uint32_t)v | ((uint32_t)ids.size() << 16);
            r[1] = (uint32_t)rest.size();
            if (wide) {
                r[2] = (uint32_t)((uint64_t)m[v] & 0xFFFFFFFFu);
                r[3] = (uint32_t)((uint64_t)m[v] >> 32);
            } else {
                r[2] = (uint32_t)m32[v];
            }
            for (size_t k = 0; k < ids.size(); ++k) {
                if (k < 8) r[4 + k / 2] |= (uint32_t)ids[k] << (16 * (k & 1));
                else rest.push_back(ids[k]);
            }
        }
        uint4** dst = wide ? &g->d_order64 : &g->d_order32;
        MOC_CUDA(cudaMalloc((void**)dst, rec.size() * 4));
        MOC_CUDA(cudaMemcpy(*dst, rec.data(), rec.size() * 4, cudaMemcpyHostToDevice));
        if (!wide) {
            MOC_CUDA(cudaMalloc((void**)&g->d_succ16, std::max<size_t>(rest.size() * 2, 16)));
            if (!rest.empty()) MOC_CUDA(cudaMemcpy(g->d_succ16, rest.data(), rest.size() * 2, cudaMemcpyHostToDevice));
        }
    }
    return MOC_OK;
}

moc::EvalParams base_params(const moc_graph* g, const Plan& pl) {
    moc::EvalParams p{};
    p.g.n = g->n;
    p.g.C = g->C;
    p.g.succ_start = g->d_succ_start;
    p.g.succ = g->d_succ;
    p.g.w = g->d_w;
    p.g.m = pl.wide ? (const void*)g->d_m64 : (const void*)g->d_m32;
    p.g.cap = g->d_cap;
    p.cnt_bytes = pl.cnt_bytes;
    p.occ_bytes = pl.occ_bytes;
    p.delta_bytes = pl.delta_bytes;
    p.group_bytes = pl.group_bytes;
    return p;
}

// Enqueues the evaluation of plan `pl`.  With `offs` the evaluation kernel reads the row offsets
// from that array, which the offsets kernel fills first from the lengths when `fill_offs` is set
// (packed rows) and which the caller has filled otherwise; with offs == nullptr (only the
// warp-per-sequence kernel can do that) the evaluation kernel finds the packed rows itself.
int enqueue_eval(const moc_graph* g, const Plan& pl, int64_t* offs, bool fill_offs, const int32_t* seqs, const int32_t* lens,
                 int32_t B, int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible,
                 cudaStream_t st) {
    int grid = (int)std::min<int64_t>(pl.grid, ((int64_t)B + pl.gpc - 1) / pl.gpc);   // lane path: gpc = sequences per group
    int block = pl.block;
    size_t smem = pl.smem;
    if (pl.pair) {
        // Shape of this launch.  A warp works through its sequences one after the other, so a launch
        // takes ceil(sequences per block / warps per block) rounds, and a round costs about as much as
        // the SM has warps (the kernel is bound by on-chip throughput) but never less than a round of a
        // half-empty SM.  Pick the warps per block and blocks per SM with the least rounds x warps.
        int64_t best_cost = INT64_MAX;
        int best_w = pl.gpc, best_nb = std::max(1, pl.grid / std::max(1, pl.sm_count));
        for (int wpb = 4; wpb <= 16; ++wpb) {
            const int nb = pl.pair_nb[wpb];
            if (nb < 1) continue;
            const int64_t blocks = (int64_t)pl.sm_count * nb;
            const int64_t per_block = (B + blocks - 1) / blocks;
            const int64_t rounds = (per_block + wpb - 1) / wpb;
            const int64_t cost = rounds * std::max(wpb * nb, 16);
            // equal cost: fewer, larger blocks (every block stages the graph in its shared memory)
            if (cost < best_cost || (cost == best_cost && nb <= best_nb)) {
                best_cost = cost;
                best_w = wpb;
                best_nb = nb;
            }
        }
        block = 32 * best_w;
        smem = pl.pair_graph_b + (size_t)best_w * pl.pair_warp_b;
        grid = (int)std::min<int64_t>((int64_t)pl.sm_count * best_nb, ((int64_t)B + best_w - 1) / best_w);
    }
    if (offs && fill_offs) {
        moc::offsets_kernel<<<(B + moc::kOffsTile - 1) / moc::kOffsTile, moc::kOffsThreads, 0, st>>>(lens, B, offs);
        ++g_launches;
    }
    if (g->ev_before) MOC_CUDA(cudaEventRecord(g->ev_before, st));
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    if (pl.quad) {
        moc::QuadParams q{};
        q.n = g->n;
        q.C = g->C;
        q.max_T = g->C * g->n;
        q.B = B;
        q.M = M;
        q.order = pl.wide ? g->d_order64 : g->d_order32;
        q.succ = g->d_succ16;
        q.m = pl.wide ? (const void*)g->d_m64 : (const void*)g->d_m32;
        q.w = g->d_w;
        q.cap = g->d_cap;
        q.seqs = seqs;
        q.lens = lens;
        q.offs = offs;
        q.out_peak = out_peak;
        q.out_dur = out_dur;
        q.out_status = out_feasible;
        q.word_bytes = pl.quad_word_b;
        q.cnt_bytes = pl.quad_cnt_b;
        MOC_CUDA(cudaLaunchKernelEx(&cfg, pl.quad_fn, q));
    } else if (pl.lane) {
        const LaneLayout& L = g->lane[5 - pl.lane_lg];
        moc::LaneParams q{};
        q.n = g->n;
        q.max_T = g->C * g->n;
        q.B = B;
        q.n_bundles = L.n_bundles;
        q.M = M;
        q.base_dur = g->sum_w;
        q.rec = (const uint4*)(pl.wide ? L.d_rec64 : L.d_rec32);
        q.succ = L.d_succ;
        q.seqs = seqs;
        q.lens = lens;
        q.offs = offs;
        q.out_peak = out_peak;
        q.out_dur = out_dur;
        q.out_status = out_feasible;
        q.rec_bytes = pl.lane_rec_b; q.succ_bytes = pl.lane_succ_b;
        q.word_bytes = pl.lane_word_b; q.delta_bytes = pl.lane_delta_b;
        MOC_CUDA(cudaLaunchKernelEx(&cfg, pl.lane_fn, q));
    } else if (pl.pair) {
        moc::PairParams q{};
        q.n = g->n;
        q.n_tiles = g->n_tiles;
        q.max_T = g->C * g->n;
        q.rec = pl.wide ? g->d_rec64 : g->d_rec32;
        q.wslot = (const uint64_t*)g->d_wslot;
        q.sell = g->d_sell;
        q.base_dur = g->sum_w;
        q.seqs = seqs;
        q.lens = lens;
        q.offs = offs;
        q.B = B;
        q.M = M;
        q.out_peak = out_peak;
        q.out_dur = out_dur;
        q.out_status = out_feasible;
        q.rec_bytes = pl.rec_bytes; q.w_bytes = pl.w_bytes; q.sell_bytes = pl.sell_bytes;
        q.word_bytes = pl.word_bytes; q.delta_bytes = pl.delta_bytes;
        MOC_CUDA(cudaLaunchKernelEx(&cfg, pl.pair_fn, q));
    } else {
        moc::EvalParams p = base_params(g, pl);
        p.seqs = seqs;
        p.lens = lens;
        p.offs = offs;
        p.B = B;
        p.M = M;
        p.out_peak = out_peak;
        p.out_dur = out_dur;
        p.out_status = out_feasible;
        p.gstate = g->d_state;
        MOC_CUDA(cudaLaunchKernelEx(&cfg, pl.fn, p));
    }
    ++g_launches;
    MOC_CUDA(cudaGetLastError());
    if (g->ev_after) MOC_CUDA(cudaEventRecord(g->ev_after, st));
    return MOC_OK;
}

// Each block of the self-addressing kernel re-reads the lengths in front of its range: worth it
// while that redundant traffic (grid * B/2 * 4 bytes from L2) stays small next to a second launch.
bool rows_without_scratch(const Plan& pl, int32_t B) {
    return (pl.pair || pl.lane) && (int64_t)pl.grid * B * 2 <= (int64_t)16 << 20;
}

int launch_eval(const moc_graph* g, const int32_t* seqs, const int32_t* lens, int32_t B, int64_t M,
                int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible, cudaStream_t st) {
    if (!g->plan_eval.valid) {
        int rc = make_plan(g, false, &g->plan_eval);
        if (rc != MOC_OK) return rc;
    }
    const Plan& pl = g->plan_eval;
    if (rows_without_scratch(pl, B))
        return enqueue_eval(g, pl, nullptr, false, seqs, lens, B, M, out_peak, out_dur, out_feasible, st);
    int rc = ensure((void**)&g->d_offs, &g->offs_cap, ((size_t)B + 1) * sizeof(int64_t));
    if (rc != MOC_OK) return rc;
    if (pl.global_state) {
        rc = ensure((void**)&g->d_state, &g->state_cap, (size_t)pl.grid * pl.group_bytes);
        if (rc != MOC_OK) return rc;
    }
    return enqueue_eval(g, pl, g->d_offs, true, seqs, lens, B, M, out_peak, out_dur, out_feasible, st);
}

}  // namespace

namespace moc_host {
int eval_rows(const moc_graph* g, const int64_t* offs, const int32_t* seqs, const int32_t* lens, int32_t B,
              int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible, cudaStream_t st) {
    if (!g->plan_eval.valid) {
        int rc = make_plan(g, false, &g->plan_eval);
        if (rc != MOC_OK) return rc;
    }
    const Plan& pl = g->plan_eval;
    if (pl.global_state) {
        int rc = ensure((void**)&g->d_state, &g->state_cap, (size_t)pl.grid * pl.group_bytes);
        if (rc != MOC_OK) return rc;
    }
    return enqueue_eval(g, pl, const_cast<int64_t*>(offs), false, seqs, lens, B, M, out_peak, out_dur, out_feasible, st);
}
}  // namespace moc_host

extern "C" {

static int upload_wslot(moc_graph* g);

const char* moc_last_error(void) { return g_err; }
int moc_last_launch_count(void) { return g_launches; }

int moc_graph_create(int32_t n, int64_t n_edges, const int32_t* edges, const int64_t* w,
                     const int64_t* m, moc_graph** out) {
    g_err[0] = 0;
    if (out) *out = nullptr;
    if (!out || !w || !m || n < 1 || n_edges < 0 || (n_edges > 0 && !edges))
        return fail(MOC_ERR_ARG, "moc_graph_create: null pointer, n < 1 or n_edges < 0");
    if (n > (1 << 27) || n_edges > (int64_t)INT32_MAX - 1)
        return fail(MOC_ERR_ARG, "moc_graph_create: n > 2^27 or n_edges >= 2^31-1");
    int64_t sum_w = 0, sum_m = 0;
    const int64_t lim = (int64_t(1) << 62) / 8;
    for (int32_t v = 0; v < n; ++v) {
        if (w[v] < 0 || m[v] < 0) return fail(MOC_ERR_OVERFLOW, "negative weight at node %d", v);
        if (w[v] >= lim - sum_w || m[v] >= lim - sum_m)
            return fail(MOC_ERR_OVERFLOW, "8*sum(w) or 8*sum(m) reaches 2^62");
        sum_w += w[v];
        sum_m += m[v];
    }
    std::vector<uint64_t> keys;
    try {
        keys.reserve((size_t)n_edges);
        for (int64_t e = 0; e < n_edges; ++e) {
            const int32_t u = edges[2 * e], v = edges[2 * e + 1];
            if (u < 0 || u >= n || v < 0 || v >= n)
                return fail(MOC_ERR_RANGE, "edge %lld = (%d,%d) outside [0,%d)", (long long)e, u, v, n);
            if (u == v) return fail(MOC_ERR_CYCLE, "self-loop at node %d", u);
            keys.push_back(((uint64_t)(uint32_t)u << 32) | (uint32_t)v);
        }
        std::sort(keys.begin(), keys.end());
        keys.erase(std::unique(keys.begin(), keys.end()), keys.end());
    } catch (const std::bad_alloc&) {
        return fail(MOC_ERR_NOMEM, "host allocation failed");
    }
    const int64_t ne = (int64_t)keys.size();
    std::vector<int32_t> succ_start, succ, indeg, queue, m32;
    try {
        succ_start.assign((size_t)n + 1, 0);
        succ.resize((size_t)std::max<int64_t>(ne, 1));
        indeg.assign((size_t)n, 0);
        m32.resize((size_t)n);
        for (int64_t e = 0; e < ne; ++e) {
            const int32_t u = (int32_t)(keys[e] >> 32), v = (int32_t)(keys[e] & 0xFFFFFFFFu);
            succ_start[u + 1]++;
            succ[e] = v;  // keys are sorted by (u, v): already grouped by producer
            indeg[v]++;
        }
        for (int32_t v = 0; v < n; ++v) succ_start[v + 1] += succ_start[v];
        // Kahn: the graph is a DAG iff every node gets removed
        queue.reserve((size_t)n);
        for (int32_t v = 0; v < n; ++v)
            if (indeg[v] == 0) queue.push_back(v);
        for (size_t h = 0; h < queue.size(); ++h) {
            const int32_t u = queue[h];
            for (int32_t e = succ_start[u]; e < succ_start[u + 1]; ++e)
                if (--indeg[succ[e]] == 0) queue.push_back(succ[e]);
        }
        if ((int32_t)queue.size() != n) return fail(MOC_ERR_CYCLE, "the edges contain a directed cycle");
        for (int32_t v = 0; v < n; ++v) m32[v] = (int32_t)std::min<int64_t>(m[v], INT32_MAX);
    } catch (const std::bad_alloc&) {
        return fail(MOC_ERR_NOMEM, "host allocation failed");
    }

    moc_graph* g = new (std::nothrow) moc_graph();
    if (!g) return fail(MOC_ERR_NOMEM, "host allocation failed");
    try {
        g->h_w.assign(w, w + n);
    } catch (const std::bad_alloc&) {
        delete g;
        return fail(MOC_ERR_NOMEM, "host allocation failed");
    }
    g->n = n;
    g->n_edges = ne;
    g->sum_m = sum_m;
    g->sum_w = sum_w;
    int rc = MOC_OK;
    cudaError_t e = cudaGetDevice(&g->device);
    int smem = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g->sm_count, cudaDevAttrMultiProcessorCount, g->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, g->device);
    g->smem_optin = (size_t)smem;
    auto up = [&](void** dst, const void* src, size_t bytes) {
        if (e != cudaSuccess) return;
        e = cudaMalloc(dst, std::max<size_t>(bytes, 16));
        if (e == cudaSuccess && bytes && src) e = cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice);
    };
    up((void**)&g->d_succ_start, succ_start.data(), ((size_t)n + 1) * 4);
    up((void**)&g->d_succ, succ.data(), (size_t)ne * 4);
    {
        // predecessor lists (grouped by consumer) and the total output size of the sinks
        std::vector<int32_t> pred_start, pred;
        try {
            pred_start.assign((size_t)n + 1, 0);
            pred.resize((size_t)std::max<int64_t>(ne, 1));
            for (int64_t k = 0; k < ne; ++k) pred_start[(keys[k] & 0xFFFFFFFFu) + 1]++;
            for (int32_t v = 0; v < n; ++v) g->max_indeg = std::max(g->max_indeg, pred_start[v + 1]);
            for (int32_t v = 0; v < n; ++v) pred_start[v + 1] += pred_start[v];
            std::vector<int32_t> fill(pred_start.begin(), pred_start.end() - 1);
            for (int64_t k = 0; k < ne; ++k) pred[fill[keys[k] & 0xFFFFFFFFu]++] = (int32_t)(keys[k] >> 32);
        } catch (const std::bad_alloc&) {
            moc_graph_destroy(g);
            return fail(MOC_ERR_NOMEM, "host allocation failed");
        }
        for (int32_t v = 0; v < n; ++v)
            if (succ_start[v + 1] == succ_start[v]) g->sink_m += m[v];
        up((void**)&g->d_pred_start, pred_start.data(), ((size_t)n + 1) * 4);
        up((void**)&g->d_pred, pred.data(), (size_t)ne * 4);
    }
    up((void**)&g->d_w, w, (size_t)n * 8);
    up((void**)&g->d_m64, m, (size_t)n * 8);
    up((void**)&g->d_m32, m32.data(), (size_t)n * 4);
    if (n <= 16000) {
        // Layout for the warp-per-sequence kernel.  Lane l serves the nodes with id = l (mod 32);
        // each residue class is sorted by out-degree (descending, ties by id); half j holds the
        // j-th node of every class, a tile is two halves.  A tile stores, row by row, the word
        // offsets (4 * id) of its nodes' successors, two halves packed per 32-bit entry, padded with
        // the offset of a dummy word (4 * n).  Within a half the order of each node's successors
        // is chosen greedily so that the 32 words a row touches fall in different banks where
        // possible.  Skipped when padding would more than double the storage (a few very high
        // degrees): such graphs use the general kernel.
        try {
            auto deg = [&](int32_t v) { return succ_start[v + 1] - succ_start[v]; };
            const int32_t n_halves = 2 * ((n + 63) / 64), n_tiles = n_halves / 2;
            std::vector<int32_t> slot((size_t)n_halves * 32, -1);  // node at (half, lane) or -1
            for (int32_t l = 0; l < 32; ++l) {
                std::vector<int32_t> cls;
                for (int32_t v = l; v < n; v += 32) cls.push_back(v);
                std::stable_sort(cls.begin(), cls.end(), [&](int32_t x, int32_t y) { return deg(x) > deg(y); });
                for (size_t j = 0; j < cls.size(); ++j) slot[j * 32 + l] = cls[j];
            }
            std::vector<int32_t> rows((size_t)n_tiles, 0);
            int64_t sell_len = 0;
            for (int32_t d = 0; d < n_tiles; ++d) {
                for (int32_t s = 0; s < 64; ++s)
                    if (slot[(size_t)d * 64 + s] >= 0)
                        rows[d] = std::max(rows[d], std::max(1, deg(slot[(size_t)d * 64 + s])));  // a sink gets one entry
                sell_len += 32 * (int64_t)rows[d];
            }
            int32_t max_rows = 0;
            for (int32_t d = 0; d < n_tiles; ++d) max_rows = std::max(max_rows, rows[d]);
            if (sell_len <= 2 * ne + 4096 && sell_len < (1 << 20) && max_rows < (1 << 12) && 4 * ((int64_t)n + 3) < 65536) {
                const uint32_t word_b = (uint32_t)align16(4 * ((size_t)n + 2));   // the constant word (1, 1) sits right after the words
                std::vector<uint32_t> rec32((size_t)n_halves * 32 * 2), rec64((size_t)n_halves * 32 * 4, 0u);
                // entry (row k, lane l) of a tile: word of the k-th successor of the node in half 0 | same for half 1 << 16;
                // a list that is used up continues with the node's own word
                std::vector<uint32_t> sell((size_t)std::max<int64_t>(sell_len, 1), word_b | (word_b << 16));
                auto own_word = [&](int32_t v) { return v >= 0 ? 4u * (uint32_t)v : word_b; };
                for (size_t r = 0; r < slot.size(); ++r) {
                    const int32_t v = slot[r];
                    const uint32_t x = own_word(v) | ((uint32_t)rows[r / 64] << 16);
                    const uint64_t mv = v >= 0 ? (uint64_t)m[v] : 0;
                    rec32[2 * r + 0] = x;
                    rec32[2 * r + 1] = v >= 0 ? (uint32_t)m32[v] : 0u;
                    rec64[4 * r + 0] = x;
                    rec64[4 * r + 2] = (uint32_t)(mv & 0xFFFFFFFFu);
                    rec64[4 * r + 3] = (uint32_t)(mv >> 32);
                }
                uint32_t pos = 0;
                std::vector<std::vector<int32_t>> rem(32);
                for (int32_t d = 0; d < n_tiles; ++d) {
                    for (int32_t h = 0; h < 2; ++h) {
                        std::vector<int32_t> lanes;
                        for (int32_t l = 0; l < 32; ++l) {
                            const int32_t v = slot[((size_t)2 * d + h) * 32 + l];
                            rem[l].clear();
                            if (v >= 0) rem[l].assign(succ.begin() + succ_start[v], succ.begin() + succ_start[v + 1]);
                            if (v >= 0 && rem[l].empty()) rem[l].push_back(n + 1);  // sink: the word that holds T
                            lanes.push_back(l);
                            for (int32_t k = 0; k < rows[d]; ++k) {
                                uint32_t& e = sell[(size_t)pos + 32 * (size_t)k + l];
                                e = h == 0 ? ((e & 0xFFFF0000u) | own_word(v)) : ((e & 0x0000FFFFu) | (own_word(v) << 16));
                            }
                        }
                        for (int32_t k = 0; k < rows[d]; ++k) {
                            int used[32] = {0};
                            for (int32_t l = 0; l < 32; ++l)
                                if (rem[l].empty()) used[l]++;   // reads its own word, which lies in bank l
                            std::stable_sort(lanes.begin(), lanes.end(),
                                             [&](int32_t x, int32_t y) { return rem[x].size() > rem[y].size(); });
                            for (int32_t l : lanes) {
                                if (rem[l].empty()) continue;  // stays the own word
                                const bool forced = (int32_t)rem[l].size() >= rows[d] - k;
                                int pick = -1;
                                for (size_t c = 0; c < rem[l].size(); ++c)
                                    if (!used[rem[l][c] & 31]) { pick = (int)c; break; }
                                if (pick < 0 && !forced) continue;  // wait for a row where its bank is free
                                if (pick < 0) pick = 0;
                                used[rem[l][pick] & 31]++;
                                uint32_t& e = sell[(size_t)pos + 32 * (size_t)k + l];
                                const uint32_t off = 4u * (uint32_t)rem[l][pick];
                                e = h == 0 ? ((e & 0xFFFF0000u) | off) : ((e & 0x0000FFFFu) | (off << 16));
                                rem[l].erase(rem[l].begin() + pick);
                            }
                        }
                    }
                    pos += 32 * (uint32_t)rows[d];
                }
                g->sell_len = (int32_t)sell_len;
                g->h_slot = slot;
                g->n_tiles = n_tiles;
                up(&g->d_rec32, rec32.data(), rec32.size() * 4);
                up(&g->d_rec64, rec64.data(), rec64.size() * 4);
                up((void**)&g->d_wslot, nullptr, slot.size() * 8);
                up((void**)&g->d_sell, sell.data(), sell.size() * 4);
            }
        } catch (const std::bad_alloc&) {
            moc_graph_destroy(g);
            return fail(MOC_ERR_NOMEM, "host allocation failed");
        }
    }
    if (e != cudaSuccess) {
        rc = fail(e == cudaErrorMemoryAllocation ? MOC_ERR_NOMEM : MOC_ERR_CUDA,
                  "moc_graph_create: %s", cudaGetErrorString(e));
        cudaGetLastError();
        moc_graph_destroy(g);
        return rc;
    }
    try {
        rc = build_lane_layouts(g, succ_start, succ, m, m32);
        if (rc == MOC_OK) rc = upload_wslot(g);
        if (rc == MOC_OK) rc = build_quad_layout(g, succ_start, succ, m, m32);
    } catch (const std::bad_alloc&) {
        rc = fail(MOC_ERR_NOMEM, "host allocation failed");
    }
    if (rc != MOC_OK) {
        cudaGetLastError();
        moc_graph_destroy(g);
        return rc;
    }
    *out = g;
    return MOC_OK;
}

int moc_graph_set_max_copies(moc_graph* g, int32_t C) {
    g_err[0] = 0;
    if (!g || C < 1 || C > MOC_MAX_COPIES) return fail(MOC_ERR_ARG, "moc_graph_set_max_copies: C must be 1..%d", MOC_MAX_COPIES);
    if (!g->h_cap.empty()) {   // caps refer to the old C: back to a uniform cap
        int rc = moc_graph_set_node_caps(g, nullptr);
        if (rc != MOC_OK) return rc;
    }
    g->C = C;
    ++g->generation;
    g->plan_eval.valid = false;
    g->plan_profile.valid = false;
    return MOC_OK;
}

// Uploads the slot durations of the warp-per-sequence layout: w | 1 << 48 (counts the node when it has
// two copies) | 1 << 63 for nodes whose cap C_v is 1.
static int upload_wslot(moc_graph* g) {
    if (!g->d_wslot) return MOC_OK;
    std::vector<uint64_t> wslot(g->h_slot.size());
    for (size_t r = 0; r < wslot.size(); ++r) {
        const int32_t v = g->h_slot[r];
        uint64_t x = 0;
        if (v >= 0) {
            x = (uint64_t)g->h_w[v] | (uint64_t(1) << moc::kPairCntShift);
            if (!g->h_cap.empty() && g->h_cap[v] == 1) x |= uint64_t(1) << 63;
        }
        wslot[r] = x;
    }
    MOC_CUDA(cudaMemcpy(g->d_wslot, wslot.data(), wslot.size() * 8, cudaMemcpyHostToDevice));
    return MOC_OK;
}

int moc_graph_set_node_caps(moc_graph* g, const int32_t* caps) {
    g_err[0] = 0;
    if (!g) return fail(MOC_ERR_ARG, "moc_graph_set_node_caps: null handle");
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    // work queued on any stream may still read the old caps
    MOC_CUDA(cudaDeviceSynchronize());
    try {
        if (!caps) {
            g->h_cap.clear();
        } else {
            for (int32_t v = 0; v < g->n; ++v)
                if (caps[v] < 1 || caps[v] > g->C)
                    return fail(MOC_ERR_ARG, "moc_graph_set_node_caps: cap %d of node %d outside [1, C = %d]", caps[v], v, g->C);
            g->h_cap.assign(caps, caps + g->n);
        }
    } catch (const std::bad_alloc&) {
        return fail(MOC_ERR_NOMEM, "host allocation failed");
    }
    ++g->generation;
    if (caps) {
        if (!g->d_cap) MOC_CUDA(cudaMalloc((void**)&g->d_cap, std::max<size_t>((size_t)g->n * 4, 16)));
        MOC_CUDA(cudaMemcpy(g->d_cap, caps, (size_t)g->n * 4, cudaMemcpyHostToDevice));
    } else if (g->d_cap) {
        MOC_CUDA(cudaFree(g->d_cap));
        g->d_cap = nullptr;
    }
    int rc = upload_wslot(g);
    if (rc != MOC_OK) return rc;
    return upload_lane_rec(g);
}

int moc_graph_set_kernel(moc_graph* g, int32_t kind, int32_t a, int32_t b) {
    g_err[0] = 0;
    if (!g) return fail(MOC_ERR_ARG, "moc_graph_set_kernel: null handle");
    bool ok = false;
    switch (kind) {
        case MOC_KERNEL_AUTO: ok = a == 0 && b == 0; break;
        case MOC_KERNEL_GROUP:
            ok = (a == 0 || a == 32 || a == 64 || a == 128 || a == 256 || a == 512 || a == 1024) && b >= 0 && b <= 32 &&
                 !(a && b && a * b > 1024);
            break;
        case MOC_KERNEL_WARP: ok = a == 0 && (b == 0 || (b >= 4 && b <= 16)); break;
        case MOC_KERNEL_BLOCK: ok = (a == 0 || (a >= 64 && a <= 1024 && a % 32 == 0)) && b == 0; break;
        case MOC_KERNEL_LANE: ok = (a == 0 || a == 8 || a == 16 || a == 32) && (b == 0 || (b >= 8 && b <= 32 && b % 8 == 0)); break;
        default: break;
    }
    if (!ok) return fail(MOC_ERR_ARG, "moc_graph_set_kernel: unsupported kind or shape (%d, %d, %d)", kind, a, b);
    g->want_kind = kind;
    g->want_a = a;
    g->want_b = b;
    g->want_G = kind == MOC_KERNEL_GROUP ? a : 0;
    g->want_gpc = (kind == MOC_KERNEL_GROUP || kind == MOC_KERNEL_WARP) ? b : 0;
    g->plan_eval.valid = false;
    return MOC_OK;
}

int moc_graph_set_launch(moc_graph* g, int32_t tps, int32_t spb) {
    g_err[0] = 0;
    const bool ok_g = tps == 0 || tps == 32 || tps == 64 || tps == 128 || tps == 256 || tps == 512 || tps == 1024;
    if (!g || !ok_g || spb < 0 || spb > 32 || (tps && spb && tps * spb > 1024))
        return fail(MOC_ERR_ARG, "moc_graph_set_launch: unsupported shape (%d threads x %d sequences)", tps, spb);
    g->want_kind = MOC_KERNEL_AUTO;
    g->want_a = g->want_b = 0;
    g->want_G = tps;
    g->want_gpc = spb;
    g->plan_eval.valid = false;
    return MOC_OK;
}

int moc_graph_set_timing_events(moc_graph* g, void* before, void* after) {
    g_err[0] = 0;
    if (!g || ((before == nullptr) != (after == nullptr)))
        return fail(MOC_ERR_ARG, "moc_graph_set_timing_events: null handle, or only one of the two events given");
    g->ev_before = (cudaEvent_t)before;
    g->ev_after = (cudaEvent_t)after;
    return MOC_OK;
}

void moc_graph_destroy(moc_graph* g) {
    if (!g) return;
    DeviceGuard dg(g->device);
    cudaFree(g->d_succ_start);
    cudaFree(g->d_succ);
    cudaFree(g->d_pred_start);
    cudaFree(g->d_pred);
    cudaFree(g->d_w);
    cudaFree(g->d_m64);
    cudaFree(g->d_m32);
    cudaFree(g->d_rec32);
    cudaFree(g->d_rec64);
    cudaFree(g->d_wslot);
    cudaFree(g->d_cap);
    cudaFree(g->d_sell);
    cudaFree(g->d_offs);
    cudaFree(g->d_state);
    cudaFree(g->d_stage_seqs);
    cudaFree(g->d_stage_u16);
    cudaFree(g->d_stage_io);
    cudaFree(g->d_order32);
    cudaFree(g->d_order64);
    cudaFree(g->d_succ16);
    if (g->h_stage) cudaFreeHost(g->h_stage);
    if (g->copy_stream) {
        cudaStreamDestroy(g->copy_stream);
        for (cudaEvent_t ev : g->chunk_ev)
            if (ev) cudaEventDestroy(ev);
    }
    for (int li = 0; li < 3; ++li) {
        cudaFree(g->lane[li].d_rec32);
        cudaFree(g->lane[li].d_rec64);
        cudaFree(g->lane[li].d_succ);
    }
    delete g;
}

int moc_graph_info(const moc_graph* g, int32_t* n, int64_t* n_edges, int32_t* C, int32_t* wide) {
    g_err[0] = 0;
    if (!g) return fail(MOC_ERR_ARG, "moc_graph_info: null handle");
    if (n) *n = g->n;
    if (n_edges) *n_edges = g->n_edges;
    if (C) *C = g->C;
    if (wide) *wide = g->sum_m > (int64_t)INT32_MAX / g->C ? 1 : 0;
    return MOC_OK;
}

int moc_eval_batch(const moc_graph* g, const int32_t* seqs, const int32_t* lens, int32_t B, int64_t M,
                   int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible, void* stream) {
    g_err[0] = 0;
    g_launches = 0;
    if (!g || B < 0) return fail(MOC_ERR_ARG, "moc_eval_batch: null handle or B < 0");
    if (B == 0) return MOC_OK;
    if (!seqs || !lens || !out_peak || !out_dur || !out_feasible)
        return fail(MOC_ERR_ARG, "moc_eval_batch: null array");
    if (reinterpret_cast<uintptr_t>(seqs) & 3) return fail(MOC_ERR_ARG, "moc_eval_batch: seqs not 4-byte aligned");
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    return launch_eval(g, seqs, lens, B, M, out_peak, out_dur, out_feasible, (cudaStream_t)stream);
}

// Host entry points.  The batch is cut into chunks of whole sequences; a copy stream owned by the
// handle brings chunk k + 1 to the device while the caller's stream evaluates chunk k (one
// cudaMemcpyAsync per chunk and an event between the two streams), and the three result arrays come
// back with one copy into a pinned staging block, from which they are handed to the caller's arrays.
namespace {
constexpr int kHostChunks = 4;

int host_streams(const moc_graph* g) {
    if (g->copy_stream) return MOC_OK;
    MOC_CUDA(cudaStreamCreateWithFlags(&g->copy_stream, cudaStreamNonBlocking));
    for (int k = 0; k < kHostChunks + 1; ++k) MOC_CUDA(cudaEventCreateWithFlags(&g->chunk_ev[k], cudaEventDisableTiming));   // chunk_ev has room for 9
    return MOC_OK;
}

// ids: host array of `need` node ids, 4 bytes each (wide_ids) or 2 bytes each.
int eval_host(const moc_graph* g, const void* ids, bool wide_ids, int64_t n_steps, const int32_t* lens, int32_t B,
              int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible, cudaStream_t st, const char* who) {
    // chunk boundaries: about equal numbers of steps, whole sequences
    int64_t need = 0;
    for (int32_t b = 0; b < B; ++b) need += lens[b] > 0 ? lens[b] : 0;
    if (need > n_steps) return fail(MOC_ERR_ARG, "%s: lens sum to %lld > n_steps %lld", who, (long long)need, (long long)n_steps);
    int32_t cb[kHostChunks + 1];
    int64_t co[kHostChunks + 1];
    int n_chunks = 0;
    {
        // Chunks of 1/2, 1/4, 1/8, 1/8 of the steps (whole sequences): the evaluation of all but the last
        // chunk hides behind the copy of the next, and the last one is small.  Short batches go in one piece.
        const int want = need >= (int64_t(1) << 21) ? kHostChunks : 1;
        int64_t run = 0, bound = need - need / 2;
        cb[0] = 0;
        co[0] = 0;
        for (int32_t b = 0; b < B; ++b) {
            run += lens[b] > 0 ? lens[b] : 0;
            if (n_chunks + 1 < want && run >= bound) {
                ++n_chunks;
                cb[n_chunks] = b + 1;
                co[n_chunks] = run;
                bound = run + (need - run + 1) / 2;
            }
        }
        ++n_chunks;
        cb[n_chunks] = B;
        co[n_chunks] = need;
    }
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    int rc = host_streams(g);
    if (rc != MOC_OK) return rc;
    rc = ensure((void**)&g->d_stage_seqs, &g->stage_seqs_cap, std::max<size_t>((size_t)need * 4 + 16, 16));
    if (rc != MOC_OK) return rc;
    if (!wide_ids) {
        rc = ensure((void**)&g->d_stage_u16, &g->stage_u16_cap, std::max<size_t>((size_t)need * 2 + 16, 16));
        if (rc != MOC_OK) return rc;
    }
    const size_t bB = (size_t)B, o_peak = 0, o_dur = bB * 8, o_st = 2 * bB * 8, o_lens = align16(o_st + bB * 4),
                 res_bytes = o_st + bB * 4, io_bytes = o_lens + bB * 4;
    rc = ensure((void**)&g->d_stage_io, &g->stage_io_cap, io_bytes);
    if (rc != MOC_OK) return rc;
    if (res_bytes > g->h_stage_cap) {
        if (g->h_stage) MOC_CUDA(cudaFreeHost(g->h_stage));
        g->h_stage = nullptr;
        g->h_stage_cap = 0;
        MOC_CUDA(cudaMallocHost((void**)&g->h_stage, res_bytes * 2));
        g->h_stage_cap = res_bytes * 2;
    }
    int64_t* d_peak = (int64_t*)(g->d_stage_io + o_peak);
    int64_t* d_dur = (int64_t*)(g->d_stage_io + o_dur);
    int32_t* d_st = (int32_t*)(g->d_stage_io + o_st);
    int32_t* d_lens = (int32_t*)(g->d_stage_io + o_lens);
    cudaStream_t cs = g->copy_stream;
    // the copy stream starts once the caller's stream has reached this call
    MOC_CUDA(cudaEventRecord(g->chunk_ev[kHostChunks], st));
    MOC_CUDA(cudaStreamWaitEvent(cs, g->chunk_ev[kHostChunks], 0));
    MOC_CUDA(cudaMemcpyAsync(d_lens, lens, bB * 4, cudaMemcpyHostToDevice, cs));
    int launches = 0;
    for (int k = 0; k < n_chunks; ++k) {
        const int64_t s0 = co[k], cnt = co[k + 1] - co[k];
        if (cnt) {
            if (wide_ids)
                MOC_CUDA(cudaMemcpyAsync(g->d_stage_seqs + s0, (const int32_t*)ids + s0, (size_t)cnt * 4, cudaMemcpyHostToDevice, cs));
            else
                MOC_CUDA(cudaMemcpyAsync(g->d_stage_u16 + s0, (const uint16_t*)ids + s0, (size_t)cnt * 2, cudaMemcpyHostToDevice, cs));
        }
        MOC_CUDA(cudaEventRecord(g->chunk_ev[k], cs));
        MOC_CUDA(cudaStreamWaitEvent(st, g->chunk_ev[k], 0));
        if (cnt && !wide_ids) {
            const int blocks = (int)std::min<int64_t>((cnt / 8 + 255) / 256 + 1, (int64_t)g->sm_count * 8);
            moc::widen_ids_kernel<<<blocks, 256, 0, st>>>(g->d_stage_u16 + s0, g->d_stage_seqs + s0, cnt);
            ++launches;
        }
        const int32_t b0 = cb[k], nb = cb[k + 1] - cb[k];
        if (nb > 0) {
            rc = launch_eval(g, g->d_stage_seqs + s0, d_lens + b0, nb, M, d_peak + b0, d_dur + b0, d_st + b0, st);
            if (rc != MOC_OK) return rc;
        }
    }
    g_launches += launches;      // the evaluation launches were counted as they were enqueued
    MOC_CUDA(cudaMemcpyAsync(g->h_stage, g->d_stage_io, res_bytes, cudaMemcpyDeviceToHost, st));
    MOC_CUDA(cudaStreamSynchronize(st));
    memcpy(out_peak, g->h_stage + o_peak, bB * 8);
    memcpy(out_dur, g->h_stage + o_dur, bB * 8);
    memcpy(out_feasible, g->h_stage + o_st, bB * 4);
    return MOC_OK;
}
}  // namespace

int moc_eval_batch_host(const moc_graph* g, const int32_t* seqs, int64_t n_steps, const int32_t* lens,
                        int32_t B, int64_t M, int64_t* out_peak, int64_t* out_dur,
                        int32_t* out_feasible, void* stream) {
    g_err[0] = 0;
    g_launches = 0;
    if (!g || B < 0 || n_steps < 0) return fail(MOC_ERR_ARG, "moc_eval_batch_host: null handle or negative size");
    if (B == 0) return MOC_OK;
    if (!lens || !out_peak || !out_dur || !out_feasible || (n_steps > 0 && !seqs))
        return fail(MOC_ERR_ARG, "moc_eval_batch_host: null array");
    return eval_host(g, seqs, true, n_steps, lens, B, M, out_peak, out_dur, out_feasible, (cudaStream_t)stream, "moc_eval_batch_host");
}

int moc_eval_batch_host16(const moc_graph* g, const uint16_t* seqs, int64_t n_steps, const int32_t* lens,
                          int32_t B, int64_t M, int64_t* out_peak, int64_t* out_dur,
                          int32_t* out_feasible, void* stream) {
    g_err[0] = 0;
    g_launches = 0;
    if (!g || B < 0 || n_steps < 0) return fail(MOC_ERR_ARG, "moc_eval_batch_host16: null handle or negative size");
    if (g->n > 65535) return fail(MOC_ERR_ARG, "moc_eval_batch_host16: n = %d does not fit 16-bit node ids", g->n);
    if (B == 0) return MOC_OK;
    if (!lens || !out_peak || !out_dur || !out_feasible || (n_steps > 0 && !seqs))
        return fail(MOC_ERR_ARG, "moc_eval_batch_host16: null array");
    return eval_host(g, seqs, false, n_steps, lens, B, M, out_peak, out_dur, out_feasible, (cudaStream_t)stream, "moc_eval_batch_host16");
}

// ---- evaluation without any allocation -----------------------------------------------------------
// Packing offsets for moc_eval_batch_noalloc live in this array of the library's device image.  In
// host code `g_noalloc_offs` is only a stand-in for the symbol, not a device address: the address a
// kernel can use comes from cudaGetSymbolAddress, asked once per device with that device current.
static __device__ __align__(256) long long g_noalloc_offs[MOC_NOALLOC_MAX_B + 1];

namespace {
constexpr int kMaxDevices = 64;
int64_t* g_noalloc_ptr[kMaxDevices] = {};  // device address of g_noalloc_offs, per device ordinal

// Caller has made `device` current.
int noalloc_offsets(int device, int64_t** out) {
    if (device < 0 || device >= kMaxDevices) return fail(MOC_ERR_ARG, "device ordinal %d not supported", device);
    int64_t* ptr = __atomic_load_n(&g_noalloc_ptr[device], __ATOMIC_ACQUIRE);
    if (!ptr) {
        cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_offs);
        if (e != cudaSuccess || !ptr)
            return fail(MOC_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
        __atomic_store_n(&g_noalloc_ptr[device], ptr, __ATOMIC_RELEASE);
    }
    *out = ptr;
    return MOC_OK;
}
}  // namespace

int moc_eval_batch_noalloc(const moc_graph* g, const int32_t* seqs, const int32_t* lens, int32_t B,
                           int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible,
                           void* stream) {
    g_err[0] = 0;
    g_launches = 0;
    if (!g || B < 0) return fail(MOC_ERR_ARG, "moc_eval_batch_noalloc: null handle or B < 0");
    if (B == 0) return MOC_OK;
    if (B > MOC_NOALLOC_MAX_B)
        return fail(MOC_ERR_ARG, "moc_eval_batch_noalloc: B = %d exceeds the fixed scratch of %d sequences; "
                    "split the batch or use moc_eval_batch", B, MOC_NOALLOC_MAX_B);
    if (!seqs || !lens || !out_peak || !out_dur || !out_feasible)
        return fail(MOC_ERR_ARG, "moc_eval_batch_noalloc: null array");
    if (reinterpret_cast<uintptr_t>(seqs) & 3) return fail(MOC_ERR_ARG, "moc_eval_batch_noalloc: seqs not 4-byte aligned");
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    int64_t* offs = nullptr;
    int rc = noalloc_offsets(g->device, &offs);
    if (rc != MOC_OK) return rc;
    if (!g->plan_eval.valid) {
        rc = make_plan(g, false, &g->plan_eval);  // attribute and occupancy queries only
        if (rc != MOC_OK) return rc;
    }
    const Plan& pl = g->plan_eval;
    if (pl.global_state)
        return fail(MOC_ERR_ARG, "moc_eval_batch_noalloc: this graph needs a global workspace "
                    "(per-sequence state exceeds shared memory); use moc_eval_batch");
    // the offsets kernel rewrites offs[0..B] before the evaluation kernel reads them
    return enqueue_eval(g, pl, offs, true, seqs, lens, B, M, out_peak, out_dur, out_feasible, (cudaStream_t)stream);
}

int moc_mem_profile(const moc_graph* g, const int32_t* seq, int32_t len, int64_t* out_profile,
                    int32_t* out_free, int32_t* out_status, void* stream) {
    g_err[0] = 0;
    g_launches = 0;
    if (!g || len < 0 || !out_status || (len > 0 && (!seq || !out_profile)))
        return fail(MOC_ERR_ARG, "moc_mem_profile: null pointer or len < 0");
    if (reinterpret_cast<uintptr_t>(seq) & 3) return fail(MOC_ERR_ARG, "moc_mem_profile: seq not 4-byte aligned");
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (!g->plan_profile.valid) {
        int rc = make_plan(g, true, &g->plan_profile);
        if (rc != MOC_OK) return rc;
    }
    const Plan& pl = g->plan_profile;
    if (pl.global_state) {
        int rc = ensure((void**)&g->d_state, &g->state_cap, (size_t)pl.group_bytes);
        if (rc != MOC_OK) return rc;
    }
    moc::EvalParams p = base_params(g, pl);
    p.seqs = seq;
    p.single_len = len;
    p.B = 1;
    p.M = INT64_MAX;
    p.out_status = out_status;
    p.out_profile = out_profile;
    p.out_free = out_free;
    p.gstate = g->d_state;
    pl.fn<<<1, pl.block, pl.smem, st>>>(p);
    ++g_launches;
    MOC_CUDA(cudaGetLastError());
    return MOC_OK;
}

}  // extern "C"

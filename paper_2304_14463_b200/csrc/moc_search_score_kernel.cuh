// One generation of the search on the cached evaluation in one kernel (paper: Section 3, the two-phase
// local search; Section 2, Eqs. 1-5 for what a proposal's score is).  A warp owns a chain: it brings the
// chain's cached copy positions, free steps and memory profile into shared memory once, draws the
// chain's E proposals with one lane each, scores them from the staged copy and settles the chain (the
// best proposal replaces the sequence when its key is not larger; the chain is then listed for the
// rebuild of its cache entry).  Same draws, same scores and same choice as the three kernels
// search_draw_kernel, edit_eval_kernel and search_pick_kernel, which remain the general path.
//
// Work split inside the warp.  Everything that is scalar per proposal runs with a lane per proposal:
// the draw, the copy-count test, the precedence test on the edges of the edited node, and the list of
// range corrections to the parent's profile (one entry per retention interval that changes: at most
// 4 for the edited node and 2 for each of its predecessors).  The one part that is long, the maximum
// of the corrected profile over the recomputed window, runs with the whole warp on one proposal at a
// time: the corrections go into a difference array, each lane takes a run of consecutive window steps,
// and a warp scan carries the running correction from run to run.
// Only proposals that passed both tests (about a fifth of random ones) reach that part.
//
// The correction lists of the lanes share `list_cap` entries of shared memory.  When the admissible
// proposals of a pass need more, they are handled in several rounds, lowest lanes first; the host
// only selects this kernel when one proposal's worst case (4 + 2 * largest in-degree) fits.
#pragma once
#include "moc_edit_kernels.cuh"
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

// Bytes of the block's copy of the graph: successor and predecessor offsets (n + 1 words each), output sizes
// (n MemT), successor and predecessor lists (16 bits per entry).
__host__ __device__ inline size_t score_graph_bytes(int32_t n, int64_t n_edges, size_t mem_sz, uint32_t* pred_b, uint32_t* m_b,
                                                    uint32_t* succ_b, uint32_t* predl_b) {
    size_t o = ((size_t)(n + 1) * 4 + 15) & ~size_t(15);
    *pred_b = (uint32_t)o;
    o += ((size_t)(n + 1) * 4 + 15) & ~size_t(15);
    *m_b = (uint32_t)o;
    o += ((size_t)n * mem_sz + 15) & ~size_t(15);
    *succ_b = (uint32_t)o;
    o += ((size_t)n_edges * 2 + 15) & ~size_t(15);
    *predl_b = (uint32_t)o;
    o += ((size_t)n_edges * 2 + 15) & ~size_t(15);
    return o;
}

// 16 bytes from global to shared memory without a register in between (completed by cp.async.wait_all).
__device__ __forceinline__ void score_copy16(void* dst_shared, const void* src_global) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_shared)), "l"(src_global) : "memory");
}

__device__ __forceinline__ int32_t score_warp_max(int32_t v) { return __reduce_max_sync(0xFFFFFFFFu, v); }
__device__ __forceinline__ int64_t score_warp_max(int64_t v) { return edit_warp_max(v); }

// kGraphOnChip: the block keeps the graph's lists and output sizes in shared memory (every lane walks them
// at its own node, and what the warps' arrays leave of the L1 is too small to hold them).
template <typename MemT, bool kGraphOnChip>
__global__ void __launch_bounds__(kScoreThreads, 1) search_score_kernel(const ScoreParams p) {
    extern __shared__ __align__(16) char smem[];
    const EditCacheDev& c = p.c;
    const SearchParams& s = p.s;
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const uint32_t* s_succ_start = reinterpret_cast<const uint32_t*>(smem);
    const uint32_t* s_pred_start = reinterpret_cast<const uint32_t*>(smem + p.gs_pred_b);
    const MemT* s_m = reinterpret_cast<const MemT*>(smem + p.gs_m_b);
    const uint16_t* s_succ = reinterpret_cast<const uint16_t*>(smem + p.gs_succ_b);
    const uint16_t* s_pred = reinterpret_cast<const uint16_t*>(smem + p.gs_predl_b);
    if (kGraphOnChip) {
        const int32_t E = __ldg(&c.succ_start[c.n]);
        for (int32_t i = threadIdx.x; i <= c.n; i += blockDim.x) {
            const_cast<uint32_t*>(s_succ_start)[i] = (uint32_t)__ldg(&c.succ_start[i]);
            const_cast<uint32_t*>(s_pred_start)[i] = (uint32_t)__ldg(&c.pred_start[i]);
            if (i < c.n) const_cast<MemT*>(s_m)[i] = (MemT)__ldg(&c.m[i]);
        }
        for (int32_t i = threadIdx.x; i < E; i += blockDim.x) {
            const_cast<uint16_t*>(s_succ)[i] = (uint16_t)__ldg(&c.succ[i]);
            const_cast<uint16_t*>(s_pred)[i] = (uint16_t)__ldg(&c.pred[i]);
        }
        __syncthreads();
    }
    auto g_succ_start = [&](int32_t v) -> int32_t { return kGraphOnChip ? (int32_t)s_succ_start[v] : __ldg(&c.succ_start[v]); };
    auto g_pred_start = [&](int32_t v) -> int32_t { return kGraphOnChip ? (int32_t)s_pred_start[v] : __ldg(&c.pred_start[v]); };
    auto g_succ = [&](int32_t k) -> int32_t { return kGraphOnChip ? (int32_t)s_succ[k] : __ldg(&c.succ[k]); };
    auto g_pred = [&](int32_t k) -> int32_t { return kGraphOnChip ? (int32_t)s_pred[k] : __ldg(&c.pred[k]); };
    auto g_m = [&](int32_t v) -> MemT { return kGraphOnChip ? s_m[v] : (MemT)__ldg(&c.m[v]); };
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
            int64_t out_pk = -1, out_du = -1;
            int32_t out_st = -2;
            bool go = live && qq < T;
            if (go && pst < 0) { out_st = kStatusParentInvalid; go = false; }
            // ---- per proposal: the edit in parent and child steps
            const int32_t x = go ? (int32_t)row[qq] : 0;
            const int32_t qd = o >= 1 ? qq : kEditNone, ji = o != 1 ? jj : kEditNone;
            const int32_t Tc = T + (o == 0 ? 1 : 0) - (o == 1 ? 1 : 0);
            auto map = [&](int32_t st) -> int32_t { const int32_t s1 = st - (st > qd ? 1 : 0); return s1 + (s1 >= ji ? 1 : 0); };
            auto inv = [&](int32_t t) -> int32_t { const int32_t t1 = t - (t > ji ? 1 : 0); return t1 + (t1 >= qd ? 1 : 0); };
            const uint32_t wx = occ[x];
            const int32_t xa = (int32_t)min(wx & 0xFFFFu, wx >> 16) - 1, xb = (int32_t)max(wx & 0xFFFFu, wx >> 16) - 1;
            const int32_t cnt = xa == xb ? 1 : 2, cnt2 = cnt - (o >= 1 ? 1 : 0) + (o != 1 ? 1 : 0);
            // Child copies of x, ascending: c0, c1 (c1 = none when one copy).  Beside each copy two thresholds in
            // 1-based parent steps, for copies r of OTHER nodes (none of them is deleted or inserted, and the
            // map from parent to child steps keeps their order): r lies behind the copy iff r > ta, in front of
            // it iff r < tb.  A surviving copy at parent step s has ta = tb = s + 1; the inserted copy has
            // ta = thr, tb = thr + 1 with thr = j + [j >= q] (parent steps below thr end up in front of it).
            int32_t c0 = kEditNone, c1 = kEditNone, ta0 = 0, tb0 = 0, ta1 = 0, tb1 = 0;
            {
                auto push = [&](int32_t cs, int32_t ta, int32_t tb) {
                    if (c0 == kEditNone) { c0 = cs; ta0 = ta; tb0 = tb; }
                    else if (cs < c0) { c1 = c0; ta1 = ta0; tb1 = tb0; c0 = cs; ta0 = ta; tb0 = tb; }
                    else { c1 = cs; ta1 = ta; tb1 = tb; }
                };
                if (xa != qd) push(map(xa), xa + 1, xa + 1);
                if (cnt == 2 && xb != qd) push(map(xb), xb + 1, xb + 1);
                if (ji != kEditNone) { const int32_t thr = ji + (ji >= qd ? 1 : 0); push(ji, thr, thr + 1); }
            }
            int32_t ps0 = 0, ps1 = 0, ss0 = 0, ss1 = 0;
            bool adm = false;
            if (go) {
                const bool x_two_ok = c.C >= 2 && (c.cap == nullptr || __ldg(&c.cap[x]) >= 2);
                if (cnt2 >= 1 && cnt2 <= 2 && (cnt2 == 1 || x_two_ok)) {
                    out_du = pdur + __ldg(&c.w[x]) * (cnt2 - cnt);
                    ps0 = g_pred_start(x); ps1 = g_pred_start(x + 1);
                    ss0 = g_succ_start(x); ss1 = g_succ_start(x + 1);
                    // ---- precedence (Eq. 5) can only break on edges that touch x: no first copy of a
                    // predecessor behind the first copy of x, no first copy of a successor in front of it
                    bool viol = false;
#pragma unroll 1
                    for (int32_t k = ps0; k < ps1; ++k) {
                        const uint32_t wv = occ[g_pred(k)];
                        viol |= (int32_t)min(wv & 0xFFFFu, wv >> 16) > ta0;
                    }
#pragma unroll 1
                    for (int32_t k = ss0; k < ss1; ++k) {
                        const uint32_t wv = occ[g_succ(k)];
                        viol |= (int32_t)min(wv & 0xFFFFu, wv >> 16) < tb0;
                    }
                    if (viol) out_st = -1;
                    else adm = true;
                }
            }
            // ---- admissible proposals: range corrections with a lane each, window maximum with the warp
            const int32_t need = 4 + 2 * (ps1 - ps0);
            uint32_t pending = __ballot_sync(kFull, adm);
            while (pending) {
                const bool wait = (pending >> lane & 1u) != 0;
                const int32_t nd = wait ? need : 0;
                const int32_t incl = edit_warp_incl_sum(nd, lane);
                const bool act = wait && incl <= p.list_cap;
                const uint32_t act_mask = __ballot_sync(kFull, act);
                if (act_mask == 0) break;                   // cannot happen: one proposal's worst case fits
                const int32_t lbase = incl - nd;
                int32_t lcnt = 0, lo_w = kEditNone, hi_w = -1;
                MemT cross = 0, edge = 0;
                if (act) {
                    const bool x_sink = ss0 == ss1;
                    auto emit = [&](int32_t l, int32_t h, MemT val) {       // += val on child steps l..h
                        if (l > h) return;
                        rl[lbase + lcnt] = (uint32_t)l | (uint32_t)(h + 1) << 16;
                        rv[lbase + lcnt] = val;
                        ++lcnt;
                        lo_w = min(lo_w, l);
                        hi_w = max(hi_w, h);
                    };
                    // old copy run at parent step ps and freed at pf, in child steps
                    auto old_range = [&](int32_t ps, int32_t pf, bool to_end, int32_t& l, int32_t& h) {
                        l = ps == qd ? (pf > qd ? map(qd + 1) : kEditNone) : map(ps);
                        h = pf == qd ? (pf > ps ? map(pf - 1) : -1) : map(pf);
                        if (to_end && ps != qd) h = Tc - 1;
                    };
                    // Latest consumer copy of a node y, per copy of y: over the words r of y's successors, in 1-based
                    // parent steps and two 16-bit halves at a time.  mx = max r gives the free step of the last
                    // copy; G = max((r - tb) mod 2^16), seeded with (ta - tb) mod 2^16, gives the latest r with
                    // ta < r < tb as tb + G (ta itself when there is none): the free step of the first of two copies.
                    auto scan_succ = [&](int32_t s0, int32_t s1, int32_t ta, int32_t tb, uint32_t& mx, uint32_t& R) {
                        const uint32_t ntb = (uint32_t)(-tb) & 0xFFFFu, nbb = ntb | ntb << 16;
                        const uint32_t seed = (uint32_t)(ta - tb) & 0xFFFFu;
                        uint32_t G = seed | seed << 16, m2 = 0;
#pragma unroll 1
                        for (int32_t z = s0; z < s1; ++z) {
                            const int32_t v = g_succ(z);
                            const uint32_t wv = v == x ? 0u : occ[v];          // the copies of x are added in child steps
                            G = __viaddmax_u16x2(wv, nbb, G);
                            m2 = max_u16x2(m2, wv);
                        }
                        mx = max(m2 & 0xFFFFu, m2 >> 16);
                        R = ((uint32_t)tb + max(G & 0xFFFFu, G >> 16)) & 0xFFFFu;
                    };
                    {   // ---- x itself: its child copies against the copies of its successors
                        const MemT mxv = g_m(x);
                        const int32_t n0 = c0, n1 = c1 == kEditNone ? c0 : c1;
                        const bool two = c1 != kEditNone;
                        uint32_t mx, R;
                        scan_succ(ss0, ss1, ta0, two ? tb1 : tb0, mx, R);
                        int32_t f1 = x_sink ? Tc - 1 : max(n1, map((int32_t)mx - 1));
                        int32_t f0 = f1;
                        if (two) f0 = (int32_t)R == (ta0 & 0xFFFF) ? n0 : map((int32_t)R - 1);
                        int32_t l, h;
                        old_range(xa, (int32_t)fre[xa], x_sink && cnt == 1, l, h);
                        emit(l, h, (MemT)(-mxv));
                        if (cnt == 2) {
                            old_range(xb, (int32_t)fre[xb], x_sink, l, h);
                            emit(l, h, (MemT)(-mxv));
                        }
                        emit(n0, f0, mxv);
                        if (two) emit(n1, f1, mxv);
                    }
#pragma unroll 1
                    for (int32_t k = ps0; k < ps1; ++k) {                   // ---- the predecessors of x
                        const int32_t y = g_pred(k);
                        const MemT my = g_m(y);
                        const uint32_t wy = occ[y];
                        const int32_t ya1 = (int32_t)min(wy & 0xFFFFu, wy >> 16), yb1 = (int32_t)max(wy & 0xFFFFu, wy >> 16);
                        const int32_t ya = ya1 - 1, yb = yb1 - 1;
                        const bool two = ya != yb;
                        const int32_t n0 = map(ya), n1 = map(yb);
                        uint32_t mx, R;
                        scan_succ(g_succ_start(y), g_succ_start(y + 1), ya1, yb1, mx, R);
                        int32_t f1 = map(max((int32_t)mx, yb1) - 1);          // consumers other than x, in parent order
                        int32_t f0 = map((int32_t)R - 1);                     // R = ya1 when none lies between the copies
                        f1 = max(f1, c1 == kEditNone ? c0 : c1);              // x consumes y
                        if (c0 > n0 && c0 < n1) f0 = max(f0, c0);
                        if (c1 != kEditNone && c1 > n0 && c1 < n1) f0 = max(f0, c1);
                        if (!two) f0 = f1;
                        int32_t l, h;
                        old_range(ya, (int32_t)fre[ya], false, l, h);
                        if (h != f0) emit(min(h, f0) + 1, max(h, f0), f0 > h ? my : (MemT)(-my));
                        if (two) {
                            old_range(yb, (int32_t)fre[yb], false, l, h);
                            if (h != f1) emit(min(h, f1) + 1, max(h, f1), f1 > h ? my : (MemT)(-my));
                        }
                    }
                    if (qd != kEditNone) {
                        // the parent's prefix / suffix maxima must not reach across the deleted step
                        const int32_t cl = qd > 0 ? map(qd - 1) : -1, cr = qd < T - 1 ? map(qd + 1) : Tc;
                        lo_w = min(lo_w, cl + 1);
                        hi_w = max(hi_w, cr - 1);
                    }
                    // usage carried across the inserted step
                    if (ji != kEditNone) {
                        if (ji + 1 < Tc) {
                            const int32_t tr = inv(ji + 1), tl = ji >= 1 ? inv(ji - 1) : -1;
                            cross = prof[tr] - g_m((int32_t)row[tr]);
                            if (qd != kEditNone && qd > tl && qd < tr && (int32_t)fre[qd] >= tr) cross -= g_m(x);
                        } else {
                            cross = (MemT)c.sink_m;
                            if (x_sink && qd == xb) cross -= g_m(x);
                        }
                    }
                    // the parent's maxima outside the window
                    if (lo_w > 0) edge = g_pm[inv(lo_w - 1)];
                    if (hi_w < Tc - 1) { const MemT v = g_sm[inv(hi_w + 1)]; edge = v > edge ? v : edge; }
                }
                __syncwarp();
                MemT best = edge;
                for (uint32_t mk = act_mask; mk; mk &= mk - 1) {
                    const int sl = __ffs(mk) - 1;
                    const int32_t lo = __shfl_sync(kFull, lo_w, sl), hi = __shfl_sync(kFull, hi_w, sl);
                    const int32_t ji_s = __shfl_sync(kFull, ji, sl), qd_s = __shfl_sync(kFull, qd, sl);
                    const int32_t lb = __shfl_sync(kFull, lbase, sl), lc = __shfl_sync(kFull, lcnt, sl);
                    const MemT cr_s = __shfl_sync(kFull, cross, sl);
                    // corrections as a difference array over the child steps (zero outside this block of code)
                    for (int32_t k = lane; k < lc; k += 32) {
                        const uint32_t lh = rl[lb + k];
                        const MemT v = rv[lb + k];
                        edit_add(&diff[lh & 0xFFFFu], v);
                        edit_add(&diff[lh >> 16], (MemT)(-v));
                    }
                    __syncwarp();
                    // lane owns a run of consecutive window steps (odd length: the runs start in different banks)
                    const int32_t L = hi - lo + 1;
                    const int32_t per = ((L + 31) / 32) | 1;
                    const int32_t t0 = lo + min(L, lane * per), t1 = lo + min(L, (lane + 1) * per);
                    // one pass: running correction and usage relative to the start of the run, then the carry
                    // from the runs in front (max over the run of carry + x = carry + max x)
                    MemT run = 0, top = sizeof(MemT) == 8 ? (MemT)INT64_MIN : (MemT)INT32_MIN;
                    const bool any = t0 < t1;
                    for (int32_t t = t0; t < t1; ++t) {
                        run += diff[t];
                        diff[t] = 0;
                        const int32_t tt = t - (t > ji_s ? 1 : 0);
                        const MemT u = run + (t == ji_s ? cr_s : prof[tt + (tt >= qd_s ? 1 : 0)]);
                        top = u > top ? u : top;
                    }
                    const MemT carry = edit_warp_incl_sum(run, lane) - run;
                    top = any ? top + carry : (MemT)0;          // usage is never negative: 0 is neutral
                    if (lane == 0) diff[hi + 1] = 0;
                    top = score_warp_max(top);
                    if (lane == sl) best = top > best ? top : best;
                    __syncwarp();
                }
                if (act) {
                    out_pk = (int64_t)best;
                    out_st = out_pk <= s.M ? 1 : 0;
                }
                pending &= ~act_mask;
                __syncwarp();
            }
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

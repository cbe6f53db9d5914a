// Scoring of up to 32 single edits of evaluated sequences, a lane each, by the lanes of one warp (Section 2,
// Eqs. 2-5: an edit of a copy of node x changes only the retention intervals of x and of its predecessors).
// Shared by the warp-per-chain kernel of the search (all 32 edits belong to one parent, staged in shared
// memory) and by the general edit kernel (every lane has its own parent in global memory).
//
// Work split inside the warp.  Everything that is scalar per edit runs with a lane per edit: the copy-count
// test, the precedence test on the edges of the edited node, and the list of range corrections to the
// parent's profile (one entry per retention interval that changes: at most 4 for the edited node and 2 for
// each of its predecessors).  Copies of other nodes keep their order under the edit, so these node passes run
// in parent steps with two packed 16-bit reductions per successor word, and only results are mapped to child
// steps.  The one part that is long, the maximum of the corrected profile over the recomputed window, runs
// with the whole warp on one edit at a time: the corrections go into a difference array, each lane takes a
// run of consecutive window steps, and a warp scan carries the running correction from run to run.
//
// The correction lists of the lanes share `list_cap` entries of shared memory.  When the admissible edits of
// a call need more, they are handled in several rounds, lowest lanes first; the host only selects kernels
// built on this when one edit's worst case (4 + 2 * largest in-degree) fits.
//
// Parent (per lane): occ(v) the node's copy-position word, fre(s), row(s), prof(s), pm(s), sm(s) of the
// lane's parent, and prof_view(l), a callable that reads the usage array of lane l's parent.
// Graph: succ_start(v), pred_start(v), succ(k), pred(k), m(v).
#pragma once
#include "moc_edit_kernels.cuh"

namespace moc {

__device__ __forceinline__ int32_t score_warp_max(int32_t v) { return __reduce_max_sync(0xFFFFFFFFu, v); }
__device__ __forceinline__ int64_t score_warp_max(int64_t v) { return edit_warp_max(v); }

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

// The graph for edit_pass: the block's copy in shared memory (kChip) or the handle's arrays.
template <typename MemT, bool kChip>
struct ScoreGraph {
    const uint32_t* s_succ_start;
    const uint32_t* s_pred_start;
    const MemT* s_m;
    const uint16_t* s_succ;
    const uint16_t* s_pred;
    const EditCacheDev* c;
    __device__ __forceinline__ int32_t succ_start(int32_t v) const { return kChip ? (int32_t)s_succ_start[v] : __ldg(&c->succ_start[v]); }
    __device__ __forceinline__ int32_t pred_start(int32_t v) const { return kChip ? (int32_t)s_pred_start[v] : __ldg(&c->pred_start[v]); }
    __device__ __forceinline__ int32_t succ(int32_t k) const { return kChip ? (int32_t)s_succ[k] : __ldg(&c->succ[k]); }
    __device__ __forceinline__ int32_t pred(int32_t k) const { return kChip ? (int32_t)s_pred[k] : __ldg(&c->pred[k]); }
    __device__ __forceinline__ MemT m(int32_t v) const { return kChip ? s_m[v] : (MemT)__ldg(&c->m[v]); }
};

// Fills the block's copy of the graph (all threads of the block; ends with a barrier).
template <typename MemT>
__device__ __forceinline__ void score_stage_graph(const EditCacheDev& c, char* smem, uint32_t pred_b, uint32_t m_b, uint32_t succ_b,
                                                  uint32_t predl_b) {
    uint32_t* ss = reinterpret_cast<uint32_t*>(smem);
    uint32_t* ps = reinterpret_cast<uint32_t*>(smem + pred_b);
    MemT* sm = reinterpret_cast<MemT*>(smem + m_b);
    uint16_t* sl = reinterpret_cast<uint16_t*>(smem + succ_b);
    uint16_t* pl = reinterpret_cast<uint16_t*>(smem + predl_b);
    const int32_t E = __ldg(&c.succ_start[c.n]);
    for (int32_t i = threadIdx.x; i <= c.n; i += blockDim.x) {
        ss[i] = (uint32_t)__ldg(&c.succ_start[i]);
        ps[i] = (uint32_t)__ldg(&c.pred_start[i]);
        if (i < c.n) sm[i] = (MemT)__ldg(&c.m[i]);
    }
    for (int32_t i = threadIdx.x; i < E; i += blockDim.x) {
        sl[i] = (uint16_t)__ldg(&c.succ[i]);
        pl[i] = (uint16_t)__ldg(&c.pred[i]);
    }
    __syncthreads();
}

// live: the lane holds an edit record whose fields are in range; pst, T, pdur: status, length and duration of its
// parent; o, qq, jj: kind (0 insert, 1 delete, 2 move), step of the parent, insertion index.  rl, rv (list_cap
// entries each) and diff (row stride + 4 entries, all zero on entry and on return) are the warp's scratch in
// shared memory.  Results: peak, duration, status (-3 parent invalid, -2 malformed, -1 precedence, 0 / 1 against
// M) and the number of child steps whose usage was recomputed.  Every lane of the warp must call.
template <typename MemT, typename Parent, typename Graph>
__device__ __forceinline__ void edit_pass(const Parent& P, const Graph& Gr, const EditCacheDev& c, int64_t M, int lane,
                                          bool live, int32_t pst, int32_t T, int64_t pdur, int32_t o, int32_t qq, int32_t jj,
                                          uint32_t* rl, MemT* rv, MemT* diff, int32_t list_cap, int64_t& out_pk,
                                          int64_t& out_du, int32_t& out_st, int32_t& out_win) {
    out_pk = -1;
    out_du = -1;
    out_st = -2;
    out_win = 0;
    constexpr uint32_t kFull = 0xFFFFFFFFu;
    bool go = live && qq < T;
    if (go && pst < 0) { out_st = kStatusParentInvalid; go = false; }
    // ---- per proposal: the edit in parent and child steps
    const int32_t x = go ? P.row(qq) : 0;
    const int32_t qd = o >= 1 ? qq : kEditNone, ji = o != 1 ? jj : kEditNone;
    const int32_t Tc = T + (o == 0 ? 1 : 0) - (o == 1 ? 1 : 0);
    auto map = [&](int32_t st) -> int32_t { const int32_t s1 = st - (st > qd ? 1 : 0); return s1 + (s1 >= ji ? 1 : 0); };
    auto inv = [&](int32_t t) -> int32_t { const int32_t t1 = t - (t > ji ? 1 : 0); return t1 + (t1 >= qd ? 1 : 0); };
    const uint32_t wx = P.occ(x);
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
            ps0 = Gr.pred_start(x); ps1 = Gr.pred_start(x + 1);
            ss0 = Gr.succ_start(x); ss1 = Gr.succ_start(x + 1);
            // ---- precedence (Eq. 5) can only break on edges that touch x: no first copy of a
            // predecessor behind the first copy of x, no first copy of a successor in front of it
            bool viol = false;
#pragma unroll 1
            for (int32_t k = ps0; k < ps1; ++k) {
                const uint32_t wv = P.occ(Gr.pred(k));
                viol |= (int32_t)min(wv & 0xFFFFu, wv >> 16) > ta0;
            }
#pragma unroll 1
            for (int32_t k = ss0; k < ss1; ++k) {
                const uint32_t wv = P.occ(Gr.succ(k));
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
        const bool act = wait && incl <= list_cap;
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
                    const int32_t v = Gr.succ(z);
                    const uint32_t wv = v == x ? 0u : P.occ(v);          // the copies of x are added in child steps
                    G = __viaddmax_u16x2(wv, nbb, G);
                    m2 = max_u16x2(m2, wv);
                }
                mx = max(m2 & 0xFFFFu, m2 >> 16);
                R = ((uint32_t)tb + max(G & 0xFFFFu, G >> 16)) & 0xFFFFu;
            };
            {   // ---- x itself: its child copies against the copies of its successors
                const MemT mxv = Gr.m(x);
                const int32_t n0 = c0, n1 = c1 == kEditNone ? c0 : c1;
                const bool two = c1 != kEditNone;
                uint32_t mx, R;
                scan_succ(ss0, ss1, ta0, two ? tb1 : tb0, mx, R);
                int32_t f1 = x_sink ? Tc - 1 : max(n1, map((int32_t)mx - 1));
                int32_t f0 = f1;
                if (two) f0 = (int32_t)R == (ta0 & 0xFFFF) ? n0 : map((int32_t)R - 1);
                int32_t l, h;
                old_range(xa, P.fre(xa), x_sink && cnt == 1, l, h);
                emit(l, h, (MemT)(-mxv));
                if (cnt == 2) {
                    old_range(xb, P.fre(xb), x_sink, l, h);
                    emit(l, h, (MemT)(-mxv));
                }
                emit(n0, f0, mxv);
                if (two) emit(n1, f1, mxv);
            }
#pragma unroll 1
            for (int32_t k = ps0; k < ps1; ++k) {                   // ---- the predecessors of x
                const int32_t y = Gr.pred(k);
                const MemT my = Gr.m(y);
                const uint32_t wy = P.occ(y);
                const int32_t ya1 = (int32_t)min(wy & 0xFFFFu, wy >> 16), yb1 = (int32_t)max(wy & 0xFFFFu, wy >> 16);
                const int32_t ya = ya1 - 1, yb = yb1 - 1;
                const bool two = ya != yb;
                const int32_t n0 = map(ya), n1 = map(yb);
                uint32_t mx, R;
                scan_succ(Gr.succ_start(y), Gr.succ_start(y + 1), ya1, yb1, mx, R);
                int32_t f1 = map(max((int32_t)mx, yb1) - 1);          // consumers other than x, in parent order
                int32_t f0 = map((int32_t)R - 1);                     // R = ya1 when none lies between the copies
                f1 = max(f1, c1 == kEditNone ? c0 : c1);              // x consumes y
                if (c0 > n0 && c0 < n1) f0 = max(f0, c0);
                if (c1 != kEditNone && c1 > n0 && c1 < n1) f0 = max(f0, c1);
                if (!two) f0 = f1;
                int32_t l, h;
                old_range(ya, P.fre(ya), false, l, h);
                if (h != f0) emit(min(h, f0) + 1, max(h, f0), f0 > h ? my : (MemT)(-my));
                if (two) {
                    old_range(yb, P.fre(yb), false, l, h);
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
                    cross = P.prof(tr) - Gr.m(P.row(tr));
                    if (qd != kEditNone && qd > tl && qd < tr && P.fre(qd) >= tr) cross -= Gr.m(x);
                } else {
                    cross = (MemT)c.sink_m;
                    if (x_sink && qd == xb) cross -= Gr.m(x);
                }
            }
            // the parent's maxima outside the window
            if (lo_w > 0) edge = P.pm(inv(lo_w - 1));
            if (hi_w < Tc - 1) { const MemT v = P.sm(inv(hi_w + 1)); edge = v > edge ? v : edge; }
        }
        __syncwarp();
        MemT best = edge;
        for (uint32_t mk = act_mask; mk; mk &= mk - 1) {
            const int sl = __ffs(mk) - 1;
            const int32_t lo = __shfl_sync(kFull, lo_w, sl), hi = __shfl_sync(kFull, hi_w, sl);
            const int32_t ji_s = __shfl_sync(kFull, ji, sl), qd_s = __shfl_sync(kFull, qd, sl);
            const int32_t lb = __shfl_sync(kFull, lbase, sl), lc = __shfl_sync(kFull, lcnt, sl);
            const MemT cr_s = __shfl_sync(kFull, cross, sl);
            const auto view = P.prof_view(sl);
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
                const MemT u = run + (t == ji_s ? cr_s : view(tt + (tt >= qd_s ? 1 : 0)));
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
            out_win = max(hi_w - lo_w + 1, 0);
            out_pk = (int64_t)best;
            out_st = out_pk <= M ? 1 : 0;
        }
        pending &= ~act_mask;
        __syncwarp();
    }
}

}  // namespace moc

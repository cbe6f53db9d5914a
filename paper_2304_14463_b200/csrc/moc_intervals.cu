// Host side of moc_check_intervals (declared in include/moc.h): argument checks and the launch.
#include <algorithm>

#include "moc_host.cuh"
#include "moc_interval_kernels.cuh"

using namespace moc_host;

extern "C" int moc_check_intervals(const moc_graph* g, const int32_t* s, const int32_t* e, const int32_t* a,
                                   int32_t B, int64_t D, const int32_t* topo_index, int64_t M, int64_t* out_peak,
                                   int64_t* out_dur, int32_t* out_mask, int32_t* out_seqs, int32_t* out_lens,
                                   void* stream) {
    clear_error();
    launch_counter() = 0;
    if (!g || B < 0) return fail(MOC_ERR_ARG, "moc_check_intervals: null handle or B < 0");
    if (B == 0) return MOC_OK;
    if (!s || !e || !a || !out_peak || !out_dur || !out_mask)
        return fail(MOC_ERR_ARG, "moc_check_intervals: null array");
    if (D < 1 || D > ((int64_t)1 << 30)) return fail(MOC_ERR_ARG, "moc_check_intervals: D outside [1, 2^30]");
    if (g->C > moc::kIvMaxC) return fail(MOC_ERR_ARG, "moc_check_intervals: C > %d", moc::kIvMaxC);
    const int64_t n = g->n, K = n * g->C;
    if (topo_index && D != n * (n + 1) / 2)
        return fail(MOC_ERR_ARG, "moc_check_intervals: the staged model needs D = n(n+1)/2 = %lld", (long long)(n * (n + 1) / 2));
    DeviceGuard dg(g->device);
    if (!dg.ok) return fail(MOC_ERR_CUDA, "cannot select device %d", g->device);
    moc::IntervalParams p{};
    p.n = g->n;
    p.C = g->C;
    p.succ_start = g->d_succ_start;
    p.succ = g->d_succ;
    p.w = g->d_w;
    p.m = g->d_m64;
    p.s = s;
    p.e = e;
    p.a = a;
    p.B = B;
    p.D = (int32_t)D;
    p.topo_index = topo_index;
    p.M = M;
    p.out_peak = out_peak;
    p.out_dur = out_dur;
    p.out_mask = out_mask;
    p.out_seqs = out_seqs;
    p.out_lens = out_lens;
    p.words = (uint32_t)((D + 32) / 32);
    const bool plain = topo_index == nullptr;
    const bool wide = g->sum_m > (int64_t)INT32_MAX / g->C;     // C * sum(m) bounds every partial usage sum
    const size_t cap = g->smem_optin > 2048 ? g->smem_optin - 2048 : 0;
    const size_t base_b = moc::interval_clear_bytes(p.words, K, plain, wide ? 8 : 4), stage_b = moc::interval_stage_bytes(K, D < 65536 ? 2 : 4);
    if (base_b > cap || K > (int64_t)INT32_MAX / 2)
        return fail(MOC_ERR_ARG, "moc_check_intervals: domain of %lld events with %lld intervals needs %zu bytes of "
                    "shared memory per solution, the device offers %zu", (long long)D, (long long)K, base_b, cap);
    // keep the solution on chip after the first pass while at least eight solutions per SM still fit
    p.byte_marks = plain && 2 * (((size_t)D + 1 + 15) & ~size_t(15)) <= ((((size_t)K + 2) * (wide ? 8 : 4) + 15) & ~size_t(15)) ? 1 : 0;
    const bool stage = (base_b + stage_b) * 8 <= cap;
    const size_t warp_b = base_b + (stage ? stage_b : 0);
    p.warp_bytes = (uint32_t)warp_b;
    // warps per block: the count that puts most warps on an SM (each block loses 1 KB to the system)
    int wpb = 1, best = 0;
    for (int k = 1; k <= moc::kIvMaxWarps; ++k) {
        const size_t blk = warp_b * k + 1024;
        const int fit = blk <= cap + 1024 ? (int)((g->smem_optin) / blk) * k : 0;
        if (fit > best) { best = fit; wpb = k; }
    }
    const size_t smem = warp_b * wpb;
    using Fn = void (*)(const moc::IntervalParams);
    const int cp = g->C <= 2 ? 2 : (g->C <= 4 ? 4 : 8);
    const bool narrow = D < 65536;
    Fn table[2][3][2][3] = {
#define MOC_IV_ROW(PL, CPV) {{(Fn)moc::check_intervals_kernel<PL, CPV, int32_t, false, int32_t>, (Fn)moc::check_intervals_kernel<PL, CPV, int32_t, true, int32_t>, \
                             (Fn)moc::check_intervals_kernel<PL, CPV, int32_t, true, uint16_t>},                                                            \
                            {(Fn)moc::check_intervals_kernel<PL, CPV, int64_t, false, int32_t>, (Fn)moc::check_intervals_kernel<PL, CPV, int64_t, true, int32_t>, \
                             (Fn)moc::check_intervals_kernel<PL, CPV, int64_t, true, uint16_t>}}
        {MOC_IV_ROW(false, 2), MOC_IV_ROW(false, 4), MOC_IV_ROW(false, 8)},
        {MOC_IV_ROW(true, 2), MOC_IV_ROW(true, 4), MOC_IV_ROW(true, 8)}
#undef MOC_IV_ROW
    };
    Fn fn = table[plain ? 1 : 0][cp == 2 ? 0 : (cp == 4 ? 1 : 2)][wide ? 1 : 0][stage ? (narrow ? 2 : 1) : 0];
    MOC_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cap));
    int nb = 0;
    MOC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, 32 * wpb, smem));
    if (nb < 1) return fail(MOC_ERR_CUDA, "moc_check_intervals: kernel does not fit on an SM");
    const int grid = (int)std::min<int64_t>((int64_t)g->sm_count * nb, ((int64_t)B + wpb - 1) / wpb);
    fn<<<grid, 32 * wpb, smem, (cudaStream_t)stream>>>(p);
    MOC_CUDA(cudaGetLastError());
    launch_counter() = 1;
    return MOC_OK;
}

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
    p.D = D;
    p.topo_index = topo_index;
    p.M = M;
    p.out_peak = out_peak;
    p.out_dur = out_dur;
    p.out_mask = out_mask;
    p.out_seqs = out_seqs;
    p.out_lens = out_lens;
    p.words = (uint32_t)((D + 32) / 32);
    const size_t smem = moc::interval_smem_bytes(p.words, K, topo_index == nullptr);
    const size_t cap = g->smem_optin > 2048 ? g->smem_optin - 2048 : 0;
    if (smem > cap)
        return fail(MOC_ERR_ARG, "moc_check_intervals: domain of %lld events with %lld intervals needs %zu bytes of "
                    "shared memory per block, the device offers %zu", (long long)D, (long long)K, smem, cap);
    MOC_CUDA(cudaFuncSetAttribute(moc::check_intervals_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cap));
    int nb = 0;
    MOC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, moc::check_intervals_kernel, moc::kIvThreads, smem));
    if (nb < 1) return fail(MOC_ERR_CUDA, "moc_check_intervals: kernel does not fit on an SM");
    const int grid = (int)std::min<int64_t>((int64_t)g->sm_count * nb, B);
    moc::check_intervals_kernel<<<grid, moc::kIvThreads, smem, (cudaStream_t)stream>>>(p);
    MOC_CUDA(cudaGetLastError());
    launch_counter() = 1;
    return MOC_OK;
}

// The cache handle of the incremental evaluation, shared by the translation units that use it.
#pragma once
#include "moc_host.cuh"
#include "moc_edit_kernels.cuh"
#include "moc_edit_lanes_kernel.cuh"

struct moc_cache {
    const moc_graph* g = nullptr;
    int device = 0;
    int32_t max_parents = 0;
    bool wide = false;
    uint64_t graph_generation = 0;   // moc_graph::generation at the last full build
    char* d_block = nullptr;
    int64_t* d_offs = nullptr;     // max_parents + 1
    moc::EditCacheDev c{};
    size_t warp_bytes = 0;
    int wpb = 0, grid_cap = 0;
    // launch of the lane-per-edit kernel, made on the first moc_eval_edits (0: not yet, -1: the graph does not fit it)
    mutable int lanes_state = 0;
    mutable moc::LanesParams lanes{};
    mutable const void* lanes_fn = nullptr;
    mutable size_t lanes_smem = 0;
    mutable int lanes_grid_cap = 0;
};

namespace moc_host {
// Enqueues the full evaluation that fills cache slots from rows seqs + offs[b] of lens[b] steps (all
// DEVICE): slots 0..P-1, or, with `todo`, the slots todo[0 .. *todo_count) (both DEVICE; slot numbers
// below P).  out_* may be null.
int cache_prepare(moc_cache* h, const int32_t* seqs, const int32_t* lens, const int64_t* offs, int32_t P,
                  const int32_t* todo, const int32_t* todo_count, int64_t M, int64_t* out_peak, int64_t* out_dur,
                  int32_t* out_status, cudaStream_t st);
}  // namespace moc_host

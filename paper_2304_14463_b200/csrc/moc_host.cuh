// Host-side types shared by the translation units of libmoc_b200.so: the graph handle, the launch
// plan of the evaluation kernels, error reporting, and the one internal entry that enqueues an
// evaluation with caller-supplied row offsets.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/moc.h"
#include "moc_kernels.cuh"
#include "moc_pair_kernel.cuh"
#include "moc_lane_kernel.cuh"
#include "moc_quad_kernel.cuh"

namespace moc_host {

using KernelFn = void (*)(const moc::EvalParams);
using PairFn = void (*)(const moc::PairParams);
using LaneFn = void (*)(const moc::LaneParams);
using QuadFn = void (*)(const moc::QuadParams);

struct Plan {
    bool valid = false;
    KernelFn fn = nullptr;
    int G = 0, gpc = 0, grid = 0, block = 0, CP = 0;
    size_t smem = 0;
    bool global_state = false, wide = false;
    uint32_t cnt_bytes = 0, occ_bytes = 0, delta_bytes = 0, group_bytes = 0;
    // fast path for C <= 2: a warp per sequence, graph staged in shared memory
    bool pair = false;
    PairFn pair_fn = nullptr;
    uint32_t rec_bytes = 0, w_bytes = 0, sell_bytes = 0, word_bytes = 0;
    // blocks per SM the fast path reaches with 1..16 warps per block (0: does not fit), and its sizes
    int pair_nb[17] = {0};
    size_t pair_graph_b = 0, pair_warp_b = 0;
    int sm_count = 0;
    // block-per-sequence path with packed words for C <= 4
    bool quad = false;
    QuadFn quad_fn = nullptr;
    uint32_t quad_word_b = 0, quad_cnt_b = 0;
    // sequence-per-lane path for C <= 2: a block keeps a group of 8, 16 or 32 sequences on chip
    bool lane = false;
    LaneFn lane_fn = nullptr;
    int lane_lg = 0;               // log2 of the sequences per group
    uint32_t lane_rec_b = 0, lane_succ_b = 0, lane_word_b = 0, lane_delta_b = 0;
};

// Graph in the order the sequence-per-lane kernel walks it, for one group size (S = 32 / g sub-lanes).
struct LaneLayout {
    bool ok = false;
    int32_t n_bundles = 0;
    int64_t succ_len = 0;                 // entries of the successor array (a multiple of 4)
    void* d_rec32 = nullptr;              // 32-byte records with 32-bit / 64-bit output sizes
    void* d_rec64 = nullptr;
    uint32_t* d_succ = nullptr;
    std::vector<int32_t> h_node;          // node of every slot (-1: none)
    std::vector<uint32_t> h_rec32, h_rec64;   // host copies of the records (durations and caps are patched in)
};


// Records the error text of the calling thread and returns `code`.
int fail(int code, const char* fmt, ...);
// Empties the error text of the calling thread (every entry point starts with this).
void clear_error();
// Counter behind moc_last_launch_count().
int& launch_counter();

#define MOC_CUDA(call)                                                                      \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess)                                                              \
            return moc_host::fail(e_ == cudaErrorMemoryAllocation ? MOC_ERR_NOMEM : MOC_ERR_CUDA, \
                                  "%s: %s", #call, cudaGetErrorString(e_));                 \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

}  // namespace moc_host

struct moc_graph {
    int32_t n = 0;
    int64_t n_edges = 0;  // distinct
    int32_t C = 2;
    uint64_t generation = 0;  // bumped whenever C or the per-node caps change: caches built before are stale
    int device = 0;
    int sm_count = 0;
    size_t smem_optin = 0;
    int64_t sum_m = 0, sum_w = 0;
    int32_t* d_succ_start = nullptr;
    int32_t* d_succ = nullptr;
    int32_t* d_pred_start = nullptr;     // predecessor lists (CSR), for the incremental evaluation
    int32_t* d_pred = nullptr;
    int64_t sink_m = 0;                   // sum of m over the nodes without successors
    int32_t max_indeg = 0;                // largest number of predecessors of a node
    int64_t* d_w = nullptr;
    int64_t* d_m64 = nullptr;
    int32_t* d_m32 = nullptr;
    int32_t want_G = 0, want_gpc = 0;
    int32_t want_kind = 0, want_a = 0, want_b = 0;   // moc_graph_set_kernel
    moc_host::LaneLayout lane[3];         // groups of 32, 16, 8 sequences
    uint4* d_order32 = nullptr;           // block-per-sequence kernel: 32-byte node records by falling out-degree (32- / 64-bit m)
    uint4* d_order64 = nullptr;
    uint16_t* d_succ16 = nullptr;         // ... and the successors beyond a node's eighth
    cudaEvent_t ev_before = nullptr, ev_after = nullptr;  // measurement hook around the evaluation kernel
    // sliced-ELL successor lists in out-degree order (null when the fast path cannot serve the graph)
    int32_t sell_len = 0, n_tiles = 0;
    void* d_rec32 = nullptr;  // node records with 32-bit / 64-bit output sizes
    void* d_rec64 = nullptr;
    uint64_t* d_wslot = nullptr;
    int32_t* d_cap = nullptr;             // per-node caps C_v, or null: uniform C
    std::vector<int32_t> h_slot;          // node of every slot of the warp-per-sequence layout (-1: none)
    std::vector<int64_t> h_w;             // durations (host copy, to rebuild d_wslot)
    std::vector<int32_t> h_cap;           // per-node caps (empty: uniform)
    uint32_t* d_sell = nullptr;
    // grow-only scratch; mutable because evaluation takes a const handle
    mutable moc_host::Plan plan_eval, plan_profile;
    mutable int64_t* d_offs = nullptr;
    mutable size_t offs_cap = 0;
    mutable char* d_state = nullptr;
    mutable size_t state_cap = 0;
    mutable int32_t* d_stage_seqs = nullptr;
    mutable size_t stage_seqs_cap = 0;
    mutable uint16_t* d_stage_u16 = nullptr;   // 16-bit node ids as they arrive from the host
    mutable size_t stage_u16_cap = 0;
    mutable char* d_stage_io = nullptr;  // peak | dur | status | lens
    mutable size_t stage_io_cap = 0;
    mutable char* h_stage = nullptr;     // pinned: peak | dur | status as they come back in one copy
    mutable size_t h_stage_cap = 0;
    mutable cudaStream_t copy_stream = nullptr;   // host entry points: brings the next chunk while one is evaluated
    mutable cudaEvent_t chunk_ev[9] = {};
};


namespace moc_host {

// Enqueues the evaluation of B rows that start at seqs + offs[b] (offs: DEVICE, B+1 entries, the
// last one the number of ints readable from seqs).  The handle's plan is made on first use and its
// global workspace grown if the graph needs one.  Same outputs as moc_eval_batch.
int eval_rows(const moc_graph* g, const int64_t* offs, const int32_t* seqs, const int32_t* lens, int32_t B,
              int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible, cudaStream_t st);

}  // namespace moc_host

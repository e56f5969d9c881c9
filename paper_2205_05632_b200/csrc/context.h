// Host-side context of a COMP-AMS handle and the kernel launchers it drives.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/compams.h"
#include "common.cuh"

namespace compams {

constexpr int kSmallMax = 4096;    // Top-k blocks up to this size are selected inside one CTA's shared memory
constexpr int kBins1 = 2048;       // radix pass 1: key bits 30..20
constexpr int kBins23 = 1024;      // radix passes 2, 3: key bits 19..10, 9..0
constexpr int kMaxTimed = 4096;    // event pairs kept for per-kernel timing

// Per (worker, large block) Top-k selection state, written by the find kernels.
struct SegState {
    uint32_t prefix;      // high key bits decided so far
    uint32_t k_rem;       // entries still to take among the keys that match the prefix
    uint32_t tau;         // threshold key (after the last pass)
    uint32_t ties_total;  // number of keys equal to tau
    uint32_t ties_take;   // how many of them belong to the kept set
    uint32_t need_order;  // 1 when ties_take < ties_total: the lowest indices must be chosen
    uint32_t emit_count;  // message slots handed out so far
    uint32_t pad;
};

// Block / tile tables shared by the tiled kernels (device pointers).
struct Tables {
    int32_t n;
    int64_t d;
    int32_t M;
    const int64_t* off;        // [M+1] block offsets
    // tiles: every listed block is cut into tiles of kTile coordinates
    int32_t ntiles;            // tiles per worker row
    const int32_t* tile_blk;   // [ntiles] block index b of the tile
    const int32_t* tile_r0;    // [ntiles] first coordinate of the tile, relative to its block
    const int32_t* tile_seg;   // [ntiles] index of the block among the tiled blocks
    const int32_t* seg_tile0;  // [nseg+1] first tile of each tiled block
    int32_t nseg;              // number of tiled blocks (all blocks for Block-Sign, large ones for Top-k)
};

struct BsBuffers {
    float* E;                 // [n, d]
    uint32_t* bits;           // [n, W]
    const int64_t* word_off;  // [M+1]
    int64_t W;
    const float* scales_prev; // [n, M]
    float* scales_cur;        // [n, M]
    double* tile_sum;         // [n, ntiles]
    uint32_t* ticket;         // [n, M]
    float *gbar, *m, *v, *vhat;
};

struct TopkBuffers {
    float* E;                  // [n, d]
    int32_t* idx;              // [n, K]
    float* val;                // [n, K]
    int64_t K;
    const int64_t* seg_off;    // [M+1] prefix sums of k_b
    const int32_t* small_blk;  // [nsmall] blocks handled by the shared-memory kernel
    int32_t nsmall;
    uint32_t* hist;            // [n * nseg, kBins1]
    SegState* seg;             // [n * nseg]
    uint32_t* tile_ties;       // [n, ntiles]
    double* acc;               // [d] binary64 accumulator of the worker average
    uint32_t* status;
    float *gbar, *m, *v, *vhat;
};

}  // namespace compams

struct compams_context {
    int device = 0;
    int32_t n = 0;
    int64_t d = 0;
    int32_t M = 0;
    int32_t compressor = 0;
    double k_ratio = 1.0;
    bool identity = false;     // Top-k with every k_b == d_b
    compams::HyperParams hp{};
    cudaStream_t stream = nullptr;
    int num_sms = 148;

    std::vector<int64_t> off;      // host copy of the block offsets
    std::vector<int64_t> seg_off;  // host prefix sums of k_b (Top-k)
    int64_t K = 0;
    int64_t W = 0;

    compams::Tables tab{};
    compams::BsBuffers bs{};
    compams::TopkBuffers tk{};
    float* scales[2] = {nullptr, nullptr};
    int scales_cur = 0;
    bool e_is_x = false;  // Block-Sign: E holds the corrected gradient x of the last step, not e

    // common device state
    float *E = nullptr, *m = nullptr, *v = nullptr, *vhat = nullptr, *gbar = nullptr;
    uint32_t* status = nullptr;
    int64_t* d_off = nullptr;
    int64_t* d_seg_off = nullptr;
    int64_t* d_word_off = nullptr;
    std::vector<void*> owned;  // every device allocation, for destroy

    // staging for compams_step_host
    float* stage_grads = nullptr;
    float* stage_theta = nullptr;

    // profiling
    uint32_t prof_mask = 0;
    int prof_used = 0;
    std::vector<cudaEvent_t> ev_start, ev_stop;
    std::vector<int> ev_kernel;
    int64_t launches = 0;
};

namespace compams {

// Each launcher enqueues one kernel on ctx->stream and returns the launch status.
cudaError_t launch_dense_mean_amsgrad(compams_context* c, const float* grads, float* theta);
cudaError_t launch_bs_sweep(compams_context* c, const float* grads);
cudaError_t launch_bs_apply(compams_context* c, float* theta);
cudaError_t launch_bs_materialize(compams_context* c);
cudaError_t launch_topk_small(compams_context* c, const float* grads);
cudaError_t launch_topk_sweep(compams_context* c, const float* grads);
cudaError_t launch_topk_hist(compams_context* c, int pass);
cudaError_t launch_topk_find(compams_context* c, int pass);
cudaError_t launch_topk_collect(compams_context* c);
cudaError_t launch_topk_ties(compams_context* c);
cudaError_t launch_topk_scatter(compams_context* c);
cudaError_t launch_amsgrad(compams_context* c, float* theta);

}  // namespace compams

// Host-side context of a COMP-AMS handle and the kernel launchers it drives.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/compams.h"
#include "common.cuh"

#ifndef COMPAMS_CHAIN_MAX
#define COMPAMS_CHAIN_MAX ((int64_t)1 << 28)
#endif

namespace compams {

constexpr int kSmallMax = 4096;    // Top-k blocks up to this size are selected inside one CTA's shared memory
constexpr int kBins1 = 2048;       // radix pass 1: key bits 30..20
constexpr int kBins23 = 1024;      // radix passes 2, 3: key bits 19..10, 9..0
constexpr int kBucketSpan = 1024;  // coordinates per server bucket: one CTA of the Top-k AMSGrad kernel
constexpr int kMaxTimed = 4096;    // event pairs kept for per-kernel timing
constexpr int64_t kMaxD = ((int64_t)1 << 31) - 4 * kTile;  // largest d: tile coordinates are 32-bit and overshoot a block's end

constexpr uint32_t kNoPrediction = 0xffffffffu;  // tau_hat value that no key reaches
constexpr int kTileCand = 1024;          // candidates one tile can stage in shared memory
constexpr int kSurvCap = 1536;           // threshold-bin candidates a select can rank in shared memory
constexpr int kSurvCapBig = 65536;       // threshold-bin candidates of a long list (kept in global memory)
constexpr int kSurvSmem = 4096;          // ... of which this many fit the finishing CTA's shared memory
constexpr int kRankMax = 256;            // ... and up to this many are ranked pair by pair
constexpr int kSelBins = 4096;           // bins of the candidate select's first histogram
constexpr int64_t kChainMaxElems = COMPAMS_CHAIN_MAX;  // n d up to which a step's kernels are chained
constexpr int kSelectSingleMax = 98304;  // candidate capacity up to which one CTA handles a segment

// Per (worker, large block) Top-k selection state.
struct SegState {
    // candidate path
    uint32_t tau_hat;     // keys >= tau_hat are collected as candidates by the sweep (kNoPrediction: none)
    uint32_t tau_prev;    // threshold key of the previous step (kNoPrediction: unknown)
    uint32_t cand_count;  // candidates counted by the sweep (may exceed what was stored)
    uint32_t sel_shift;   // log2 of the bin width of the select's first histogram
    uint32_t fallback;    // 1: the candidate path could not decide this step, the dense passes run
    uint32_t edge;        // dense path: bin edge chosen as the next tau_hat
    // dense radix passes
    uint32_t prefix;      // high key bits decided so far
    uint32_t k_rem;       // entries still to take among the keys that match the prefix
    uint32_t tau;         // threshold key (after the last pass)
    uint32_t ties_total;  // number of keys equal to tau
    uint32_t ties_take;   // how many of them belong to the kept set
    uint32_t need_order;  // 1 when ties_take < ties_total: the lowest indices must be chosen
    uint32_t emit_count;  // message slots handed out so far
    uint32_t sel_ready;   // multi-CTA select: the threshold bin has been found, the emit kernel may run
    uint32_t boost;       // the candidate margin is doubled this many times (raised when a list came up short)
    uint32_t streak;      // selections decided inside the list since the margin last changed
    uint32_t hold;        // a doubling is taken back after 32 << hold such selections in a row
    uint32_t probing;     // 1: the margin was last changed by taking a doubling back
};

// Block / tile tables shared by the tiled kernels (device pointers).
struct Tables {
    int32_t n;
    int64_t d;
    int32_t M;
    const int64_t* off;     // [M+1] block offsets
    int32_t ntiles;         // tiles per worker row
    const TileInfo* tiles;  // [ntiles]
    int32_t nseg;           // number of tiled blocks (all blocks for Block-Sign, large ones for Top-k)
    const SegInfo* segs;    // [nseg]
};

struct BsBuffers {
    float* E;                 // [n, d]
    uint32_t* bits;           // [n, W]
    const int64_t* word_off;  // [M+1]
    int64_t W;
    const float* scales_prev; // [n, M]
    float* scales_cur;        // [n, M]
    double* tile_sum;         // [n, ntiles]
    uint2* edge;              // [n, ntiles] a tile's share of the sign words it has in common with its neighbours
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
    uint2* cand;               // [n, cand_total] (coordinate, bits of x) pairs collected by the sweep
    int64_t cand_total;        // candidate slots per worker
    uint32_t* dense_count;     // [1] segments currently marked for the dense passes
    uint32_t* sel_hist;        // [n * long lists, kSelBins] histogram a long list's slices add into
    uint32_t* sel_ticket;      // [n * long lists, 2] slices arrived; threshold-bin candidates appended
    uint2* sel_surv;           // [n * long lists, kSurvCapBig] threshold-bin candidates of a long list
    double* acc;               // [d] binary64 accumulator, used only by entries that overflow their bucket
    uint32_t* thr;             // [n * nseg] bits of the magnitude from which on the segment's last selection kept
                               // everything: E still holds x at those elements; their e is 0
    int use_thr;               // 1: E holds the last step's x at the kept coordinates (the sweep treats them as 0)
    uint2* bucket;             // [nbucket, bucket_cap] (coordinate inside the bucket, bits of x) per kept entry
    uint32_t* bcount;          // [nbucket] entries appended this step (may exceed bucket_cap)
    uint32_t* bdirty;          // [nbucket] 1: some entries of this bucket went to acc instead
    int32_t bucket_cap;
    int32_t nbucket;
    uint32_t* status;
    float *gbar, *m, *v, *vhat;
};

}  // namespace compams

struct compams_context {
    int device = 0;
    int32_t n = 0;        // workers whose gradients and error accumulators this handle holds
    int32_t n_total = 0;  // workers the server averages over (> n when the workers are sharded over several handles)
    int32_t row0 = 0;     // index of this handle's first worker among the n_total
    int64_t d = 0;
    bool chain = false;      // n d <= kChainMaxElems: the kernels of a step are launched as programmatic dependents
    bool grad_bf16 = false;  // the gradients of the call being enqueued are bfloat16 (16-bit patterns), not fp32
    int32_t M = 0;
    int32_t compressor = 0;
    double k_ratio = 1.0;
    bool identity = false;     // Top-k or Random-k with every k_b == d_b
    bool record_gbar = false;  // the server kernels also write gbar_t (an intermediate; 4 bytes per coordinate and step)
    bool randk = false;        // Random-k: the kept sets are drawn, not selected
    uint64_t seed = 0;         // Random-k: seed of the index sets
    uint64_t iter = 0;         // iterations so far (Random-k keys its sets by the iteration index, from 1)
    bool sparse() const { return compressor != COMPAMS_BLOCKSIGN; }  // Top-k or Random-k: (index, value) messages
    compams::HyperParams hp{};
    cudaStream_t stream = nullptr;
    int num_sms = 148;

    std::vector<int64_t> off;      // host copy of the block offsets
    std::vector<int64_t> seg_off;  // host prefix sums of k_b (Top-k)
    std::vector<uint32_t> seg_cap_host;  // candidate capacity of every tiled block (Top-k)
    int64_t K = 0;
    int64_t W = 0;

    compams::Tables tab{};
    compams::SegParams segp{};  // kernel-argument copy of the tiled blocks (nseg = 0: not usable)
    compams::BsBuffers bs{};
    compams::TopkBuffers tk{};
    int32_t* sel_small = nullptr;  // tiled blocks whose candidate lists one CTA selects from
    int32_t* sel_big = nullptr;    // tiled blocks whose candidate lists are cut into slices over many CTAs
    int n_sel_small = 0, n_sel_big = 0;
    int sel_parts = 1;  // slices a long candidate list is cut into
    std::vector<compams::SegState> seg_init_host;  // Top-k: the segments' state before the first step (set_state restores it)
    uint32_t dense_count_init = 0;
    uint64_t steps_done = 0;
    bool e_mask_pending = false;  // Top-k: E still holds x at the coordinates kept in the last step
    int dense_grid = 0;  // CTAs of the cooperative dense-pass kernel (0: not yet sized)
    float* scales[2] = {nullptr, nullptr};
    int scales_cur = 0;
    bool e_is_x = false;  // Block-Sign: E holds the corrected gradient x of the last step, not e
    bool compressed = false;  // compams_compress has run and its compams_apply has not: the step is half done


    // common device state
    float *E = nullptr, *m = nullptr, *v = nullptr, *vhat = nullptr, *gbar = nullptr;
    uint32_t* status = nullptr;
    int64_t* d_off = nullptr;
    int64_t* d_seg_off = nullptr;
    int64_t* d_word_off = nullptr;
    std::vector<void*> owned;  // every device allocation of the library's own, for destroy
    // state placed in caller memory (compams_create_in_workspace), or only sized (compams_workspace_bytes)
    bool plan_only = false;          // nothing is allocated or touched: the buffers are only added up
    unsigned char* ws = nullptr;     // caller's device memory the buffers are cut from (null: cudaMalloc each)
    size_t ws_bytes = 0, ws_used = 0;

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

// Adds a successfully enqueued kernel to the handle's launch count; passes the launch status through.
inline cudaError_t counted(compams_context* c, cudaError_t e) {
    if (e == cudaSuccess) ++c->launches;
    return e;
}

// Each launcher enqueues its kernel(s) on ctx->stream and returns the launch status.
cudaError_t launch_dense_mean_amsgrad(compams_context* c, const void* grads, float* theta);
cudaError_t launch_bs_sweep(compams_context* c, const void* grads);
cudaError_t launch_bs_scales(compams_context* c);
cudaError_t launch_bs_apply(compams_context* c, float* theta);
cudaError_t launch_bs_materialize(compams_context* c);
cudaError_t launch_topk_small(compams_context* c, const void* grads);
cudaError_t launch_topk_sweep(compams_context* c, const void* grads);
cudaError_t launch_topk_select(compams_context* c);
cudaError_t launch_topk_dense(compams_context* c);
cudaError_t launch_topk_materialize(compams_context* c);
cudaError_t launch_topk_scatter(compams_context* c, bool close);
cudaError_t launch_randk_emit(compams_context* c, bool deliver);
cudaError_t launch_amsgrad(compams_context* c, float* theta);

}  // namespace compams

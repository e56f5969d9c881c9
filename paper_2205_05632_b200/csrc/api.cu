// C ABI of the COMP-AMS library (see include/compams.h): argument checks, state allocation,
// the per-step launch sequence and the inspection calls.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>

#include "context.h"

using namespace compams;

namespace {

thread_local std::string g_last_cuda_error;

int cuda_fail(cudaError_t e, const char* what) {
    g_last_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    return COMPAMS_ERR_CUDA;
}

#define CU(call)                                          \
    do {                                                  \
        cudaError_t _e = (call);                          \
        if (_e != cudaSuccess) return cuda_fail(_e, #call); \
    } while (0)

template <typename T>
int dev_alloc(compams_context* c, T** out, size_t count, bool zero = true) {
    *out = nullptr;
    if (count == 0) count = 1;
    if (c->plan_only || c->ws) {
        // buffers are cut from one region, each on a 256-byte boundary
        const size_t off = (c->ws_used + 255) & ~(size_t)255;
        c->ws_used = off + count * sizeof(T);
        if (c->plan_only) return COMPAMS_OK;
        if (c->ws_used > c->ws_bytes) return COMPAMS_ERR_INVALID_ARG;  // the caller's region is too small
        if (zero) CU(cudaMemsetAsync(c->ws + off, 0, count * sizeof(T), c->stream));
        *out = (T*)(c->ws + off);
        return COMPAMS_OK;
    }
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, count * sizeof(T));
    if (e != cudaSuccess) {
        g_last_cuda_error = std::string("cudaMalloc: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return COMPAMS_ERR_ALLOC;
    }
    c->owned.push_back(p);
    if (zero) CU(cudaMemsetAsync(p, 0, count * sizeof(T), c->stream));
    *out = (T*)p;
    return COMPAMS_OK;
}

template <typename T>
int dev_upload(compams_context* c, T** out, const std::vector<T>& host) {
    int rc = dev_alloc(c, out, host.size(), false);
    if (rc) return rc;
    if (!host.empty() && !c->plan_only) CU(cudaMemcpy(*out, host.data(), host.size() * sizeof(T), cudaMemcpyHostToDevice));
    return COMPAMS_OK;
}

#define RC(call)              \
    do {                      \
        int _rc = (call);     \
        if (_rc) return _rc;  \
    } while (0)

// Every enqueueing call must run with the handle's device current: its buffers live there, and on the
// default stream a launch goes to whatever device is current.
int on_handle_device(const compams_context* c) {
    int dev = -1;
    CU(cudaGetDevice(&dev));
    return dev == c->device ? COMPAMS_OK : COMPAMS_ERR_INVALID_ARG;
}

int64_t kept_per_block(double k_ratio, int64_t d_b) {
    int64_t k = (int64_t)std::floor(k_ratio * (double)d_b);
    if (k < 1) k = 1;
    if (k > d_b) k = d_b;
    return k;
}

// Cuts the listed blocks into tiles of kTile coordinates and uploads the tile and segment tables.
// For Top-k (`topk` true) every listed block also gets its message slots and candidate capacity.
int build_tiles(compams_context* c, const std::vector<int32_t>& blocks, bool topk) {
    std::vector<TileInfo> tiles;
    std::vector<SegInfo> segs;
    int64_t cand_total = 0;
    for (size_t s = 0; s < blocks.size(); ++s) {
        const int32_t b = blocks[s];
        const int64_t len = c->off[b + 1] - c->off[b];
        // The sweeps shift a worker's tiles down by the phase of the block's first element within a
        // 128-byte line, (i d + o) mod 32, so that every warp access covers whole lines; the block
        // needs enough tiles for the largest shift among the workers.
        int64_t smax = 0;
        for (int32_t i = 0; i < c->n && smax < 31; ++i) smax = std::max<int64_t>(smax, ((int64_t)i * c->d + c->off[b]) & 31);
        const int64_t nt = (len + smax + kTile - 1) / kTile;
        if ((int64_t)tiles.size() + nt > (int64_t)0x7fffffff) return COMPAMS_ERR_INVALID_ARG;
        SegInfo si{};
        si.o = c->off[b];
        si.len = (int32_t)len;
        si.blk = b;
        si.tile0 = (int32_t)tiles.size();
        si.ntile_b = (int32_t)nt;
        if (topk) {
            const int64_t kb = c->seg_off[(size_t)b + 1] - c->seg_off[(size_t)b];
            si.slot0 = c->seg_off[(size_t)b];
            si.kb = (uint32_t)kb;
            // the candidate path pays off for sparse selections only: at most 1/32 of the block kept
            int64_t cap = (!c->randk && kb * 32 <= len) ? 8 * kb + 1024 : 0;
            if (cap > len) cap = len;
            si.cap = (uint32_t)cap;
            si.cand_off = cand_total;
            cand_total += cap;
        }
        for (int64_t r0 = 0; r0 < nt * kTile; r0 += kTile) {
            TileInfo ti{};
            ti.o = c->off[b];
            ti.len = (int32_t)len;
            ti.r0 = (int32_t)r0;
            ti.blk = b;
            ti.seg = (int32_t)s;
            ti.tile0 = si.tile0;
            ti.ntile_b = si.ntile_b;
            tiles.push_back(ti);
        }
        segs.push_back(si);
    }
    TileInfo* d_tiles;
    SegInfo* d_segs;
    RC(dev_upload(c, &d_tiles, tiles));
    RC(dev_upload(c, &d_segs, segs));
    c->tab.ntiles = (int32_t)tiles.size();
    c->tab.tiles = d_tiles;
    c->tab.nseg = (int32_t)blocks.size();
    c->tab.segs = d_segs;
    c->segp = SegParams{};
    if (segs.size() <= (size_t)kParamSegs) {
        c->segp.nseg = (int32_t)segs.size();
        for (size_t s = 0; s < segs.size(); ++s) {
            c->segp.tile0[s] = segs[s].tile0;
            c->segp.len[s] = segs[s].len;
            c->segp.blk[s] = segs[s].blk;
            c->segp.o[s] = segs[s].o;
        }
        c->segp.tile0[segs.size()] = (int32_t)tiles.size();
    }
    c->tk.cand_total = cand_total;
    c->seg_cap_host.clear();
    for (const SegInfo& si : segs) c->seg_cap_host.push_back(si.cap);
    if (topk) {
        // Short candidate lists get one CTA each; a long one is cut into slices that many CTAs work on
        // (two kernels that meet through a global histogram). Slices finish one list sooner, but with
        // many long lists (layer-wise selection over many workers) one CTA per list has the higher
        // throughput.
        size_t n_long = 0;
        for (const SegInfo& si : segs) n_long += si.cap > (uint32_t)kSelectSingleMax ? 1 : 0;
        const uint32_t single_max = (n_long * (size_t)c->n >= 64) ? (1u << 20) : (uint32_t)kSelectSingleMax;
        std::vector<int32_t> small_l, big_l;
        for (size_t s = 0; s < segs.size(); ++s) {
            if (segs[s].cap == 0) continue;  // never predicts: always the dense passes, no select needed
            (segs[s].cap <= single_max ? small_l : big_l).push_back((int32_t)s);
        }
        // one-CTA lists are worked on longest first (their CTAs differ in length by the lists' lengths)
        std::stable_sort(small_l.begin(), small_l.end(),
                         [&](int32_t a, int32_t b) { return segs[(size_t)a].cap > segs[(size_t)b].cap; });
        RC(dev_upload(c, &c->sel_small, small_l));
        RC(dev_upload(c, &c->sel_big, big_l));
        c->n_sel_small = (int)small_l.size();
        c->n_sel_big = (int)big_l.size();
        if (c->n_sel_big > 0) {
            // enough slices for about four CTAs per SM over all long lists, and short enough (about
            // 12 K of the expected 2.5 k_b candidates each) that a slice is a few dozen loads per thread
            const int64_t lists = (int64_t)c->n * c->n_sel_big;
            int64_t parts = (4 * (int64_t)c->num_sms + lists - 1) / lists;
            int64_t kb_max = 0;
            for (int32_t sg : big_l) kb_max = std::max<int64_t>(kb_max, segs[(size_t)sg].kb);
            parts = std::max<int64_t>(parts, (5 * kb_max / 2 + 12287) / 12288);
            c->sel_parts = (int)(parts < 1 ? 1 : parts > 1024 ? 1024 : parts);
            RC(dev_alloc(c, &c->tk.sel_hist, (size_t)lists * kSelBins));
            RC(dev_alloc(c, &c->tk.sel_ticket, (size_t)lists * 2));
            RC(dev_alloc(c, &c->tk.sel_surv, (size_t)lists * kSurvCapBig, false));
        }
    }
    return COMPAMS_OK;
}

int init_context(compams_context* c, const int64_t* block_offsets) {
    if (!c->plan_only) {
        CU(cudaGetDevice(&c->device));
        CU(cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device));
    }
    const int32_t n = c->n, M = c->M;
    const int64_t d = c->d;
    c->off.assign(block_offsets, block_offsets + M + 1);
    c->tab.n = n;
    c->tab.d = d;
    c->tab.M = M;
    RC(dev_upload(c, &c->d_off, c->off));
    c->tab.off = c->d_off;

    RC(dev_alloc(c, &c->m, (size_t)d));
    RC(dev_alloc(c, &c->v, (size_t)d));
    RC(dev_alloc(c, &c->vhat, (size_t)d));
    RC(dev_alloc(c, &c->gbar, (size_t)d));
    RC(dev_alloc(c, &c->status, 8));

    if (c->sparse()) {
        c->seg_off.assign((size_t)M + 1, 0);
        bool identity = true;
        for (int32_t b = 0; b < M; ++b) {
            const int64_t db = c->off[b + 1] - c->off[b];
            const int64_t kb = kept_per_block(c->k_ratio, db);
            identity = identity && (kb == db);
            c->seg_off[(size_t)b + 1] = c->seg_off[(size_t)b] + kb;
        }
        c->identity = identity;
        c->K = identity ? 0 : c->seg_off[(size_t)M];
    }

    if (c->sparse() && c->identity) {
        // full-precision distributed AMSGrad: e is identically zero and not stored
    } else if (c->sparse()) {
        RC(dev_alloc(c, &c->E, (size_t)n * (size_t)d));
        RC(dev_upload(c, &c->d_seg_off, c->seg_off));
        std::vector<int32_t> small, large;
        // (Random-k has no selection: every block is tiled for the sweep, none goes to the shared-memory select)
        for (int32_t b = 0; b < M; ++b)
            ((!c->randk && c->off[b + 1] - c->off[b] <= kSmallMax) ? small : large).push_back(b);
        RC(build_tiles(c, large, true));
        TopkBuffers& t = c->tk;
        t.E = c->E;
        t.K = c->K;
        t.seg_off = c->d_seg_off;
        int32_t* d_small;
        RC(dev_upload(c, &d_small, small));
        t.small_blk = d_small;
        t.nsmall = (int32_t)small.size();
        // the messages of all n_total workers: this handle's selection fills its own rows, the other
        // rows are filled by the caller's exchange before compams_apply
        RC(dev_alloc(c, &t.idx, (size_t)c->n_total * (size_t)c->K));
        RC(dev_alloc(c, &t.val, (size_t)c->n_total * (size_t)c->K));
        RC(dev_alloc(c, &t.hist, c->randk ? 1 : (size_t)n * (size_t)c->tab.nseg * kBins1));
        {
            SegState init{};
            init.tau_hat = kNoPrediction;
            init.tau_prev = kNoPrediction;
            std::vector<SegState> seg0((size_t)n * (size_t)c->tab.nseg, init);
            uint32_t never = 0;
            for (uint32_t cap : c->seg_cap_host) never += cap ? 0u : 1u;
            for (size_t k = 0; k < seg0.size(); ++k)
                seg0[k].fallback = c->seg_cap_host[k % (size_t)c->tab.nseg] ? 0u : 1u;
            RC(dev_upload(c, &t.seg, seg0));
            c->seg_init_host = seg0;
            c->dense_count_init = never * (uint32_t)n;
            std::vector<uint32_t> dc(1, never * (uint32_t)n);
            RC(dev_upload(c, &t.dense_count, dc));
        }
        RC(dev_alloc(c, &t.tile_ties, c->randk ? 1 : (size_t)n * (size_t)c->tab.ntiles));
        RC(dev_alloc(c, &t.cand, (size_t)n * (size_t)t.cand_total, false));
        RC(dev_alloc(c, &t.acc, (size_t)d));
        {
            std::vector<uint32_t> none((size_t)n * (size_t)std::max(c->tab.nseg, 1), 0xffffffffu);
            RC(dev_upload(c, &t.thr, none));
        }
        {
            // kept entries are handed to the server grouped by coordinate range: room for four times the
            // average load of a bucket, the rare excess goes through the binary64 accumulator
            t.nbucket = (int32_t)((d + kBucketSpan - 1) / kBucketSpan);
            const int64_t avg = ((int64_t)c->n_total * c->K + t.nbucket - 1) / t.nbucket;
            int64_t cap = 4 * avg + 64;
            if (cap > (int64_t)c->n_total * kBucketSpan) cap = (int64_t)c->n_total * kBucketSpan;
            t.bucket_cap = (int32_t)((cap + 31) / 32 * 32);
            RC(dev_alloc(c, &t.bucket, (size_t)t.nbucket * (size_t)t.bucket_cap, false));
            RC(dev_alloc(c, &t.bcount, (size_t)t.nbucket));
            RC(dev_alloc(c, &t.bdirty, (size_t)t.nbucket));
        }
        t.status = c->status;
        t.gbar = nullptr;  // set by compams_record_average
        t.m = c->m;
        t.v = c->v;
        t.vhat = c->vhat;
    } else {
        RC(dev_alloc(c, &c->E, (size_t)n * (size_t)d));
        std::vector<int32_t> all((size_t)M);
        for (int32_t b = 0; b < M; ++b) all[(size_t)b] = b;
        RC(build_tiles(c, all, false));
        std::vector<int64_t> word_off((size_t)M + 1, 0);
        for (int32_t b = 0; b < M; ++b)
            word_off[(size_t)b + 1] = word_off[(size_t)b] + (c->off[b + 1] - c->off[b] + 31) / 32;
        c->W = word_off[(size_t)M];
        RC(dev_upload(c, &c->d_word_off, word_off));
        if (c->W > (int64_t)INT32_MAX) c->segp.nseg = 0;  // word offsets would not fit the kernel-argument copy
        for (int32_t sg = 0; sg < c->segp.nseg; ++sg) c->segp.wofs[sg] = (int32_t)word_off[(size_t)c->segp.blk[sg]];
        BsBuffers& s = c->bs;
        s.E = c->E;
        s.word_off = c->d_word_off;
        s.W = c->W;
        // sign words and scales of all n_total workers (see the Top-k messages above)
        RC(dev_alloc(c, &s.bits, (size_t)c->n_total * (size_t)c->W));
        RC(dev_alloc(c, &c->scales[0], (size_t)c->n_total * (size_t)M));
        RC(dev_alloc(c, &c->scales[1], (size_t)c->n_total * (size_t)M));
        RC(dev_alloc(c, &s.tile_sum, (size_t)n * (size_t)c->tab.ntiles));
        RC(dev_alloc(c, &s.edge, (size_t)n * (size_t)c->tab.ntiles));
        s.gbar = nullptr;  // set by compams_record_average
        s.m = c->m;
        s.v = c->v;
        s.vhat = c->vhat;
    }
    if (!c->plan_only) CU(cudaDeviceSynchronize());
    return COMPAMS_OK;
}

void free_context(compams_context* c) {
    for (void* p : c->owned) cudaFree(p);
    c->owned.clear();
    if (c->stage_grads) cudaFree(c->stage_grads);
    if (c->stage_theta) cudaFree(c->stage_theta);
    for (cudaEvent_t e : c->ev_start) cudaEventDestroy(e);
    for (cudaEvent_t e : c->ev_stop) cudaEventDestroy(e);
    delete c;
}

// Runs one launcher, optionally bracketed by an event pair for per-kernel timing.
template <typename F>
int run_kernel(compams_context* c, int kernel, F&& launch) {
    const bool timed = (c->prof_mask >> kernel) & 1u;
    int slot = -1;
    if (timed && c->prof_used < kMaxTimed) {
        slot = c->prof_used++;
        if ((size_t)slot >= c->ev_start.size()) {
            cudaEvent_t a, b;
            CU(cudaEventCreate(&a));
            CU(cudaEventCreate(&b));
            c->ev_start.push_back(a);
            c->ev_stop.push_back(b);
            c->ev_kernel.push_back(kernel);
        }
        c->ev_kernel[(size_t)slot] = kernel;
        CU(cudaEventRecord(c->ev_start[(size_t)slot], c->stream));
    }
    cudaError_t e = launch();  // the launchers count the kernels they enqueue in c->launches
    if (e != cudaSuccess) return cuda_fail(e, compams_kernel_name(kernel));
    if (slot >= 0) CU(cudaEventRecord(c->ev_stop[(size_t)slot], c->stream));
    return COMPAMS_OK;
}

// Worker side of one iteration (Algorithm 2, the workers' loop) for this handle's workers: x = g + e, the
// compression, the residual; the compressed gradients land in this handle's rows of the message buffers.
int compress_device(compams_context* c, const void* grads) {
    ++c->steps_done;
    ++c->iter;
    if (c->compressor == COMPAMS_BLOCKSIGN) {
        c->scales_cur ^= 1;
        RC(run_kernel(c, COMPAMS_K_BS_SWEEP, [&] { return launch_bs_sweep(c, grads); }));
        c->e_is_x = true;
        RC(run_kernel(c, COMPAMS_K_BS_SCALES, [&] { return launch_bs_scales(c); }));
        return COMPAMS_OK;
    }
    // a selection leaves x in E at the coordinates it keeps, and the pair that delimits them; their e is zeroed
    // when E is next read (by the next sweep, or by topk_materialize when the caller asks for E)
    c->tk.use_thr = c->e_mask_pending ? 1 : 0;
    if (c->randk) {
        // no selection: the sweep leaves x in E, then every message slot fetches the x of its drawn coordinate and
        // zeroes it; with all workers in this handle the pairs go to the server in the same kernel, otherwise
        // compams_apply delivers the exchanged messages
        RC(run_kernel(c, COMPAMS_K_TOPK_SWEEP, [&] { return launch_topk_sweep(c, grads); }));
        RC(run_kernel(c, COMPAMS_K_RANDK_EMIT, [&] { return launch_randk_emit(c, c->n == c->n_total); }));
        return COMPAMS_OK;
    }
    if (c->tk.nsmall > 0) RC(run_kernel(c, COMPAMS_K_TOPK_SMALL, [&] { return launch_topk_small(c, grads); }));
    if (c->tab.ntiles > 0) {
        RC(run_kernel(c, COMPAMS_K_TOPK_SWEEP, [&] { return launch_topk_sweep(c, grads); }));
        RC(run_kernel(c, COMPAMS_K_TOPK_SELECT, [&] { return launch_topk_select(c); }));
        RC(run_kernel(c, COMPAMS_K_TOPK_DENSE, [&] { return launch_topk_dense(c); }));
        c->e_mask_pending = true;
    }
    return COMPAMS_OK;
}

// Server side (Algorithm 2, the server's part): average of the n_total compressed gradients and AMSGrad.
int apply_device(compams_context* c, float* theta) {
    if (c->compressor == COMPAMS_BLOCKSIGN) {
        return run_kernel(c, COMPAMS_K_BS_APPLY, [&] { return launch_bs_apply(c, theta); });
    }
    // (a Random-k step with every worker in this handle has delivered its messages already)
    if (!(c->randk && c->n == c->n_total))
        RC(run_kernel(c, COMPAMS_K_TOPK_SCATTER, [&] { return launch_topk_scatter(c, !c->randk); }));
    RC(run_kernel(c, COMPAMS_K_AMSGRAD, [&] { return launch_amsgrad(c, theta); }));
    return COMPAMS_OK;
}

int step_device(compams_context* c, const void* grads, float* theta) {
    if (c->sparse() && c->identity) {
        ++c->steps_done;
        ++c->iter;
        return run_kernel(c, COMPAMS_K_DENSE_MEAN_AMSGRAD, [&] { return launch_dense_mean_amsgrad(c, grads, theta); });
    }
    RC(compress_device(c, grads));
    return apply_device(c, theta);
}

// `ws` null: every buffer is the library's own allocation. `ws` non-null: the buffers are cut from the caller's
// region of `ws_bytes` bytes. `plan` non-null: nothing is created; *plan receives the bytes such a region needs.
int create_handle(compams_handle* out, int32_t n, int32_t n_total, int32_t row0, int64_t d, const int64_t* block_offsets,
                  int32_t num_blocks, int32_t compressor, double k_ratio, float lr, float beta1, float beta2, float eps,
                  void* ws = nullptr, size_t ws_bytes = 0, size_t* plan = nullptr) {
    if ((!out && !plan) || !block_offsets) return COMPAMS_ERR_INVALID_ARG;
    // the tiled kernels address a block with 32-bit coordinates that may run up to two tiles past its end
    if (n < 1 || n_total > 65535 || row0 < 0 || (int64_t)row0 + n > n_total || d < 1 || d > kMaxD ||
        num_blocks < 1 || (int64_t)num_blocks > d)
        return COMPAMS_ERR_INVALID_ARG;
    if (compressor != COMPAMS_TOPK && compressor != COMPAMS_BLOCKSIGN && compressor != COMPAMS_RANDK)
        return COMPAMS_ERR_INVALID_ARG;
    if (compressor != COMPAMS_BLOCKSIGN && !(k_ratio > 0.0 && k_ratio <= 1.0)) return COMPAMS_ERR_INVALID_ARG;
    if (!(lr == lr) || !(beta1 == beta1) || !(beta2 == beta2) || !(eps == eps)) return COMPAMS_ERR_INVALID_ARG;
    if (block_offsets[0] != 0 || block_offsets[num_blocks] != d) return COMPAMS_ERR_INVALID_ARG;
    for (int32_t b = 0; b < num_blocks; ++b)
        if (block_offsets[b + 1] <= block_offsets[b]) return COMPAMS_ERR_INVALID_ARG;

    compams_context* c = new (std::nothrow) compams_context();
    if (!c) return COMPAMS_ERR_ALLOC;
    c->n = n;
    c->n_total = n_total;
    c->row0 = row0;
    c->d = d;
    c->M = num_blocks;
    c->compressor = compressor;
    c->k_ratio = (compressor != COMPAMS_BLOCKSIGN) ? k_ratio : 1.0;
    c->randk = compressor == COMPAMS_RANDK;
    c->hp.lr = lr;
    c->hp.beta1 = beta1;
    c->hp.beta2 = beta2;
    c->hp.omb1 = 1.0f - beta1;
    c->hp.omb2 = 1.0f - beta2;
    c->hp.eps = eps;
    c->chain = (int64_t)n * d <= kChainMaxElems;
    c->hp.nf = (float)n_total;
    c->hp.inv_nf = ((n_total & (n_total - 1)) == 0) ? 1.0f / (float)n_total : 0.0f;
    c->plan_only = plan != nullptr;
    c->ws = (unsigned char*)ws;
    c->ws_bytes = ws_bytes;
    int rc;
    try {
        rc = init_context(c, block_offsets);
    } catch (const std::bad_alloc&) {
        rc = COMPAMS_ERR_ALLOC;
    }
    // sharded workers exchange compressed gradients; the uncompressed mode (k = d) has none to exchange
    if (!rc && n != n_total && c->identity) rc = COMPAMS_ERR_INVALID_ARG;
    if (rc || plan) {
        if (!rc) *plan = (c->ws_used + 255) & ~(size_t)255;
        free_context(c);
        return rc;
    }
    *out = c;
    return COMPAMS_OK;
}

}  // namespace

extern "C" {

int compams_create(compams_handle* out, int32_t n, int64_t d, const int64_t* block_offsets, int32_t num_blocks,
                   int32_t compressor, double k_ratio, float lr, float beta1, float beta2, float eps) {
    return create_handle(out, n, n, 0, d, block_offsets, num_blocks, compressor, k_ratio, lr, beta1, beta2, eps);
}

int compams_create_sharded(compams_handle* out, int32_t n_local, int32_t n_total, int32_t first_worker, int64_t d,
                           const int64_t* block_offsets, int32_t num_blocks, int32_t compressor, double k_ratio, float lr,
                           float beta1, float beta2, float eps) {
    return create_handle(out, n_local, n_total, first_worker, d, block_offsets, num_blocks, compressor, k_ratio, lr, beta1,
                         beta2, eps);
}

int compams_workspace_bytes(size_t* bytes, int32_t n_local, int32_t n_total, int64_t d, const int64_t* block_offsets,
                            int32_t num_blocks, int32_t compressor, double k_ratio) {
    if (!bytes) return COMPAMS_ERR_INVALID_ARG;
    return create_handle(nullptr, n_local, n_total, 0, d, block_offsets, num_blocks, compressor, k_ratio, 0.0f, 0.0f, 0.0f,
                         0.0f, nullptr, 0, bytes);
}

int compams_create_in_workspace(compams_handle* out, void* workspace, size_t workspace_bytes, int32_t n_local,
                                int32_t n_total, int32_t first_worker, int64_t d, const int64_t* block_offsets,
                                int32_t num_blocks, int32_t compressor, double k_ratio, float lr, float beta1, float beta2,
                                float eps) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return COMPAMS_ERR_INVALID_ARG;
    return create_handle(out, n_local, n_total, first_worker, d, block_offsets, num_blocks, compressor, k_ratio, lr, beta1,
                         beta2, eps, workspace, workspace_bytes);
}

static int compress_any(compams_handle c, const void* grads, bool bf16) {
    if (!c || !grads || (reinterpret_cast<uintptr_t>(grads) & (bf16 ? 1u : 3u))) return COMPAMS_ERR_INVALID_ARG;
    if (c->sparse() && c->identity) return COMPAMS_ERR_INVALID_ARG;  // k = d: nothing is compressed
    if (c->compressed) return COMPAMS_ERR_INVALID_ARG;  // the previous compress has not been applied yet
    RC(on_handle_device(c));
    c->grad_bf16 = bf16;
    int rc;
    try {
        rc = compress_device(c, grads);
    } catch (const std::bad_alloc&) {
        rc = COMPAMS_ERR_ALLOC;
    }
    if (!rc) c->compressed = true;
    return rc;
}

int compams_compress(compams_handle c, const float* grads) { return compress_any(c, grads, false); }
int compams_compress_bf16(compams_handle c, const void* grads_bf16) { return compress_any(c, grads_bf16, true); }

int compams_apply(compams_handle c, float* theta) {
    if (!c || !theta || (reinterpret_cast<uintptr_t>(theta) & 15u)) return COMPAMS_ERR_INVALID_ARG;
    if (c->sparse() && c->identity) return COMPAMS_ERR_INVALID_ARG;
    if (!c->compressed) return COMPAMS_ERR_INVALID_ARG;  // nothing to apply: compams_compress comes first
    RC(on_handle_device(c));
    c->compressed = false;
    try {
        return apply_device(c, theta);
    } catch (const std::bad_alloc&) {
        return COMPAMS_ERR_ALLOC;
    }
}

static int step_any(compams_handle c, const void* grads, float* theta, bool bf16) {
    if (!c || !grads || !theta) return COMPAMS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(grads) & (bf16 ? 1u : 3u)) || (reinterpret_cast<uintptr_t>(theta) & 15u))
        return COMPAMS_ERR_INVALID_ARG;
    if (c->n != c->n_total) return COMPAMS_ERR_INVALID_ARG;  // the other workers' messages have to be exchanged first
    if (c->compressed) return COMPAMS_ERR_INVALID_ARG;       // a compams_compress is waiting for its compams_apply
    RC(on_handle_device(c));
    c->grad_bf16 = bf16;
    try {
        return step_device(c, grads, theta);
    } catch (const std::bad_alloc&) {
        return COMPAMS_ERR_ALLOC;
    }
}

int compams_step(compams_handle c, const float* grads, float* theta) { return step_any(c, grads, theta, false); }
int compams_step_bf16(compams_handle c, const void* grads_bf16, float* theta) { return step_any(c, grads_bf16, theta, true); }

int compams_step_host(compams_handle c, const float* grads_host, float* theta_host) {
    if (!c || !grads_host || !theta_host || c->n != c->n_total || c->compressed) return COMPAMS_ERR_INVALID_ARG;
    RC(on_handle_device(c));
    const size_t gbytes = (size_t)c->n * (size_t)c->d * sizeof(float);
    const size_t tbytes = (size_t)c->d * sizeof(float);
    if (!c->stage_grads) {
        cudaError_t e = cudaMalloc((void**)&c->stage_grads, gbytes);
        if (e != cudaSuccess) {
            c->stage_grads = nullptr;
            cudaGetLastError();
            return COMPAMS_ERR_ALLOC;
        }
        e = cudaMalloc((void**)&c->stage_theta, tbytes);
        if (e != cudaSuccess) {
            c->stage_theta = nullptr;
            cudaGetLastError();
            return COMPAMS_ERR_ALLOC;
        }
    }
    CU(cudaMemcpyAsync(c->stage_grads, grads_host, gbytes, cudaMemcpyHostToDevice, c->stream));
    CU(cudaMemcpyAsync(c->stage_theta, theta_host, tbytes, cudaMemcpyHostToDevice, c->stream));
    int rc;
    c->grad_bf16 = false;
    try {
        rc = step_device(c, c->stage_grads, c->stage_theta);
    } catch (const std::bad_alloc&) {
        rc = COMPAMS_ERR_ALLOC;
    }
    if (rc) return rc;
    CU(cudaMemcpyAsync(theta_host, c->stage_theta, tbytes, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    return COMPAMS_OK;
}

int compams_destroy(compams_handle c) {
    if (!c) return COMPAMS_OK;
    cudaStreamSynchronize(c->stream);
    free_context(c);
    return COMPAMS_OK;
}

int compams_set_stream(compams_handle c, void* cuda_stream) {
    if (!c) return COMPAMS_ERR_INVALID_ARG;
    c->stream = (cudaStream_t)cuda_stream;
    return COMPAMS_OK;
}

int compams_set_seed(compams_handle c, uint64_t seed, uint64_t iterations_done) {
    if (!c || c->compressed) return COMPAMS_ERR_INVALID_ARG;
    c->seed = seed;
    c->iter = iterations_done;
    return COMPAMS_OK;
}

int compams_record_average(compams_handle c, int on) {
    if (!c) return COMPAMS_ERR_INVALID_ARG;
    c->record_gbar = on != 0;
    c->tk.gbar = c->record_gbar ? c->gbar : nullptr;
    c->bs.gbar = c->record_gbar ? c->gbar : nullptr;
    return COMPAMS_OK;
}

int compams_set_lr(compams_handle c, float lr) {
    if (!c || !(lr == lr)) return COMPAMS_ERR_INVALID_ARG;
    c->hp.lr = lr;
    return COMPAMS_OK;
}

// Finishes the residual update where it has been deferred, so that E holds e.
static int finish_residual(compams_context* c) {
    if (c->sparse() && !c->identity && c->e_mask_pending) {
        RC(run_kernel(c, COMPAMS_K_TOPK_MATERIALIZE, [&] { return launch_topk_materialize(c); }));
        c->e_mask_pending = false;
    }
    if (c->compressor == COMPAMS_BLOCKSIGN && c->e_is_x) {
        RC(run_kernel(c, COMPAMS_K_BS_MATERIALIZE, [&] { return launch_bs_materialize(c); }));
        c->e_is_x = false;
    }
    return COMPAMS_OK;
}

int compams_get_state(compams_handle c, float* e, float* m, float* v, float* vhat) {
    if (!c || c->compressed) return COMPAMS_ERR_INVALID_ARG;  // between compress and apply the step is half done
    RC(on_handle_device(c));
    const size_t nd = (size_t)c->n * (size_t)c->d * sizeof(float), db = (size_t)c->d * sizeof(float);
    if (e) {
        if (c->E) {
            RC(finish_residual(c));
            CU(cudaMemcpyAsync(e, c->E, nd, cudaMemcpyDeviceToDevice, c->stream));
        } else {
            CU(cudaMemsetAsync(e, 0, nd, c->stream));
        }
    }
    if (m) CU(cudaMemcpyAsync(m, c->m, db, cudaMemcpyDeviceToDevice, c->stream));
    if (v) CU(cudaMemcpyAsync(v, c->v, db, cudaMemcpyDeviceToDevice, c->stream));
    if (vhat) CU(cudaMemcpyAsync(vhat, c->vhat, db, cudaMemcpyDeviceToDevice, c->stream));
    return COMPAMS_OK;
}

int compams_set_state(compams_handle c, const float* e, const float* m, const float* v, const float* vhat) {
    if (!c || c->compressed) return COMPAMS_ERR_INVALID_ARG;
    RC(on_handle_device(c));
    const size_t nd = (size_t)c->n * (size_t)c->d * sizeof(float), db = (size_t)c->d * sizeof(float);
    if (e && c->E) {
        CU(cudaMemcpyAsync(c->E, e, nd, cudaMemcpyDeviceToDevice, c->stream));
        // E now holds e itself; predictions made from the replaced accumulators are dropped
        c->e_is_x = false;
        c->e_mask_pending = false;
        if (c->tk.seg && !c->seg_init_host.empty()) {
            CU(cudaMemcpyAsync(c->tk.seg, c->seg_init_host.data(), c->seg_init_host.size() * sizeof(SegState),
                               cudaMemcpyHostToDevice, c->stream));
            CU(cudaMemcpyAsync(c->tk.dense_count, &c->dense_count_init, sizeof(uint32_t), cudaMemcpyHostToDevice,
                               c->stream));
        }
    }
    if (m) CU(cudaMemcpyAsync(c->m, m, db, cudaMemcpyDeviceToDevice, c->stream));
    if (v) CU(cudaMemcpyAsync(c->v, v, db, cudaMemcpyDeviceToDevice, c->stream));
    if (vhat) CU(cudaMemcpyAsync(c->vhat, vhat, db, cudaMemcpyDeviceToDevice, c->stream));
    return COMPAMS_OK;
}

int compams_bits_transmitted(compams_handle c, uint64_t* out) {
    if (!c || !out) return COMPAMS_ERR_INVALID_ARG;
    const uint64_t full = 32ull * (uint64_t)c->n * (uint64_t)c->d;
    uint64_t payload = full, index = 0;
    if (c->compressor == COMPAMS_BLOCKSIGN) {
        payload = (uint64_t)c->n * ((uint64_t)c->d + 32ull * (uint64_t)c->M);
    } else if (!c->identity) {
        payload = 32ull * (uint64_t)c->n * (uint64_t)c->K;
        index = payload;
    }
    out[0] = full * c->steps_done;
    out[1] = payload * c->steps_done;
    out[2] = index * c->steps_done;
    return COMPAMS_OK;
}

int compams_get_buffer(compams_handle c, int32_t which, void** dev_ptr, int64_t* count) {
    if (!c || !dev_ptr || !count) return COMPAMS_ERR_INVALID_ARG;
    void* p = nullptr;
    int64_t cnt = 0;
    const bool topk = c->sparse() && !c->identity;
    const bool sign = c->compressor == COMPAMS_BLOCKSIGN;
    switch (which) {
        case COMPAMS_BUF_E:
            if (c->compressed) return COMPAMS_ERR_INVALID_ARG;  // the residual is closed by compams_apply
            if (!c->E) break;  // every k_b = d_b: e is identically zero and not stored
            RC(on_handle_device(c));
            RC(finish_residual(c));
            p = c->E;
            cnt = (int64_t)c->n * c->d;
            break;
        case COMPAMS_BUF_M: p = c->m; cnt = c->d; break;
        case COMPAMS_BUF_V: p = c->v; cnt = c->d; break;
        case COMPAMS_BUF_VHAT: p = c->vhat; cnt = c->d; break;
        case COMPAMS_BUF_GBAR:
            if (!c->record_gbar) return COMPAMS_ERR_INVALID_ARG;  // not being written
            p = c->gbar; cnt = c->d; break;
        case COMPAMS_BUF_TOPK_IDX: if (topk) { p = c->tk.idx; cnt = (int64_t)c->n_total * c->K; } break;
        case COMPAMS_BUF_TOPK_VAL: if (topk) { p = c->tk.val; cnt = (int64_t)c->n_total * c->K; } break;
        case COMPAMS_BUF_TOPK_SEG_OFFSETS: if (topk) { p = c->d_seg_off; cnt = c->M + 1; } break;
        case COMPAMS_BUF_SIGN_BITS: if (sign) { p = c->bs.bits; cnt = (int64_t)c->n_total * c->W; } break;
        case COMPAMS_BUF_SIGN_WORD_OFFSETS: if (sign) { p = c->d_word_off; cnt = c->M + 1; } break;
        case COMPAMS_BUF_SCALES: if (sign) { p = c->scales[c->scales_cur]; cnt = (int64_t)c->n_total * c->M; } break;
        case COMPAMS_BUF_STATUS: p = c->status; cnt = 8; break;
        default: return COMPAMS_ERR_INVALID_ARG;
    }
    *dev_ptr = p;
    *count = cnt;
    return COMPAMS_OK;
}

int compams_check_status(compams_handle c, uint32_t* status_word) {
    if (!c) return COMPAMS_ERR_INVALID_ARG;
    CU(cudaStreamSynchronize(c->stream));
    uint32_t w = 0;
    CU(cudaMemcpy(&w, c->status, sizeof w, cudaMemcpyDeviceToHost));
    if (status_word) *status_word = w;
    return w ? COMPAMS_ERR_DEVICE_STATUS : COMPAMS_OK;
}

int compams_set_profiling(compams_handle c, uint32_t kernel_mask) {
    if (!c) return COMPAMS_ERR_INVALID_ARG;
    CU(cudaStreamSynchronize(c->stream));
    c->prof_mask = kernel_mask;
    c->prof_used = 0;
    return COMPAMS_OK;
}

int compams_get_kernel_time(compams_handle c, int32_t kernel, double* total_ms, int64_t* launches) {
    if (!c || !total_ms || !launches || kernel < 0 || kernel >= COMPAMS_K_COUNT) return COMPAMS_ERR_INVALID_ARG;
    CU(cudaStreamSynchronize(c->stream));
    double ms = 0.0;
    int64_t cnt = 0;
    for (int s = 0; s < c->prof_used; ++s) {
        if (c->ev_kernel[(size_t)s] != kernel) continue;
        float t = 0.0f;
        CU(cudaEventElapsedTime(&t, c->ev_start[(size_t)s], c->ev_stop[(size_t)s]));
        ms += (double)t;
        ++cnt;
    }
    *total_ms = ms;
    *launches = cnt;
    return COMPAMS_OK;
}

int64_t compams_launch_count(compams_handle c) { return c ? c->launches : 0; }

const char* compams_error_string(int status) {
    switch (status) {
        case COMPAMS_OK: return "ok";
        case COMPAMS_ERR_INVALID_ARG: return "invalid argument";
        case COMPAMS_ERR_ALLOC: return "allocation failed";
        case COMPAMS_ERR_CUDA: return "CUDA runtime error";
        case COMPAMS_ERR_DEVICE_STATUS: return "device status word is set";
        case COMPAMS_ERR_TOO_LARGE: return "problem size exceeds the fixed scratch capacity";
        default: return "unknown status";
    }
}

const char* compams_kernel_name(int32_t kernel) {
    static const char* names[COMPAMS_K_COUNT] = {
        "dense_mean_amsgrad", "bs_sweep", "bs_apply", "bs_materialize", "topk_sweep", "topk_dense",
        "topk_materialize", "randk_emit", "reserved", "topk_scatter", "amsgrad", "topk_small", "topk_select", "bs_scales"};
    return (kernel >= 0 && kernel < COMPAMS_K_COUNT) ? names[kernel] : "unknown";
}

const char* compams_last_cuda_error(void) { return g_last_cuda_error.c_str(); }

}  // extern "C"

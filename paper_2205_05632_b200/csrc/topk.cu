// Top-k path (Definition 1) of the COMP-AMS step: exact selection of the k_b largest magnitudes
// of every (worker, block), ties at the threshold going to the lower index.
//
// Keys are the fp32 bit patterns of x = g + e with the sign cleared (31 bits); selection is a
// most-significant-digit radix select over them.
//
//   Blocks of at most kSmallMax coordinates: topk_small - one CTA holds the block in shared
//   memory and does every radix pass there; E is written once.
//
//   Larger blocks, cut into tiles of kTile coordinates.
//   Candidate path (one pass over [n, d]):
//     topk_sweep    x = g + e written over E (Algorithm 2, the corrected-gradient step); every key >= tau_hat, a threshold
//                   predicted from the previous step, is appended to the segment's candidate list
//     topk_select   if the list holds at least k_b and at most its capacity, the exact Top-k is inside it.
//                   A histogram of the key offsets above tau_hat (bins sized from the last step) finds
//                   the threshold bin; winners above it are emitted, the bin's few candidates are
//                   ordered by (key, lower index first), the best kept, and the next tau_hat predicted.
//                   Otherwise the segment is marked for the dense passes. Short lists: one 1024-thread
//                   CTA per list (topk_select). A few long lists (whole-vector selection): every list
//                   is cut into slices handled by two kernels of ordinary CTAs (topk_selhist, topk_selemit)
//                   that meet through a global histogram and last-slice-finishes tickets.
//   Dense passes (only for marked segments; exact for any input, e.g. all-equal values), one
//   cooperative kernel topk_dense whose stages are separated by grid-wide barriers:
//     hist<1..3> / find<1..3>  three histogram passes over x, 11 + 10 + 10 key bits
//     collect       keys above the threshold are emitted; threshold ties too unless only some fit,
//                   in which case they are counted per tile
//     ties          takes the lowest-index threshold ties, tile by tile in index order
//   topk_scatter    closes the step per segment (count check, counters reset) and walks the
//                   (index, value) messages: each pair is appended to the bucket of its coordinate range
//                   for the server kernel (the server's average)
//   The residual update at a kept coordinate (e = x - x = 0) is deferred: E keeps x there, and every selection
//   leaves one magnitude per segment such that the kept elements are exactly those with |x| at or above it;
//   whoever reads E next - the next sweep, or topk_materialize - treats them as 0. Where a selection cuts through
//   a group of equal magnitudes (some kept, some not), it zeroes the few kept ones in E itself and leaves the
//   next larger magnitude.
#include <cooperative_groups.h>

#include "context.h"
#include "scatter.cuh"

namespace cg = cooperative_groups;

namespace compams {

// ------------------------------------------------------------------------------------------
// tile addressing shared by the large-block kernels

// First of the 4 consecutive coordinates (relative to the block) that lane `lane` of warp `warp`
// handles at iteration `it` of a tile starting at r0.
__device__ __forceinline__ int lane_r(int r0, int warp, int it, int lane) {
    return r0 + warp * kWarpSpan + it * 128 + lane * 4;
}

// Loads the 32 values of this thread's share of a tile of x (already stored in E).
// Coordinates past the block end read as +0 (callers mask them).
__device__ __forceinline__ void load_x_tile(const float* __restrict__ e, int len, int r0, int warp, int lane,
                                            float4 (&xv)[kIters]) {
    const int ce = align_class(e);
    if (r0 + kTile <= len) {
#pragma unroll
        for (int it = 0; it < kIters; ++it) xv[it] = load4(e + lane_r(r0, warp, it, lane), ce);
    } else {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int r = lane_r(r0, warp, it, lane);
            if (r + 3 < len) {
                xv[it] = load4(e + r, ce);
            } else {
                float tmp[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) tmp[k] = (r + k < len) ? e[r + k] : 0.0f;
                xv[it] = make_float4(tmp[0], tmp[1], tmp[2], tmp[3]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// sweep: x = g + e -> E; keys >= tau_hat go to the candidate list

// "Nothing kept": as a float this pattern is a NaN, which no magnitude reaches.
constexpr uint32_t kNothingKept = 0xffffffffu;

// One tile of the sweep. The tile starts at r0 (relative to the block), which is the block's tile
// boundary shifted down to a 128-byte line of G and E: r0 may be negative and the tile may reach
// past the block; such coordinates are skipped.
// `kept_from`: elements of E whose magnitude is at or above it were kept by the last step's selection and still
// hold x; their e is 0 (one float comparison: the key order is the order of |x|).
template <bool FULL, typename GT>
__device__ __forceinline__ void topk_sweep_tile(const GT* __restrict__ g, float* __restrict__ e, int len, int r0,
                                                int warp, int lane, uint32_t tau_hat, uint32_t coord0,
                                                uint2* sh_cand, uint32_t* sh_cnt, uint32_t* g_cnt, uint2* g_out,
                                                uint32_t cap, float kept_from) {
    const int cg_ = align_class(g + r0), ce = align_class(e + r0);
    constexpr int NB = 2;  // iterations whose loads are in flight together
#pragma unroll
    for (int bt = 0; bt < kIters / NB; ++bt) {
        float4 gv[NB], ev[NB];
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int r = lane_r(r0, warp, bt * NB + u, lane);
            if (FULL || (r >= 0 && r + 3 < len)) {
                gv[u] = load4_stream(g + r, cg_);
                ev[u] = load4(e + r, ce);
            } else {
                float gt[4], et[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const bool live = (unsigned)(r + k) < (unsigned)len;
                    gt[k] = live ? load1_stream(g + r + k) : 0.0f;
                    et[k] = live ? e[r + k] : 0.0f;
                }
                gv[u] = make_float4(gt[0], gt[1], gt[2], gt[3]);
                ev[u] = make_float4(et[0], et[1], et[2], et[3]);
            }
        }
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int r = lane_r(r0, warp, bt * NB + u, lane);
            float xs[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // coordinates kept in the last step still hold x in E: their e is 0 (Algorithm 2, the residual update)
                const float eo = lane_elem(ev[u], k);
                const float ek = fabsf(eo) >= kept_from ? 0.0f : eo;
                xs[k] = __fadd_rn(lane_elem(gv[u], k), ek);  // the corrected-gradient step: x = g + e
                if ((FULL || (unsigned)(r + k) < (unsigned)len) && mag_key(xs[k]) >= tau_hat) {
                    const uint2 cv = make_uint2(coord0 + (uint32_t)(r + k), __float_as_uint(xs[k]));
                    const uint32_t slot = atomicAdd(sh_cnt, 1u);
                    if (slot < (uint32_t)kTileCand) {
                        sh_cand[slot] = cv;
                    } else {  // a tile dense with candidates: the staging buffer is full, append directly
                        const uint32_t p = atomicAdd(g_cnt, 1u);
                        if (p < cap) g_out[p] = cv;
                    }
                }
            }
            if (FULL || (r >= 0 && r + 3 < len)) {
                store4(e + r, ce, make_float4(xs[0], xs[1], xs[2], xs[3]));
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if ((unsigned)(r + k) < (unsigned)len) e[r + k] = xs[k];
            }
        }
    }
}

// The same for bfloat16 gradients on a whole tile whose rows of G and E are 16-byte aligned: 8 coordinates per
// lane and iteration, so that the gradient load is 128 bits wide like the loads and stores of E (with 4
// coordinates per lane the 64-bit gradient loads leave too few bytes in flight). A warp's 1024 coordinates are
// 4 chunks of 256; the next chunk's loads are in flight while one is worked on.
__device__ __forceinline__ void topk_sweep_tile_bf16x8(const bf16_bits* __restrict__ g, float* __restrict__ e, int r0,
                                                       int warp, int lane, uint32_t tau_hat, uint32_t coord0,
                                                       uint2* sh_cand, uint32_t* sh_cnt, uint32_t* g_cnt, uint2* g_out,
                                                       uint32_t cap, float kept_from) {
    constexpr int NC = kWarpSpan / 256;
    const int rw = r0 + warp * kWarpSpan;
    uint4 gbuf[2];
    float4 ebuf[2][2];
    auto load_chunk = [&](int c, uint4& gv, float4 (&ev)[2]) {
        const int r = rw + c * 256 + lane * 8;
        gv = __ldg(reinterpret_cast<const uint4*>(g + r));
        ev[0] = *reinterpret_cast<const float4*>(e + r);
        ev[1] = *reinterpret_cast<const float4*>(e + r + 4);
    };
    load_chunk(0, gbuf[0], ebuf[0]);
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const uint4 gv = gbuf[c & 1];
        float4 (&ev)[2] = ebuf[c & 1];
        if (c + 1 < NC) load_chunk(c + 1, gbuf[(c + 1) & 1], ebuf[(c + 1) & 1]);
        const int r = rw + c * 256 + lane * 8;
        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float xs[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t word = gw[h * 2 + (k >> 1)];
                const float gk = __uint_as_float((k & 1) ? (word & 0xffff0000u) : (word << 16));  // exact widening
                // coordinates kept in the last step still hold x in E: their e is 0 (Algorithm 2, the residual update)
                const float eo = lane_elem(ev[h], k);
                const float ek = fabsf(eo) >= kept_from ? 0.0f : eo;
                xs[k] = __fadd_rn(gk, ek);  // the corrected-gradient step: x = g + e
                if (mag_key(xs[k]) >= tau_hat) {
                    const uint2 cv = make_uint2(coord0 + (uint32_t)(r + h * 4 + k), __float_as_uint(xs[k]));
                    const uint32_t slot = atomicAdd(sh_cnt, 1u);
                    if (slot < (uint32_t)kTileCand) {
                        sh_cand[slot] = cv;
                    } else {  // a tile dense with candidates: the staging buffer is full, append directly
                        const uint32_t p = atomicAdd(g_cnt, 1u);
                        if (p < cap) g_out[p] = cv;
                    }
                }
            }
            *reinterpret_cast<float4*>(e + r + h * 4) = make_float4(xs[0], xs[1], xs[2], xs[3]);
        }
    }
}

// Tiles are shifted down by (i d + o) mod 32, the position of the block's first element within a
// 128-byte line of G and E, so that every warp access covers whole lines (with rows that start
// mid-line a warp's 512 bytes straddle five lines instead of four: measured 7 % slower).
#ifndef COMPAMS_BF16_TOPK_SWEEP_CTAS
#define COMPAMS_BF16_TOPK_SWEEP_CTAS 5
#endif
template <typename GT>
__global__ void __launch_bounds__(kThreads, sizeof(GT) == 2 ? COMPAMS_BF16_TOPK_SWEEP_CTAS : 6) topk_sweep_kernel(Tables t, TopkBuffers b, const GT* __restrict__ G,
                                                                 const __grid_constant__ SegParams sp_) {
    dependency_wait();   // launched as a programmatic dependent while n d <= kChainMaxElems: the kernel before must be done
    allow_dependents();  // ... and the next one may move in behind this one's last wave
    __shared__ uint2 sh_cand[kTileCand];
    __shared__ uint32_t sh_cnt, sh_base;
    const TileInfo ti = sp_.nseg ? find_tile(sp_, blockIdx.x) : load_tile(t.tiles, blockIdx.x);
    const int i = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t sg = (size_t)i * t.nseg + ti.seg;
    SegState* st = b.seg + sg;
    const uint32_t tau_hat = st->tau_hat;
    const SegInfo* si = t.segs + ti.seg;
    const uint32_t cap = si->cap;
    uint2* out = b.cand + (size_t)i * (size_t)b.cand_total + (size_t)si->cand_off;
    if (threadIdx.x == 0) sh_cnt = 0u;
    __syncthreads();
    const int64_t row0 = (int64_t)i * t.d + ti.o;
    const GT* g = G + row0;
    float* e = b.E + row0;
    const int r0s = ti.r0 - (int)(row0 & 31);
    const float kept_from = __uint_as_float(b.use_thr ? b.thr[sg] : kNothingKept);
    const bool whole = r0s >= 0 && r0s + kTile <= ti.len;
    bool wide = false;
    if constexpr (sizeof(GT) == 2)
        wide = whole && ((reinterpret_cast<uintptr_t>(g + r0s) | reinterpret_cast<uintptr_t>(e + r0s)) & 15u) == 0;
    if (wide) {
        if constexpr (sizeof(GT) == 2)
            topk_sweep_tile_bf16x8(g, e, r0s, warp, lane, tau_hat, (uint32_t)ti.o, sh_cand, &sh_cnt, &st->cand_count, out,
                                   cap, kept_from);
    } else if (whole)
        topk_sweep_tile<true>(g, e, ti.len, r0s, warp, lane, tau_hat, (uint32_t)ti.o, sh_cand, &sh_cnt,
                              &st->cand_count, out, cap, kept_from);
    else
        topk_sweep_tile<false>(g, e, ti.len, r0s, warp, lane, tau_hat, (uint32_t)ti.o, sh_cand, &sh_cnt,
                               &st->cand_count, out, cap, kept_from);
    __syncthreads();
    const uint32_t cnt = sh_cnt;
    if (cnt == 0u) return;
    const uint32_t stored = cnt < (uint32_t)kTileCand ? cnt : (uint32_t)kTileCand;
    if (threadIdx.x == 0) sh_base = atomicAdd(&st->cand_count, stored);
    __syncthreads();
    const uint32_t base = sh_base;
    for (uint32_t k = threadIdx.x; k < stored; k += kThreads)
        if (base + k < cap) out[base + k] = sh_cand[k];
}

// ------------------------------------------------------------------------------------------
// select: exact Top-k inside the candidate list

// Prediction for the next step's sweep, from this step's threshold key `tau` and the bin edge
// `edge` at or above which about the wanted number of candidates (want_candidates) lay: the threshold keeps rising while the error
// accumulators fill, so tau_hat follows half of the last rise. `sel_shift` sizes the bins of the
// next select so that the expected threshold lands near the middle of its 4096 bins.
__device__ __forceinline__ void predict_next(SegState* st, uint32_t tau, uint32_t edge, bool enabled) {
    const uint32_t prev = st->tau_prev;
    uint32_t rise = 0;
    if (prev != kNoPrediction && tau > prev) rise = (tau - prev) >> 1;
    if (edge > tau) edge = tau;
    uint32_t next = edge + rise;
    if (next >= 0x7f800000u) next = edge;
    const uint32_t tau_pred = tau + rise;
    uint32_t span = tau_pred > next ? tau_pred - next : 1u;
    // ... but never so fine that the bins end close above the prediction: they cover at least a quarter of a
    // binade (values up to about 19 % above tau_hat), so a threshold that lands higher than predicted - gradients
    // that alternate between two levels do that - is still found inside the list
    if (span < (1u << 19)) span = 1u << 19;
    st->sel_shift = 32u - (uint32_t)__clz(span >> 11);  // smallest S with span >> S < 2048
    st->tau_hat = enabled ? next : kNoPrediction;
    st->tau_prev = tau;
}

// How many candidates the next step's predicted threshold should let through for a segment that keeps kb: the
// count of keys above a fixed threshold moves by about sqrt(kb) from one step to the next (eight of those are
// allowed for), plus a quarter of kb for drift of the gradient scale. A segment whose list came up short gets
// its margin doubled (`boost` times, at most three); the doubling is taken back one step at a time after enough
// selections in a row were decided inside the list (margin_held). Long lists thus carry about 1.26 kb entries, short ones
// (kb = 50: 170) proportionally more.
__device__ __forceinline__ uint32_t want_candidates(uint32_t kb, uint32_t boost) {
    const uint32_t margin = ((kb >> 2) + (uint32_t)(8.0f * sqrtf((float)kb)) + 32u) << (boost < 3u ? boost : 3u);
    const uint32_t most = 4u * kb + 512u;  // half the list's capacity
    return kb + (margin < most - kb ? margin : most - kb);
}
// Taking a doubling back is a probe: if the smaller margin comes up short (a dense-pass step, which costs several
// ordinary steps), the margin was needed, and the next probe waits twice as long (32, 64, ... 32768 selections). A
// probe that holds for a whole waiting time halves the wait again. Gradients that alternate between two levels
// need the first doubling for good: with a fixed wait of 32 every 33rd step ran the dense passes (n = 32,
// d = 2^27: 9.1 -> 9.6 ms per step on average).
constexpr uint32_t kHoldMax = 10u;
__device__ __forceinline__ void margin_came_up_short(SegState* st) {
    if (st->boost < 3u) ++st->boost;
    if (st->probing && st->hold < kHoldMax) ++st->hold;
    st->probing = 0u;
    st->streak = 0u;
}
__device__ __forceinline__ void margin_held(SegState* st) {
    if (++st->streak >= (32u << st->hold)) {
        st->streak = 0u;
        if (st->probing && st->hold) --st->hold;
        st->probing = 0u;
        if (st->boost) {
            --st->boost;
            st->probing = 1u;
        }
    }
}

// After a selection decided inside its list of c candidates: a list that held by less than a quarter of its margin
// was a near miss and is treated like a list that came up short, only without the dense passes (thresholds that
// swing from step to step announce themselves this way: d = 2^24, n = 8, two alternating batches: 1.01 k_b
// candidates a dozen steps before 0.94 k_b).
__device__ __forceinline__ void margin_after_selection(SegState* st, uint32_t kb, uint32_t c) {
    if (c - kb < (want_candidates(kb, st->boost) - kb) >> 2) margin_came_up_short(st);
    else margin_held(st);
}

constexpr int kSelUnroll = 4;   // candidate loads in flight per thread while scanning a list
// One CTA per short list, 2048 threads to the SM at 32 registers. 1024 threads per list keep enough loads in flight
// to finish one list soonest (few lists: d = 2^20, n = 8: step 0.051 ms against 0.058 with 512); with more lists
// than the GPU holds CTAs, 512 threads per list and twice as many lists in flight get through them sooner
// (ResNet-50 shapes layer-wise, n = 32, 1696 lists: select 0.121 -> 0.111 ms; with 256: 0.178).
constexpr int kSelThreads = 1024;
constexpr int kSelThreadsMany = 512;

// Adds the `pred` lanes of a warp to a shared counter with one atomic; returns this lane's slot.
__device__ __forceinline__ uint32_t warp_slot(bool pred, uint32_t* counter, int lane) {
    const unsigned m = __ballot_sync(0xffffffffu, pred);
    uint32_t base = 0;
    if (m) {
        const int leader = __ffs(m) - 1;
        if (lane == leader) base = atomicAdd(counter, (uint32_t)__popc(m));
        base = __shfl_sync(0xffffffffu, base, leader);
    }
    return base + (uint32_t)__popc(m & ((1u << lane) - 1u));
}

// A histogram of nb bins scanned from its top bin down: every thread owns nb / kThreads
// consecutive bins (from the top) and learns how many entries lie above and inside its bins.
struct BinScan {
    uint32_t incl, excl;
};
template <int NT>
__device__ __forceinline__ BinScan scan_from_top(const uint32_t* hm, int nb, uint32_t* scratch, uint32_t* total) {
    const int per = nb / NT > 0 ? nb / NT : 1;
    uint32_t sum = 0;
    for (int j = 0; j < per; ++j) {
        const int bin = nb - 1 - ((int)threadIdx.x * per + j);
        if (bin >= 0) sum += hm[bin];
    }
    BinScan r;
    r.incl = block_inclusive_scan<NT / 32>(sum, scratch, total);
    r.excl = r.incl - sum;
    return r;
}
// The thread whose bins hold the `target`-th entry from the top writes
// sh_out[0] = bin, sh_out[1] = entries above the bin, sh_out[2] = entries in the bin.
template <int NT>
__device__ __forceinline__ void locate(const uint32_t* hm, int nb, const BinScan& sc, uint32_t target, uint32_t* sh_out) {
    if (sc.excl < target && target <= sc.incl) {
        const int per = nb / NT > 0 ? nb / NT : 1;
        uint32_t running = sc.excl;
        for (int j = 0; j < per; ++j) {
            const int bin = nb - 1 - ((int)threadIdx.x * per + j);
            const uint32_t cj = bin >= 0 ? hm[bin] : 0u;
            if (running < target && target <= running + cj) {
                sh_out[0] = (uint32_t)bin;
                sh_out[1] = running;
                sh_out[2] = cj;
            }
            running += cj;
        }
    }
}

__device__ __forceinline__ uint32_t offset_digit(uint32_t xbits, uint32_t tau_hat, int S) {
    const uint32_t dg = ((xbits & 0x7fffffffu) - tau_hat) >> S;  // every candidate has key >= tau_hat
    return dg < (uint32_t)(kSelBins - 1) ? dg : (uint32_t)(kSelBins - 1);
}

template <int NT>
__global__ void __launch_bounds__(NT, 2048 / NT) topk_select_kernel(Tables t, TopkBuffers b, const int32_t* __restrict__ seg_list,
                                                               int nlist) {
    dependency_wait();   // launched as a programmatic dependent while n d <= kChainMaxElems: the kernel before must be done
    allow_dependents();  // ... and the next one may move in behind this one's last wave
    __shared__ uint32_t local[kSelBins];  // histogram of the list
    __shared__ uint2 surv[kSurvCap];
    __shared__ uint32_t scratch[NT / 32];
    __shared__ uint32_t sh_bin[3], sh_edge[3], sh_base, sh_wcnt, sh_scnt;
    const int lane = threadIdx.x & 31;
    // the lists come longest first, every worker's copy of one block side by side: the CTAs that take longest
    // start first and the last wave holds the shortest lists
    const int i = (int)(blockIdx.x % (unsigned)t.n);
    const int seg = seg_list[blockIdx.x / (unsigned)t.n];
    const size_t sg = (size_t)i * t.nseg + seg;
    const SegInfo* si = t.segs + seg;
    SegState* st = b.seg + sg;
    const uint32_t kb = si->kb, cap = si->cap;
    const uint32_t c = st->cand_count;
    const uint32_t tau_hat = st->tau_hat;
    const int S = (int)st->sel_shift;
    if (!(tau_hat != kNoPrediction && c >= kb && c <= cap)) {
        if (threadIdx.x == 0) {
            st->fallback = 1u;
            atomicAdd(b.dense_count, 1u);
            if (tau_hat != kNoPrediction) atomicAdd(b.status + (c < kb ? 3 : 4), 1u);  // too few / too many candidates
            if (tau_hat != kNoPrediction && c < kb) margin_came_up_short(st);
        }
        return;
    }
    const uint2* list = b.cand + (size_t)i * (size_t)b.cand_total + (size_t)si->cand_off;
    const uint32_t lo = 0u, hi = c;
    auto digit0 = [&](uint32_t xbits) -> uint32_t { return offset_digit(xbits, tau_hat, S); };

    // ---- pass 0: histogram of the key offsets above tau_hat in bins of 2^S; the last bin is open-ended
    for (int k = threadIdx.x; k < kSelBins; k += NT) local[k] = 0u;
    if (threadIdx.x == 0) sh_scnt = 0u;
    __syncthreads();
    for (uint32_t p0 = lo; p0 < hi; p0 += kSelUnroll * NT) {
        uint32_t y[kSelUnroll];
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const uint32_t p = p0 + u * NT + threadIdx.x;
            y[u] = p < hi ? list[p].y : 0xffffffffu;  // no candidate has this pattern (NaN)
        }
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const bool valid = y[u] != 0xffffffffu;
            const uint32_t dg = valid ? digit0(y[u]) : 0u;
            // the open-ended last bin collects every far-above-threshold candidate: one atomic per warp
            const bool far = valid && dg == (uint32_t)(kSelBins - 1);
            const unsigned m = __ballot_sync(0xffffffffu, far);
            if (m && lane == __ffs(m) - 1) atomicAdd(&local[kSelBins - 1], (uint32_t)__popc(m));
            if (valid && !far) atomicAdd(&local[dg], 1u);
        }
    }
    __syncthreads();
    uint32_t total;
    {
        const BinScan sc = scan_from_top<NT>(local, kSelBins, scratch, &total);
        const uint32_t want = want_candidates(kb, st->boost);
        if (threadIdx.x == 0) sh_edge[0] = 0xffffffffu;  // "fewer than `want` candidates"
        __syncthreads();
        locate<NT>(local, kSelBins, sc, kb, sh_bin);
        locate<NT>(local, kSelBins, sc, want, sh_edge);
    }
    __syncthreads();
    const uint32_t b0 = sh_bin[0];
    uint32_t k_rem = kb - sh_bin[1];
    const uint32_t c0 = sh_bin[2];
    const uint32_t edge_bin = sh_edge[0];
    const bool take_all0 = (c0 == k_rem);
    // the number of winners, from the histogram
    uint32_t mine = 0;
    for (int k = threadIdx.x; k < kSelBins; k += NT)
        if ((uint32_t)k > b0 || (take_all0 && (uint32_t)k == b0)) mine += local[k];
    uint32_t my_winners;
    block_inclusive_scan<NT / 32>(mine, scratch, &my_winners);
    __syncthreads();
    if (b0 == (uint32_t)(kSelBins - 1) && !take_all0) {
        // the threshold lies in the open-ended bin: the prediction was far off, let the dense passes decide
        if (threadIdx.x == 0) {
            st->fallback = 1u;
            atomicAdd(b.dense_count, 1u);
            atomicAdd(b.status + 5, 1u);
        }
        return;
    }

    // ---- second scan of the list: winners to the message, threshold-bin candidates to shared memory
    const size_t slot0 = (size_t)i * (size_t)b.K + (size_t)si->slot0;
    uint2* surv0 = &surv[0];
    uint32_t* scnt0 = &sh_scnt;
    if (threadIdx.x == 0) {
        sh_base = my_winners ? atomicAdd(&st->emit_count, my_winners) : 0u;
        sh_wcnt = 0u;
    }
    __syncthreads();
    for (uint32_t p0 = lo; p0 < hi; p0 += kSelUnroll * NT) {
        uint2 cvs[kSelUnroll];
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const uint32_t p = p0 + u * NT + threadIdx.x;
            cvs[u] = p < hi ? list[p] : make_uint2(0u, 0xffffffffu);
        }
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const uint2 cv = cvs[u];
            const bool valid = cv.y != 0xffffffffu;
            const uint32_t dg = valid ? digit0(cv.y) : 0u;
            const bool win = valid && (dg > b0 || (take_all0 && dg == b0));
            const bool keep = valid && !take_all0 && dg == b0;
            const uint32_t wpos = sh_base + warp_slot(win, &sh_wcnt, lane);
            if (win) {
                if (wpos < kb) {
                    b.idx[slot0 + wpos] = (int32_t)cv.x;
                    b.val[slot0 + wpos] = __uint_as_float(cv.y);
                } else {
                    atomicOr(b.status, 1u);
                }
            }
            if (__any_sync(0xffffffffu, keep)) {  // rare: only the threshold bin's candidates
                const uint32_t spos = warp_slot(keep, scnt0, lane);
                if (keep && spos < (uint32_t)kSurvCap) surv0[spos] = cv;
            }
        }
    }
    // threshold key of this step (a lower bound if every candidate of the threshold bin is kept)
    const unsigned long long tau_wide = (unsigned long long)tau_hat + ((unsigned long long)b0 << S);
    uint32_t tau = tau_wide < 0x7f7fffffull ? (uint32_t)tau_wide : 0x7f7fffffu;
    // the magnitude from which on everything was kept. With the whole threshold bin kept that is the bin's lower
    // edge; otherwise the kept candidates of the bin are zeroed in E right here and the next key above the
    // threshold is left
    uint32_t kept_from = tau_wide < 0xffffffffull ? (uint32_t)tau_wide : kNothingKept;
    float* erow = b.E + (size_t)i * (size_t)t.d;
    if (!take_all0) {
        __syncthreads();
        const uint32_t nsurv = sh_scnt;
        if (nsurv > (uint32_t)kSurvCap) {
            // too many candidates share the threshold bin (heavily duplicated values): dense passes
            if (threadIdx.x == 0) {
                st->fallback = 1u;
                atomicAdd(b.dense_count, 1u);
                atomicAdd(b.status + 6, 1u);
            }
            return;
        }
        // ---- the survivors are ordered by (key, lower index first): survivor q is kept when fewer
        // than k_rem survivors beat it
        const uint32_t lowmask = S ? ((1u << S) - 1u) : 0u;
        auto comp_of = [&](const uint2& cv) -> unsigned long long {
            const uint32_t o = (cv.y & 0x7fffffffu) - tau_hat;
            return ((unsigned long long)(o & lowmask) << 32) | (unsigned long long)(0xffffffffu - cv.x);
        };
        for (uint32_t q0 = 0; q0 < nsurv; q0 += NT) {  // uniform trip count: the loop holds barriers
            const uint32_t q = q0 + threadIdx.x;
            bool kept = false;
            uint2 cv = make_uint2(0u, 0u);
            if (q < nsurv) {
                cv = surv[q];
                const unsigned long long mine_c = comp_of(cv);
                uint32_t beaten = 0;
                for (uint32_t p = 0; p < nsurv; ++p) beaten += (comp_of(surv[p]) > mine_c) ? 1u : 0u;
                kept = beaten < k_rem;
                if (beaten == k_rem - 1u) sh_edge[1] = (cv.y & 0x7fffffffu);  // the k-th largest key overall
            }
            uint32_t tot3;
            const uint32_t incl = block_inclusive_scan<NT / 32>(kept ? 1u : 0u, scratch, &tot3);
            if (threadIdx.x == 0) sh_base = tot3 ? atomicAdd(&st->emit_count, tot3) : 0u;
            __syncthreads();
            if (kept) {
                const uint32_t pos = sh_base + incl - 1u;
                if (pos < kb) {
                    b.idx[slot0 + pos] = (int32_t)cv.x;
                    b.val[slot0 + pos] = __uint_as_float(cv.y);
                } else {
                    atomicOr(b.status, 1u);
                }
                erow[cv.x] = 0.0f;  // the residual of a kept coordinate: e = x - x
            }
            __syncthreads();
        }
        tau = sh_edge[1];
        kept_from = tau + 1u;
    }
    if (threadIdx.x == 0) {
        b.thr[sg] = kept_from;
        uint32_t edge;
        if (edge_bin != 0xffffffffu) {
            const unsigned long long ew = (unsigned long long)tau_hat + ((unsigned long long)edge_bin << S);
            edge = ew < 0x7f7fffffull ? (uint32_t)ew : 0x7f7fffffu;
        } else {
            // fewer candidates than wanted: reach further down next time, by half the distance to the threshold
            const uint32_t gap = ((tau - tau_hat) >> 1) + (1u << 16);
            edge = tau_hat > gap ? tau_hat - gap : 0u;
        }
        predict_next(st, tau, edge, true);
        margin_after_selection(st, kb, c);
        st->fallback = 0u;
        atomicAdd(b.status + 2, 1u);  // selections decided inside their candidate list
    }
}

// ------------------------------------------------------------------------------------------
// select for a few long lists (whole-vector selection): every list is cut into `parts` slices and
// two kernels of ordinary CTAs work on all slices at once. The slices of a list meet through a
// histogram in global memory and "the last slice to arrive does the serial part" tickets; nobody
// waits for anybody.
//   topk_selhist  slice histograms of the key offsets above tau_hat, added into the list's global
//                 histogram; the last slice finds the threshold bin and the next tau_hat's bin edge
//   topk_selemit  winners above the threshold bin go to the message, the bin's candidates to the
//                 list's survivor buffer; the last slice ranks the survivors, emits the best and predicts

__global__ void __launch_bounds__(kThreads) topk_selhist_kernel(Tables t, TopkBuffers b, const int32_t* __restrict__ seg_list,
                                                                int nlist, int parts) {
    dependency_wait();   // launched as a programmatic dependent while n d <= kChainMaxElems: the kernel before must be done
    allow_dependents();  // ... and the next one may move in behind this one's last wave
    __shared__ uint32_t local[kSelBins];
    __shared__ uint32_t scratch[kWarps];
    __shared__ uint32_t sh_bin[3], sh_edge[3];
    __shared__ int is_last;
    const int lane = threadIdx.x & 31;
    const int part = blockIdx.x % parts;
    const size_t item = blockIdx.x / parts;  // (worker, list)
    const int i = (int)(item / (size_t)nlist);
    const int seg = seg_list[item % (size_t)nlist];
    const size_t sg = (size_t)i * t.nseg + seg;
    const SegInfo* si = t.segs + seg;
    SegState* st = b.seg + sg;
    const uint32_t kb = si->kb, cap = si->cap;
    const uint32_t c = st->cand_count;
    const uint32_t tau_hat = st->tau_hat;
    const int S = (int)st->sel_shift;
    // the same decision in every slice of the list: nobody writes these words in this kernel
    if (!(tau_hat != kNoPrediction && c >= kb && c <= cap)) {
        if (part == 0 && threadIdx.x == 0) {
            st->fallback = 1u;
            atomicAdd(b.dense_count, 1u);
            if (tau_hat != kNoPrediction) atomicAdd(b.status + (c < kb ? 3 : 4), 1u);  // too few / too many candidates
            if (tau_hat != kNoPrediction && c < kb) margin_came_up_short(st);
        }
        return;
    }
    const uint2* list = b.cand + (size_t)i * (size_t)b.cand_total + (size_t)si->cand_off;
    const uint32_t per = (c + parts - 1) / parts;
    const uint32_t lo = (uint32_t)part * per < c ? (uint32_t)part * per : c;
    const uint32_t hi = (lo + per < c) ? lo + per : c;
    for (int k = threadIdx.x; k < kSelBins; k += kThreads) local[k] = 0u;
    __syncthreads();
    for (uint32_t p0 = lo; p0 < hi; p0 += kSelUnroll * kThreads) {
        uint32_t y[kSelUnroll];
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const uint32_t p = p0 + u * kThreads + threadIdx.x;
            y[u] = p < hi ? list[p].y : 0xffffffffu;  // no candidate has this pattern (NaN)
        }
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const bool valid = y[u] != 0xffffffffu;
            const uint32_t dg = valid ? offset_digit(y[u], tau_hat, S) : 0u;
            // the open-ended last bin collects every far-above-threshold candidate: one atomic per warp
            const bool far = valid && dg == (uint32_t)(kSelBins - 1);
            const unsigned m = __ballot_sync(0xffffffffu, far);
            if (m && lane == __ffs(m) - 1) atomicAdd(&local[kSelBins - 1], (uint32_t)__popc(m));
            if (valid && !far) atomicAdd(&local[dg], 1u);
        }
    }
    __syncthreads();
    uint32_t* gh = b.sel_hist + item * kSelBins;
    for (int k = threadIdx.x; k < kSelBins; k += kThreads) {
        const uint32_t v = local[k];
        if (v) atomicAdd(gh + k, v);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(b.sel_ticket + 2 * item, 1u) == (uint32_t)(parts - 1));
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // ---- the last slice: the list's histogram is complete
    for (int k = threadIdx.x; k < kSelBins; k += kThreads) {
        local[k] = __ldcg(gh + k);
        gh[k] = 0u;  // clean for the next step
    }
    __syncthreads();
    uint32_t total;
    const BinScan sc = scan_from_top<kThreads>(local, kSelBins, scratch, &total);
    const uint32_t want = want_candidates(kb, st->boost);
    if (threadIdx.x == 0) sh_edge[0] = 0xffffffffu;  // "fewer than `want` candidates"
    __syncthreads();
    locate<kThreads>(local, kSelBins, sc, kb, sh_bin);
    locate<kThreads>(local, kSelBins, sc, want, sh_edge);
    __syncthreads();
    if (threadIdx.x == 0) {
        b.sel_ticket[2 * item] = 0u;
        const uint32_t b0 = sh_bin[0], k_rem = kb - sh_bin[1];
        const bool take_all0 = (sh_bin[2] == k_rem);
        if (b0 == (uint32_t)(kSelBins - 1) && !take_all0) {
            // the threshold lies in the open-ended bin: the prediction was far off, let the dense passes decide
            st->fallback = 1u;
            atomicAdd(b.dense_count, 1u);
            atomicAdd(b.status + 5, 1u);
        } else {
            st->prefix = b0;  // the dense passes' fields are free while the candidate path owns the segment
            st->k_rem = k_rem;
            st->ties_total = take_all0 ? 1u : 0u;
            st->edge = sh_edge[0];
            st->sel_ready = 1u;
        }
    }
}

__global__ void __launch_bounds__(kThreads) topk_selemit_kernel(Tables t, TopkBuffers b, const int32_t* __restrict__ seg_list,
                                                                int nlist, int parts) {
    dependency_wait();   // launched as a programmatic dependent while n d <= kChainMaxElems: the kernel before must be done
    allow_dependents();  // ... and the next one may move in behind this one's last wave
    __shared__ uint2 surv[kSurvSmem];
    __shared__ uint32_t sh_hist[kThreads];
    __shared__ uint32_t scratch[kWarps];
    __shared__ uint32_t sh_base, sh_wcnt, sh_tau;
    __shared__ int is_last;
    const int lane = threadIdx.x & 31;
    const int part = blockIdx.x % parts;
    const size_t item = blockIdx.x / parts;
    const int i = (int)(item / (size_t)nlist);
    const int seg = seg_list[item % (size_t)nlist];
    const size_t sg = (size_t)i * t.nseg + seg;
    const SegInfo* si = t.segs + seg;
    SegState* st = b.seg + sg;
    if (st->sel_ready == 0u) return;  // not decided by the candidate path (same word for every slice)
    const uint32_t kb = si->kb;
    const uint32_t c = st->cand_count;
    const uint32_t tau_hat = st->tau_hat;
    const int S = (int)st->sel_shift;
    const uint32_t b0 = st->prefix, k_rem = st->k_rem, edge_bin = st->edge;
    const bool take_all0 = st->ties_total != 0u;
    const uint2* list = b.cand + (size_t)i * (size_t)b.cand_total + (size_t)si->cand_off;
    const uint32_t per = (c + parts - 1) / parts;
    const uint32_t lo = (uint32_t)part * per < c ? (uint32_t)part * per : c;
    const uint32_t hi = (lo + per < c) ? lo + per : c;
    const size_t slot0 = (size_t)i * (size_t)b.K + (size_t)si->slot0;
    uint2* gsurv = b.sel_surv + item * kSurvCapBig;
    uint32_t* gscnt = b.sel_ticket + 2 * item + 1;  // survivors appended so far (second word of the pair)

    // one pass over the slice, a chunk of kSelUnroll candidates per thread at a time: the chunk's winners are
    // counted (a scan over the CTA), get one contiguous range of message slots with a single atomic, and are
    // written there
    for (uint32_t p0 = lo; p0 < hi; p0 += kSelUnroll * kThreads) {  // uniform trip count: the loop holds barriers
        uint2 cvs[kSelUnroll];
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const uint32_t p = p0 + u * kThreads + threadIdx.x;
            cvs[u] = p < hi ? list[p] : make_uint2(0u, 0xffffffffu);
        }
        uint32_t winmask = 0, keepmask = 0;
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            const bool valid = cvs[u].y != 0xffffffffu;
            const uint32_t dg = valid ? offset_digit(cvs[u].y, tau_hat, S) : 0u;
            if (valid && (dg > b0 || (take_all0 && dg == b0))) winmask |= 1u << u;
            if (valid && !take_all0 && dg == b0) keepmask |= 1u << u;
        }
        const uint32_t mine = (uint32_t)__popc(winmask);
        uint32_t chunk_winners;
        const uint32_t incl = block_inclusive_scan(mine, scratch, &chunk_winners);
        if (threadIdx.x == 0) sh_base = chunk_winners ? atomicAdd(&st->emit_count, chunk_winners) : 0u;
        __syncthreads();
        uint32_t wpos = sh_base + incl - mine;
#pragma unroll
        for (int u = 0; u < kSelUnroll; ++u) {
            if ((winmask >> u) & 1u) {
                if (wpos < kb) {
                    b.idx[slot0 + wpos] = (int32_t)cvs[u].x;
                    b.val[slot0 + wpos] = __uint_as_float(cvs[u].y);
                } else {
                    atomicOr(b.status, 1u);
                }
                ++wpos;
            }
            const bool keep = (keepmask >> u) & 1u;
            if (__any_sync(0xffffffffu, keep)) {  // rare: only the threshold bin's candidates
                const uint32_t spos = warp_slot(keep, gscnt, lane);
                if (keep && spos < (uint32_t)kSurvCapBig) gsurv[spos] = cvs[u];
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(b.sel_ticket + 2 * item, 1u) == (uint32_t)(parts - 1));
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // ---- the last slice finishes the list
    const uint32_t nsurv = take_all0 ? 0u : __ldcg(gscnt);
    __syncthreads();
    if (threadIdx.x == 0) {
        b.sel_ticket[2 * item] = 0u;
        b.sel_ticket[2 * item + 1] = 0u;
        st->sel_ready = 0u;
    }
    if (nsurv > (uint32_t)kSurvCapBig) {
        // too many candidates share the threshold bin (heavily duplicated values): dense passes
        if (threadIdx.x == 0) {
            st->fallback = 1u;
            atomicAdd(b.dense_count, 1u);
            atomicAdd(b.status + 6, 1u);
        }
        return;
    }
    const unsigned long long tau_wide = (unsigned long long)tau_hat + ((unsigned long long)b0 << S);
    uint32_t tau = tau_wide < 0x7f7fffffull ? (uint32_t)tau_wide : 0x7f7fffffu;
    // the magnitude from which on everything was kept. With the whole threshold bin kept that is the bin's lower
    // edge; otherwise the kept candidates of the bin are zeroed in E right here and the next key above the
    // threshold is left
    uint32_t kept_from = tau_wide < 0xffffffffull ? (uint32_t)tau_wide : kNothingKept;
    float* erow = b.E + (size_t)i * (size_t)t.d;
    if (!take_all0 && nsurv > (uint32_t)kRankMax) {
        // Too many candidates in the threshold bin to rank pair by pair. They differ in the low S key
        // bits and the index; the k_rem-th largest of these (low bits, lower index first) composites
        // is found digit by digit, 8 bits at a time from the top, with a 256-bin histogram over the
        // candidates that match the digits found so far. The composites sit in shared memory when
        // they fit, otherwise every pass reads the candidates again.
        static_assert(kThreads == 256, "one histogram bin per thread");
        unsigned long long* comp = reinterpret_cast<unsigned long long*>(surv);
        uint32_t* hist = sh_hist;
        const uint32_t lowmask = S ? ((1u << S) - 1u) : 0u;
        auto comp_of = [&](const uint2& cv) -> unsigned long long {
            const uint32_t o = (cv.y & 0x7fffffffu) - tau_hat;
            return ((unsigned long long)(o & lowmask) << 32) | (unsigned long long)(0xffffffffu - cv.x);
        };
        const bool in_smem = nsurv <= (uint32_t)kSurvSmem;
        if (in_smem)
            for (uint32_t q = threadIdx.x; q < nsurv; q += kThreads) comp[q] = comp_of(__ldcg(gsurv + q));
        unsigned long long prefix = 0ull;  // digits found so far, right-aligned
        uint32_t need = k_rem;             // rank still to be located among the candidates matching `prefix`
        const int top = ((S + 32 + 7) / 8 - 1) * 8;
        for (int shift = top; shift >= 0; shift -= 8) {
            __syncthreads();
            hist[threadIdx.x] = 0u;
            __syncthreads();
            for (uint32_t q = threadIdx.x; q < nsurv; q += kThreads) {
                const unsigned long long cq = in_smem ? comp[q] : comp_of(__ldcg(gsurv + q));
                const bool match = (shift + 8 >= 64) || ((cq >> (shift + 8)) == prefix);
                if (match) atomicAdd(&hist[(uint32_t)(cq >> shift) & 255u], 1u);
            }
            __syncthreads();
            // thread t looks at digit 255 - t: `incl` candidates have this digit or a larger one
            const uint32_t hv = hist[255 - threadIdx.x];
            uint32_t tot;
            const uint32_t incl = block_inclusive_scan(hv, scratch, &tot);
            if (incl - hv < need && need <= incl) {
                sh_base = 255u - threadIdx.x;
                sh_wcnt = incl - hv;
            }
            __syncthreads();
            prefix = (prefix << 8) | (unsigned long long)sh_base;
            need -= sh_wcnt;
        }
        // `prefix` is now the composite of the k_rem-th largest candidate (composites are distinct)
        const unsigned long long thr = prefix;
        tau = tau_hat + (uint32_t)(((unsigned long long)b0 << S) | (thr >> 32));
        kept_from = tau + 1u;
        __syncthreads();
        if (threadIdx.x == 0) {
            sh_base = atomicAdd(&st->emit_count, k_rem);
            sh_wcnt = 0u;
        }
        __syncthreads();
        for (uint32_t q = threadIdx.x; q < nsurv; q += kThreads) {
            const uint2 cv = __ldcg(gsurv + q);
            if (comp_of(cv) >= thr) {
                const uint32_t pos = sh_base + atomicAdd(&sh_wcnt, 1u);
                if (pos < kb) {
                    b.idx[slot0 + pos] = (int32_t)cv.x;
                    b.val[slot0 + pos] = __uint_as_float(cv.y);
                } else {
                    atomicOr(b.status, 1u);
                }
                erow[cv.x] = 0.0f;  // the residual of a kept coordinate: e = x - x
            }
        }
        __syncthreads();
        if (threadIdx.x == 0 && sh_wcnt != k_rem) atomicOr(b.status, 1u);
    } else if (!take_all0) {
        for (uint32_t q = threadIdx.x; q < nsurv; q += kThreads) surv[q] = __ldcg(gsurv + q);
        __syncthreads();
        // survivor q is kept when fewer than k_rem survivors beat it in (key, lower index first) order
        const uint32_t lowmask = S ? ((1u << S) - 1u) : 0u;
        auto comp_of = [&](const uint2& cv) -> unsigned long long {
            const uint32_t o = (cv.y & 0x7fffffffu) - tau_hat;
            return ((unsigned long long)(o & lowmask) << 32) | (unsigned long long)(0xffffffffu - cv.x);
        };
        for (uint32_t q0 = 0; q0 < nsurv; q0 += kThreads) {  // uniform trip count: the loop holds barriers
            const uint32_t q = q0 + threadIdx.x;
            bool kept = false;
            uint2 cv = make_uint2(0u, 0u);
            if (q < nsurv) {
                cv = surv[q];
                const unsigned long long mine_c = comp_of(cv);
                uint32_t beaten = 0;
                for (uint32_t p = 0; p < nsurv; ++p) beaten += (comp_of(surv[p]) > mine_c) ? 1u : 0u;
                kept = beaten < k_rem;
                if (beaten == k_rem - 1u) sh_tau = (cv.y & 0x7fffffffu);  // the k-th largest key overall
            }
            uint32_t tot3;
            const uint32_t incl = block_inclusive_scan(kept ? 1u : 0u, scratch, &tot3);
            if (threadIdx.x == 0) sh_base = tot3 ? atomicAdd(&st->emit_count, tot3) : 0u;
            __syncthreads();
            if (kept) {
                const uint32_t pos = sh_base + incl - 1u;
                if (pos < kb) {
                    b.idx[slot0 + pos] = (int32_t)cv.x;
                    b.val[slot0 + pos] = __uint_as_float(cv.y);
                } else {
                    atomicOr(b.status, 1u);
                }
                erow[cv.x] = 0.0f;  // the residual of a kept coordinate: e = x - x
            }
            __syncthreads();
        }
        tau = sh_tau;
        kept_from = tau + 1u;
    }
    if (threadIdx.x == 0) {
        b.thr[sg] = kept_from;
        uint32_t edge;
        if (edge_bin != 0xffffffffu) {
            const unsigned long long ew = (unsigned long long)tau_hat + ((unsigned long long)edge_bin << S);
            edge = ew < 0x7f7fffffull ? (uint32_t)ew : 0x7f7fffffu;
        } else {
            // fewer candidates than wanted: reach further down next time, by half the distance to the threshold
            const uint32_t gap = ((tau - tau_hat) >> 1) + (1u << 16);
            edge = tau_hat > gap ? tau_hat - gap : 0u;
        }
        predict_next(st, tau, edge, true);
        margin_after_selection(st, kb, c);
        st->fallback = 0u;
        atomicAdd(b.status + 2, 1u);  // selections decided inside their candidate list
    }
}

// ------------------------------------------------------------------------------------------
// dense passes, only for segments marked `fallback`

template <int PASS>
__device__ __forceinline__ void dense_hist(const Tables& t, const TopkBuffers& b, uint32_t* sh) {
    constexpr int NB = (PASS == 1) ? kBins1 : kBins23;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t total = (int64_t)t.n * t.ntiles;
    for (int64_t w = blockIdx.x; w < total; w += gridDim.x) {
        const int i = (int)(w / t.ntiles);
        const TileInfo ti = load_tile(t.tiles, (int)(w % t.ntiles));
        const size_t sg = (size_t)i * t.nseg + ti.seg;
        if (b.seg[sg].fallback == 0u) continue;
        const uint32_t prefix = b.seg[sg].prefix;
        for (int k = threadIdx.x; k < NB; k += kThreads) sh[k] = 0u;
        __syncthreads();
        const float* e = b.E + (size_t)i * (size_t)t.d + (size_t)ti.o;
        float4 xv[kIters];
        load_x_tile(e, ti.len, ti.r0, warp, lane, xv);
        int any = 0;
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int r = lane_r(ti.r0, warp, it, lane);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t key = mag_key(lane_elem(xv[it], k));
                const bool match = (PASS == 1) ? true : (PASS == 2) ? ((key >> 20) == prefix) : ((key >> 10) == prefix);
                if (match && r + k < ti.len) {
                    atomicAdd(&sh[(PASS == 1) ? (key >> 20) : (PASS == 2) ? ((key >> 10) & 1023u) : (key & 1023u)], 1u);
                    any = 1;
                }
            }
        }
        if (__syncthreads_or(any)) {
            uint32_t* h = b.hist + sg * kBins1;
            for (int k = threadIdx.x; k < NB; k += kThreads) {
                const uint32_t v = sh[k];
                if (v) atomicAdd(h + k, v);
            }
        }
        __syncthreads();
    }
}

constexpr int kLowBins = 64;  // fine bins at the bottom of the threshold's pass-1 bin that give the density there

template <int NBINS, int BITS, int PASS>
__device__ __forceinline__ void dense_find(const Tables& t, const TopkBuffers& b, size_t sg, uint32_t* scratch) {
    constexpr int PER = NBINS / kThreads;
    SegState* st = b.seg + sg;
    if (st->fallback == 0u) return;
    const SegInfo* si = t.segs + (sg % (size_t)t.nseg);
    uint32_t* h = b.hist + sg * kBins1;
    const uint32_t kb = si->kb;
    const uint32_t k_rem = (PASS == 1) ? kb : st->k_rem;
    const uint32_t prefix = (PASS == 1) ? 0u : st->prefix;
    // thread t owns the PER bins NBINS-1-t*PER ... downwards, so a scan over threads runs from the top bin down
    uint32_t cnt[PER];
    uint32_t sum = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const int bin = NBINS - 1 - ((int)threadIdx.x * PER + j);
        cnt[j] = h[bin];
        h[bin] = 0u;  // leave the histogram clean for the next pass / next step
        sum += cnt[j];
    }
    uint32_t total;
    const uint32_t incl = block_inclusive_scan(sum, scratch, &total);
    const uint32_t excl = incl - sum;
    if (excl < k_rem && k_rem <= incl) {
        uint32_t running = excl;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (running < k_rem && k_rem <= running + cnt[j]) {
                const uint32_t bin = (uint32_t)(NBINS - 1 - ((int)threadIdx.x * PER + j));
                const uint32_t np = (prefix << BITS) | bin;
                const uint32_t nk = k_rem - running;
                st->prefix = np;
                st->k_rem = nk;
                if (PASS == 3) {
                    // every key above np is kept, and the ties at np too unless only some fit: then the walk over
                    // the ties zeroes in E the ones it takes and everything from the next key up counts as kept
                    b.thr[sg] = (nk < cnt[j]) ? np + 1u : np;
                    st->tau = np;
                    st->ties_total = cnt[j];
                    st->ties_take = nk;
                    st->need_order = (nk < cnt[j]) ? 1u : 0u;
                    // prediction for the next step's sweep (blocks without a candidate buffer never predict)
                    predict_next(st, np, st->edge, si->cap != 0u);
                }
            }
            running += cnt[j];
        }
    }
    if (PASS == 1) {
        // the highest pass-1 bin edge at or above which at least the wanted number of candidates lie (0 if there
        // are fewer); a candidate path that gave up may have handed out message slots: start over
        const uint32_t want = want_candidates(kb, st->boost);
        if (threadIdx.x == 0) {
            st->emit_count = 0u;
            if (total < want) st->edge = 0u;
        }
        if (excl < want && want <= incl) {
            uint32_t running = excl;
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                if (running < want && want <= running + cnt[j])
                    st->edge = (uint32_t)(NBINS - 1 - ((int)threadIdx.x * PER + j)) << 20;
                running += cnt[j];
            }
        }
    }
    if constexpr (PASS == 2) {
        // Pass 1 places that edge on a grid of an eighth of a binade. Under error feedback the magnitudes pile up
        // just below the threshold (a coordinate grows until it is kept), so a bin edge a few per cent below the
        // threshold can let through many times the wanted number, more than the list holds, and the segment came
        // back to the dense passes step after step. When the wanted number is reached inside the threshold's own
        // pass-1 bin, this pass places the edge 1024 times finer; when that bin and the bins above hold fewer than
        // wanted, the edge is extrapolated below the bin's lower edge (see there).
        const uint32_t want = want_candidates(kb, st->boost);
        const uint32_t above = kb - k_rem;     // keys in the pass-1 bins above the threshold's
        const uint32_t want2 = want - above;   // want > kb > above
        if (excl < want2 && want2 <= incl) {
            uint32_t running = excl;
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                if (running < want2 && want2 <= running + cnt[j])
                    st->edge = (prefix << 20) | ((uint32_t)(NBINS - 1 - ((int)threadIdx.x * PER + j)) << 10);
                running += cnt[j];
            }
        } else if (total < want2 && threadIdx.x == kThreads - 1 - kLowBins / PER) {
            // The wanted count is reached below the threshold's pass-1 bin (the threshold sits just above a bin
            // boundary): the edge goes below the boundary by as far as the missing candidates need at the density
            // of the bin's lowest kLowBins fine bins. Further down the density only grows, so at least the wanted
            // number comes through, and far fewer than down to the next boundary. This thread's bins end where
            // those fine bins begin: `incl` counts everything above them.
            const uint32_t low = total - incl;
            if (low) {
                const unsigned long long ext = (unsigned long long)(want2 - total) * ((unsigned long long)kLowBins << 10) / low;
                const uint32_t top = prefix << 20;
                const uint32_t fine = ext < (unsigned long long)top ? top - (uint32_t)ext : 0u;
                if (fine > st->edge) st->edge = fine;  // never below the pass-1 edge, which is known to suffice
            }
        }
    }
    if (threadIdx.x == 0 && total < k_rem) atomicOr(b.status, 2u);
}

__device__ __forceinline__ void dense_collect(const Tables& t, const TopkBuffers& b, uint32_t* scratch,
                                              uint32_t* sh_base_p) {
    uint32_t& sh_base = *sh_base_p;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t total = (int64_t)t.n * t.ntiles;
    for (int64_t w = blockIdx.x; w < total; w += gridDim.x) {
        const int i = (int)(w / t.ntiles);
        const int tile = (int)(w % t.ntiles);
        const TileInfo ti = load_tile(t.tiles, tile);
        const size_t sg = (size_t)i * t.nseg + ti.seg;
        SegState* st = b.seg + sg;
        if (st->fallback == 0u) continue;
        const uint32_t tau = st->tau;
        const bool need_order = st->need_order != 0u;
        const float* e = b.E + (size_t)i * (size_t)t.d + (size_t)ti.o;
        float4 xv[kIters];
        load_x_tile(e, ti.len, ti.r0, warp, lane, xv);
        uint32_t n_emit = 0, n_tie = 0;
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int r = lane_r(ti.r0, warp, it, lane);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t key = mag_key(lane_elem(xv[it], k));
                const bool live = r + k < ti.len;
                n_emit += (live && key > tau) ? 1u : 0u;
                n_tie += (live && key == tau) ? 1u : 0u;
            }
        }
        if (!need_order) n_emit += n_tie;
        uint32_t tot, tie_tot = 0;
        const uint32_t incl = block_inclusive_scan(n_emit, scratch, &tot);
        if (need_order) {
            block_inclusive_scan(n_tie, scratch, &tie_tot);
            if (threadIdx.x == 0) b.tile_ties[(size_t)i * t.ntiles + tile] = tie_tot;
        }
        if (tot) {
            if (threadIdx.x == 0) sh_base = atomicAdd(&st->emit_count, tot);
            __syncthreads();
            const SegInfo* si = t.segs + ti.seg;
            const uint32_t kb = si->kb;
            const size_t slot0 = (size_t)i * (size_t)b.K + (size_t)si->slot0;
            uint32_t pos = sh_base + (incl - n_emit);
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int r = lane_r(ti.r0, warp, it, lane);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float x = lane_elem(xv[it], k);
                    const uint32_t key = mag_key(x);
                    const bool live = r + k < ti.len;
                    if (live && (key > tau || (!need_order && key == tau))) {
                        if (pos < kb) {
                            b.idx[slot0 + pos] = (int32_t)(ti.o + r + k);
                            b.val[slot0 + pos] = x;
                        } else {
                            atomicOr(b.status, 1u);
                        }
                        ++pos;
                    }
                }
            }
        }
        __syncthreads();  // sh_base and scratch are reused by the next tile
    }
}

// When the dense passes left threshold ties to order, takes those with the lowest index, tile by
// tile. The ties land in the message slots after the `emit_count` winners; the count itself is
// checked (with the ties added) when the step is closed.
__device__ __forceinline__ void dense_ties(const Tables& t, const TopkBuffers& b, size_t sg, uint32_t* scratch,
                                           uint32_t* sh_c, uint32_t* sh_excl) {
    const int i = (int)(sg / (size_t)t.nseg);
    const SegInfo* si = t.segs + (sg % (size_t)t.nseg);
    const SegState* st = b.seg + sg;
    if (st->fallback == 0u || st->need_order == 0u) return;
    const uint32_t kb = si->kb;
    const uint32_t emitted = st->emit_count;
    const uint32_t tau = st->tau;
    const uint32_t want = st->ties_take;
    if (emitted + want != kb) return;  // inconsistent: reported when the step is closed
    const int tile0 = si->tile0, tile_end = si->tile0 + si->ntile_b;
    const int64_t o = si->o;
    const int len = si->len;
    float* e = b.E + (size_t)i * (size_t)t.d + (size_t)o;
    const size_t slot0 = (size_t)i * (size_t)b.K + (size_t)si->slot0;
    uint32_t taken = 0;  // ties already assigned to earlier tiles (uniform across the CTA)
    for (int tb = tile0; tb < tile_end && taken < want; tb += kThreads) {
        const int tt = tb + (int)threadIdx.x;
        const uint32_t c = (tt < tile_end) ? b.tile_ties[(size_t)i * t.ntiles + tt] : 0u;
        uint32_t batch_total;
        const uint32_t incl = block_inclusive_scan(c, scratch, &batch_total);
        sh_c[threadIdx.x] = c;
        sh_excl[threadIdx.x] = incl - c;
        __syncthreads();
        const int nb = (tile_end - tb < kThreads) ? tile_end - tb : kThreads;
        for (int q = 0; q < nb; ++q) {
            const uint32_t cq = sh_c[q];
            if (cq == 0u) continue;
            const uint32_t before = taken + sh_excl[q];
            if (before >= want) break;
            const uint32_t take = (cq < want - before) ? cq : want - before;
            // tile tb+q in index order: thread j owns the 32 consecutive coordinates r0 + 32 j ...
            const int rs = (tb + q - tile0) * kTile + (int)threadIdx.x * 32;
            uint32_t mine = 0;
            for (int k = 0; k < 32; ++k) {
                const int r = rs + k;
                if (r < len && mag_key(e[r]) == tau) mine |= 1u << k;
            }
            uint32_t tile_tot;
            uint32_t rank = block_inclusive_scan((uint32_t)__popc(mine), scratch, &tile_tot) - __popc(mine);
            while (mine && rank < take) {
                const int k = __ffs(mine) - 1;
                mine &= mine - 1;
                const int r = rs + k;
                const uint32_t pos = emitted + before + rank;
                if (pos < kb) {
                    b.idx[slot0 + pos] = (int32_t)(o + r);
                    b.val[slot0 + pos] = e[r];
                }
                e[r] = 0.0f;  // the residual of a kept coordinate: e = x - x (this thread alone reads and writes e[r])
                ++rank;
            }
            __syncthreads();
        }
        taken += batch_total;
        __syncthreads();
    }
    if (threadIdx.x == 0 && taken < want) atomicOr(b.status, 1u);
}

// Closes the step for one large-block segment: exactly k_b entries must have been emitted; the counters go
// back to their resting values.
__device__ __forceinline__ void close_segment(const TopkBuffers& b, const SegInfo* si, SegState* st) {
    const bool dense = st->fallback != 0u;
    const uint32_t ties = (dense && st->need_order) ? st->ties_take : 0u;
    if (st->emit_count + ties != si->kb) atomicOr(b.status, 1u);
    if (dense) atomicAdd(b.status + 1, 1u);              // selections decided by the dense passes
    if (dense && si->cap) atomicSub(b.dense_count, 1u);  // back to the number of blocks that never predict
    st->emit_count = 0u;
    st->cand_count = 0u;
    st->fallback = si->cap ? 0u : 1u;  // blocks without a candidate buffer always take the dense passes
    st->need_order = 0u;
}

// All dense passes in one cooperative launch: the grid is resident as a whole and the passes are
// separated by grid-wide barriers. When no segment is marked every CTA returns at once, so in the
// steady state the dense path costs one empty launch per step.
__global__ void __launch_bounds__(kThreads) topk_dense_kernel(Tables t, TopkBuffers b) {
    __shared__ uint32_t sh[kBins1];
    __shared__ uint32_t scratch[kWarps];
    __shared__ uint32_t sh_c[kThreads], sh_excl[kThreads];
    __shared__ uint32_t sh_base;
    // the same word for every CTA; it only changes when the step is closed, in a later kernel
    if (*b.dense_count == 0u) return;
    cg::grid_group grid = cg::this_grid();
    const size_t nsg = (size_t)t.n * (size_t)t.nseg;
    dense_hist<1>(t, b, sh);
    grid.sync();
    for (size_t sg = blockIdx.x; sg < nsg; sg += gridDim.x) {
        dense_find<kBins1, 11, 1>(t, b, sg, scratch);
        __syncthreads();
    }
    grid.sync();
    dense_hist<2>(t, b, sh);
    grid.sync();
    for (size_t sg = blockIdx.x; sg < nsg; sg += gridDim.x) {
        dense_find<kBins23, 10, 2>(t, b, sg, scratch);
        __syncthreads();
    }
    grid.sync();
    dense_hist<3>(t, b, sh);
    grid.sync();
    for (size_t sg = blockIdx.x; sg < nsg; sg += gridDim.x) {
        dense_find<kBins23, 10, 3>(t, b, sg, scratch);
        __syncthreads();
    }
    grid.sync();
    dense_collect(t, b, scratch, &sh_base);
    grid.sync();
    for (size_t sg = blockIdx.x; sg < nsg; sg += gridDim.x) {
        dense_ties(t, b, sg, scratch, sh_c, sh_excl);
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------
// small blocks: the whole selection inside one CTA's shared memory

template <typename GT>
__global__ void __launch_bounds__(kThreads) topk_small_kernel(Tables t, TopkBuffers b, const GT* __restrict__ G) {
    __shared__ uint32_t xs[kSmallMax];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t scratch[kWarps];
    __shared__ uint32_t sh_prefix, sh_krem, sh_cnt, sh_rlast;
    const int blk = b.small_blk[blockIdx.x];
    const int i = blockIdx.y;
    const int64_t o = t.off[blk];
    const int len = (int)(t.off[blk + 1] - o);
    const uint32_t kb = (uint32_t)(b.seg_off[blk + 1] - b.seg_off[blk]);
    const GT* g = G + (size_t)i * (size_t)t.d + (size_t)o;
    float* e = b.E + (size_t)i * (size_t)t.d + (size_t)o;
    for (int r = threadIdx.x; r < len; r += kThreads) xs[r] = __float_as_uint(__fadd_rn(load1_stream(g + r), e[r]));

    // radix select over the 31-bit key: digits of 8, 8, 8 and 7 bits from the top
    uint32_t prefix = 0, k_rem = kb;
    int shift = 31;         // bits below `shift` are still undecided
    bool take_all = false;  // every key in the chosen bin is kept: no tie to break
#pragma unroll 1
    for (int pass = 0; pass < 4 && !take_all; ++pass) {
        const int width = (pass == 3) ? 7 : 8;
        const int nshift = shift - width;
        hist[threadIdx.x] = 0u;
        __syncthreads();
        for (int r = threadIdx.x; r < len; r += kThreads) {
            const uint32_t key = xs[r] & 0x7fffffffu;
            if (pass == 0 || (key >> shift) == prefix) atomicAdd(&hist[(key >> nshift) & ((1u << width) - 1u)], 1u);
        }
        __syncthreads();
        const uint32_t c = hist[255 - threadIdx.x];  // scan from the top bin down
        uint32_t total;
        const uint32_t incl = block_inclusive_scan(c, scratch, &total);
        const uint32_t excl = incl - c;
        if (excl < k_rem && k_rem <= incl) {
            sh_prefix = (prefix << width) | (uint32_t)(255 - threadIdx.x);
            sh_krem = k_rem - excl;
            sh_cnt = c;
        }
        __syncthreads();
        prefix = sh_prefix;
        k_rem = sh_krem;
        take_all = (sh_cnt == k_rem);
        shift = nshift;
        __syncthreads();
    }
    // kept: key >> shift > prefix, or == prefix and (take_all, or among the first k_rem such keys by index)
    const int chunk = (len + kThreads - 1) / kThreads;
    const int lo = (int)threadIdx.x * chunk;
    const int hi = (lo + chunk < len) ? lo + chunk : len;
    if (threadIdx.x == 0) sh_rlast = take_all ? 0x7fffffffu : 0u;
    __syncthreads();
    if (!take_all) {
        uint32_t mine = 0;
        for (int r = lo; r < hi; ++r) mine += ((xs[r] & 0x7fffffffu) == prefix) ? 1u : 0u;  // shift == 0 here
        uint32_t total;
        uint32_t rank = block_inclusive_scan(mine, scratch, &total) - mine;
        for (int r = lo; r < hi; ++r) {
            if ((xs[r] & 0x7fffffffu) == prefix) {
                if (rank == k_rem - 1) sh_rlast = (uint32_t)r;
                ++rank;
            }
        }
        __syncthreads();
    }
    const uint32_t rlast = sh_rlast;
    auto kept = [&](int r) -> bool {
        const uint32_t top = (xs[r] & 0x7fffffffu) >> shift;
        return top > prefix || (top == prefix && (uint32_t)r <= rlast);
    };
    uint32_t mine = 0;
    for (int r = lo; r < hi; ++r) mine += kept(r) ? 1u : 0u;
    uint32_t total;
    uint32_t pos = block_inclusive_scan(mine, scratch, &total) - mine;
    const size_t slot0 = (size_t)i * (size_t)b.K + (size_t)b.seg_off[blk];
    for (int r = lo; r < hi; ++r) {
        if (kept(r)) {
            if (pos < kb) {
                b.idx[slot0 + pos] = (int32_t)(o + r);
                b.val[slot0 + pos] = __uint_as_float(xs[r]);
            }
            ++pos;
        }
    }
    if (threadIdx.x == 0 && total != kb) atomicOr(b.status, 1u);
    // Algorithm 2, the residual update: e = x - g~ (0 where kept, x elsewhere)
    for (int r = threadIdx.x; r < len; r += kThreads) e[r] = kept(r) ? 0.0f : __uint_as_float(xs[r]);
}

// ------------------------------------------------------------------------------------------
// scatter: the kept (index, value) pairs of the messages are handed to the server grouped by coordinate range.

// All messages at once: `count` pairs of every worker the server averages over. The first n * nseg threads also
// close the step for one large-block segment each when `close` is set (Top-k; Random-k has no selection to close).
__global__ void __launch_bounds__(kThreads) topk_scatter_kernel(Tables t, TopkBuffers b, int64_t count, int close) {
    dependency_wait();
    allow_dependents();
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (close && p < (int64_t)t.n * t.nseg) close_segment(b, t.segs + (p % t.nseg), b.seg + p);
    const bool valid = p < count;
    int32_t j = 0;
    uint32_t xbits = 0;
    if (valid) {
        j = __ldg(b.idx + p);
        xbits = __float_as_uint(__ldg(b.val + p));
    }
    scatter_warp(b, valid, j, xbits);
}

// E holds x at the coordinates kept in the last step: zero them (Algorithm 2, the residual update). One CTA per
// (tile, worker); the kept elements of a segment are those whose magnitude reaches what its selection left.
__global__ void __launch_bounds__(kThreads) topk_materialize_kernel(Tables t, TopkBuffers b) {
    const int i = blockIdx.y;
    const TileInfo ti = load_tile(t.tiles, blockIdx.x);
    const float kept_from = __uint_as_float(b.thr[(size_t)i * t.nseg + ti.seg]);
    float* e = b.E + (size_t)i * (size_t)t.d + (size_t)ti.o;
    const int end = (ti.r0 + kTile < ti.len) ? ti.r0 + kTile : ti.len;
    for (int r = ti.r0 + (int)threadIdx.x; r < end; r += kThreads)
        if (fabsf(e[r]) >= kept_from) e[r] = 0.0f;
}

// ------------------------------------------------------------------------------------------

// The selection kernels see this handle's own rows of the message buffers; the server-side
// kernels see the rows of all n_total workers.
static TopkBuffers own_rows(const compams_context* c) {
    TopkBuffers b = c->tk;
    b.idx = c->tk.idx + (size_t)c->row0 * (size_t)c->K;
    b.val = c->tk.val + (size_t)c->row0 * (size_t)c->K;
    return b;
}

cudaError_t launch_topk_small(compams_context* c, const void* grads) {
    dim3 grid((unsigned)c->tk.nsmall, (unsigned)c->n);
    if (c->grad_bf16)
        topk_small_kernel<bf16_bits><<<grid, kThreads, 0, c->stream>>>(c->tab, own_rows(c), (const bf16_bits*)grads);
    else
        topk_small_kernel<float><<<grid, kThreads, 0, c->stream>>>(c->tab, own_rows(c), (const float*)grads);
    return counted(c, cudaGetLastError());
}

cudaError_t launch_topk_sweep(compams_context* c, const void* grads) {
    dim3 grid((unsigned)c->tab.ntiles, (unsigned)c->n);
    if (c->chain) {
        if (c->grad_bf16)
            return counted(c, launch_after(topk_sweep_kernel<bf16_bits>, grid, dim3(kThreads), c->stream, c->tab, own_rows(c),
                                (const bf16_bits*)grads, c->segp));
        return counted(c, launch_after(topk_sweep_kernel<float>, grid, dim3(kThreads), c->stream, c->tab, own_rows(c),
                            (const float*)grads, c->segp));
    }
    if (c->grad_bf16)
        topk_sweep_kernel<bf16_bits><<<grid, kThreads, 0, c->stream>>>(c->tab, own_rows(c), (const bf16_bits*)grads,
                                                                       c->segp);
    else
        topk_sweep_kernel<float><<<grid, kThreads, 0, c->stream>>>(c->tab, own_rows(c), (const float*)grads, c->segp);
    return counted(c, cudaGetLastError());
}

// While n d <= kChainMaxElems the kernels of a step are launched as programmatic dependents of one another (each
// waits for its predecessor before its first global access): the launch latency and the prologue of a
// kernel then overlap the tail of the one before, which is most of what such a step costs.
template <typename... KArgs, typename... Args>
static cudaError_t launch_chained(compams_context* c, void (*kernel)(KArgs...), dim3 grid, dim3 block, Args... args) {
    if (c->chain) return counted(c, launch_after(kernel, grid, block, c->stream, args...));
    kernel<<<grid, block, 0, c->stream>>>(static_cast<KArgs>(args)...);
    return counted(c, cudaGetLastError());
}

cudaError_t launch_topk_select(compams_context* c) {
    cudaError_t e = cudaSuccess;
    const TopkBuffers b = own_rows(c);
    if (c->n_sel_small > 0) {
        const int64_t lists = (int64_t)c->n * c->n_sel_small;
        if (lists >= 4 * (int64_t)c->num_sms)
            e = launch_chained(c, topk_select_kernel<kSelThreadsMany>, dim3((unsigned)lists), dim3(kSelThreadsMany), c->tab, b,
                               (const int32_t*)c->sel_small, c->n_sel_small);
        else
            e = launch_chained(c, topk_select_kernel<kSelThreads>, dim3((unsigned)lists), dim3(kSelThreads), c->tab, b,
                               (const int32_t*)c->sel_small, c->n_sel_small);
    }
    if (e != cudaSuccess || c->n_sel_big == 0) return e;
    const dim3 grid((unsigned)((int64_t)c->n * c->n_sel_big * c->sel_parts));
    e = launch_chained(c, topk_selhist_kernel, grid, dim3(kThreads), c->tab, b, (const int32_t*)c->sel_big, c->n_sel_big,
                       c->sel_parts);
    if (e != cudaSuccess) return e;
    return launch_chained(c, topk_selemit_kernel, grid, dim3(kThreads), c->tab, b, (const int32_t*)c->sel_big,
                          c->n_sel_big, c->sel_parts);
}

cudaError_t launch_topk_dense(compams_context* c) {
    if (c->dense_grid == 0) {
        int per_sm = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, topk_dense_kernel, kThreads, 0);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorLaunchOutOfResources;
        c->dense_grid = per_sm * c->num_sms;  // every CTA resident at once, as a cooperative launch requires
    }
    TopkBuffers b = own_rows(c);
    void* args[] = {(void*)&c->tab, (void*)&b};
    return counted(c, cudaLaunchCooperativeKernel((const void*)topk_dense_kernel, dim3((unsigned)c->dense_grid),
                                                  dim3(kThreads), args, 0, c->stream));
}

cudaError_t launch_topk_materialize(compams_context* c) {
    dim3 grid((unsigned)c->tab.ntiles, (unsigned)c->n);
    topk_materialize_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    return counted(c, cudaGetLastError());
}

cudaError_t launch_topk_scatter(compams_context* c, bool close) {
    // one thread per message entry of every worker (>= n * nseg: every block keeps at least one entry)
    const int64_t count = (int64_t)c->n_total * c->K;
    const unsigned grid = (unsigned)((count + kThreads - 1) / kThreads);
    // (a sharded handle's exchange sits in front of this kernel: a plain launch waits for it)
    if (c->chain && c->n == c->n_total)
        return counted(c, launch_after(topk_scatter_kernel, dim3(grid), dim3(kThreads), c->stream, c->tab, c->tk, count,
                                       close ? 1 : 0));
    topk_scatter_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk, count, close ? 1 : 0);
    return counted(c, cudaGetLastError());
}

}  // namespace compams

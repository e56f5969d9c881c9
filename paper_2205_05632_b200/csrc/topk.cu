// Top-k path (Definition 1) of the COMP-AMS step: exact selection of the k_b largest magnitudes
// of every (worker, block), ties at the threshold going to the lower index.
//
// Keys are the fp32 bit patterns of x = g + e with the sign cleared (31 bits); selection is a
// most-significant-digit radix select over them.
//
//   Blocks of at most kSmallMax coordinates: topk_small - one CTA holds the block in shared
//   memory and does every radix pass there; E is written once.
//
//   Larger blocks, cut into tiles of kTile coordinates:
//     topk_sweep    x = g + e written over E (Algorithm 2, line 7), histogram of key bits 30..20
//     topk_find     threshold bin of the pass just histogrammed; narrows (prefix, k_rem)
//     topk_hist     histogram of the next 10 key bits among the keys that match the prefix
//     topk_collect  after the last find: keys above the threshold are emitted as (index, value);
//                   threshold ties are emitted too unless only some of them fit, in which case
//                   they are counted per tile
//     topk_ties     takes the lowest-index threshold ties, tile by tile in index order
//   topk_scatter    walks the (index, value) messages: sum_i g~_i accumulated into a binary64
//                   buffer (line 12) and e zeroed at every kept coordinate (line 8: e = x - x)
#include "context.h"

namespace compams {

// ------------------------------------------------------------------------------------------
// tile loads shared by the large-block kernels

struct TileCoord {
    int i, tile, seg, blk;
    int64_t o, len, r0;
    size_t sg;  // i * nseg + seg
};

__device__ __forceinline__ TileCoord tile_coord(const Tables& t, int i, int tile) {
    TileCoord c;
    c.i = i;
    c.tile = tile;
    c.seg = t.tile_seg[tile];
    c.blk = t.tile_blk[tile];
    c.o = t.off[c.blk];
    c.len = t.off[c.blk + 1] - c.o;
    c.r0 = t.tile_r0[tile];
    c.sg = (size_t)i * t.nseg + c.seg;
    return c;
}

// Coordinates of lane `lane` of warp `warp` at iteration `it`: 4 consecutive ones starting here.
__device__ __forceinline__ int64_t lane_r(int64_t r0, int warp, int it, int lane) {
    return r0 + (int64_t)warp * kWarpSpan + it * 128 + lane * 4;
}

// Loads the 32 values of this thread's share of a tile of x (already stored in E).
// Coordinates past the block end read as +0 (callers mask them with `live`).
__device__ __forceinline__ void load_x_tile(const float* __restrict__ e, int64_t len, int64_t r0, int warp, int lane,
                                            float4 (&xv)[kIters]) {
    const int ce = align_class(e);
    if (r0 + kTile <= len) {
#pragma unroll
        for (int it = 0; it < kIters; ++it) xv[it] = load4(e + lane_r(r0, warp, it, lane), ce);
    } else {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int64_t r = lane_r(r0, warp, it, lane);
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
// sweep: x = g + e -> E, histogram of the top 11 key bits

template <bool FULL>
__device__ __forceinline__ void topk_sweep_tile(const float* __restrict__ g, float* __restrict__ e, int64_t len,
                                                int64_t r0, int warp, int lane, uint32_t* sh) {
    const int cg = align_class(g), ce = align_class(e);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        float4 gv[4], ev[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t r = lane_r(r0, warp, half * 4 + u, lane);
            if (FULL || r + 3 < len) {
                gv[u] = load4_stream(g + r, cg);
                ev[u] = load4_stream(e + r, ce);
            } else {
                float gt[4], et[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    gt[k] = (r + k < len) ? __ldcs(g + r + k) : 0.0f;
                    et[k] = (r + k < len) ? __ldcs(e + r + k) : 0.0f;
                }
                gv[u] = make_float4(gt[0], gt[1], gt[2], gt[3]);
                ev[u] = make_float4(et[0], et[1], et[2], et[3]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t r = lane_r(r0, warp, half * 4 + u, lane);
            float xs[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                xs[k] = __fadd_rn(lane_elem(gv[u], k), lane_elem(ev[u], k));  // line 7: x = g + e
                if (FULL || r + k < len) atomicAdd(&sh[mag_key(xs[k]) >> 20], 1u);
            }
            if (FULL || r + 3 < len) {
                store4(e + r, ce, make_float4(xs[0], xs[1], xs[2], xs[3]));
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (r + k < len) e[r + k] = xs[k];
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) topk_sweep_kernel(Tables t, TopkBuffers b, const float* __restrict__ G) {
    __shared__ uint32_t sh[kBins1];
    const TileCoord c = tile_coord(t, blockIdx.y, blockIdx.x);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int k = threadIdx.x; k < kBins1; k += kThreads) sh[k] = 0u;
    __syncthreads();
    const float* g = G + (size_t)c.i * (size_t)t.d + (size_t)c.o;
    float* e = b.E + (size_t)c.i * (size_t)t.d + (size_t)c.o;
    if (c.r0 + kTile <= c.len)
        topk_sweep_tile<true>(g, e, c.len, c.r0, warp, lane, sh);
    else
        topk_sweep_tile<false>(g, e, c.len, c.r0, warp, lane, sh);
    __syncthreads();
    uint32_t* h = b.hist + c.sg * kBins1;
    for (int k = threadIdx.x; k < kBins1; k += kThreads) {
        uint32_t v = sh[k];
        if (v) atomicAdd(h + k, v);
    }
}

// ------------------------------------------------------------------------------------------
// find: locate the bin that holds the k_rem-th largest key of a pass

template <int NBINS, int BITS, int PASS>
__global__ void __launch_bounds__(kThreads) topk_find_kernel(Tables t, TopkBuffers b) {
    __shared__ uint32_t scratch[kWarps];
    constexpr int PER = NBINS / kThreads;
    const size_t sg = blockIdx.x;
    const int seg = (int)(sg % (size_t)t.nseg);
    const int blk = t.tile_blk[t.seg_tile0[seg]];
    SegState* st = b.seg + sg;
    uint32_t* h = b.hist + sg * kBins1;
    const uint32_t kb = (uint32_t)(b.seg_off[blk + 1] - b.seg_off[blk]);
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
                    st->tau = np;
                    st->ties_total = cnt[j];
                    st->ties_take = nk;
                    st->need_order = (nk < cnt[j]) ? 1u : 0u;
                    st->emit_count = 0u;
                }
            }
            running += cnt[j];
        }
    }
    if (threadIdx.x == 0 && total < k_rem) atomicOr(b.status, 2u);
}

// ------------------------------------------------------------------------------------------
// hist: passes 2 and 3 over x (read back from E), restricted to keys that match the prefix

template <int PASS>
__global__ void __launch_bounds__(kThreads) topk_hist_kernel(Tables t, TopkBuffers b) {
    __shared__ uint32_t sh[kBins23];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t total = (int64_t)t.n * t.ntiles;
    for (int64_t w = blockIdx.x; w < total; w += gridDim.x) {
        const TileCoord c = tile_coord(t, (int)(w / t.ntiles), (int)(w % t.ntiles));
        const uint32_t prefix = b.seg[c.sg].prefix;
        for (int k = threadIdx.x; k < kBins23; k += kThreads) sh[k] = 0u;
        __syncthreads();
        const float* e = b.E + (size_t)c.i * (size_t)t.d + (size_t)c.o;
        float4 xv[kIters];
        load_x_tile(e, c.len, c.r0, warp, lane, xv);
        int any = 0;
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int64_t r = lane_r(c.r0, warp, it, lane);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t key = mag_key(lane_elem(xv[it], k));
                const bool match = (PASS == 2) ? ((key >> 20) == prefix) : ((key >> 10) == prefix);
                if (match && r + k < c.len) {
                    atomicAdd(&sh[(PASS == 2) ? ((key >> 10) & 1023u) : (key & 1023u)], 1u);
                    any = 1;
                }
            }
        }
        if (__syncthreads_or(any)) {
            uint32_t* h = b.hist + c.sg * kBins1;
            for (int k = threadIdx.x; k < kBins23; k += kThreads) {
                uint32_t v = sh[k];
                if (v) atomicAdd(h + k, v);
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------
// collect: emit everything above the threshold (and the ties when all of them fit)

__global__ void __launch_bounds__(kThreads) topk_collect_kernel(Tables t, TopkBuffers b) {
    __shared__ uint32_t scratch[kWarps];
    __shared__ uint32_t sh_base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t total = (int64_t)t.n * t.ntiles;
    for (int64_t w = blockIdx.x; w < total; w += gridDim.x) {
        const TileCoord c = tile_coord(t, (int)(w / t.ntiles), (int)(w % t.ntiles));
        SegState* st = b.seg + c.sg;
        const uint32_t tau = st->tau;
        const bool need_order = st->need_order != 0u;
        float* e = b.E + (size_t)c.i * (size_t)t.d + (size_t)c.o;
        float4 xv[kIters];
        load_x_tile(e, c.len, c.r0, warp, lane, xv);
        uint32_t n_emit = 0, n_tie = 0;
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int64_t r = lane_r(c.r0, warp, it, lane);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t key = mag_key(lane_elem(xv[it], k));
                const bool live = r + k < c.len;
                n_emit += (live && key > tau) ? 1u : 0u;
                n_tie += (live && key == tau) ? 1u : 0u;
            }
        }
        if (!need_order) n_emit += n_tie;
        uint32_t tot, tie_tot = 0;
        const uint32_t incl = block_inclusive_scan(n_emit, scratch, &tot);
        if (need_order) {
            block_inclusive_scan(n_tie, scratch, &tie_tot);
            if (threadIdx.x == 0) b.tile_ties[(size_t)c.i * t.ntiles + c.tile] = tie_tot;
        }
        if (tot) {
            if (threadIdx.x == 0) sh_base = atomicAdd(&st->emit_count, tot);
            __syncthreads();
            const uint32_t kb = (uint32_t)(b.seg_off[c.blk + 1] - b.seg_off[c.blk]);
            const size_t slot0 = (size_t)c.i * (size_t)b.K + (size_t)b.seg_off[c.blk];
            uint32_t pos = sh_base + (incl - n_emit);
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int64_t r = lane_r(c.r0, warp, it, lane);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float x = lane_elem(xv[it], k);
                    const uint32_t key = mag_key(x);
                    const bool live = r + k < c.len;
                    if (live && (key > tau || (!need_order && key == tau))) {
                        if (pos < kb) {
                            b.idx[slot0 + pos] = (int32_t)(c.o + r + k);
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

// ------------------------------------------------------------------------------------------
// ties: when only some of the keys equal to the threshold fit, take those with the lowest index

__global__ void __launch_bounds__(kThreads) topk_ties_kernel(Tables t, TopkBuffers b) {
    __shared__ uint32_t scratch[kWarps];
    __shared__ uint32_t sh_c[kThreads], sh_excl[kThreads];
    const size_t sg = blockIdx.x;
    const int i = (int)(sg / (size_t)t.nseg);
    const int seg = (int)(sg % (size_t)t.nseg);
    const int tile0 = t.seg_tile0[seg], tile_end = t.seg_tile0[seg + 1];
    const int blk = t.tile_blk[tile0];
    SegState* st = b.seg + sg;
    const uint32_t kb = (uint32_t)(b.seg_off[blk + 1] - b.seg_off[blk]);
    const uint32_t emitted = st->emit_count;
    if (!st->need_order) {
        if (threadIdx.x == 0 && emitted != kb) atomicOr(b.status, 1u);
        return;
    }
    const uint32_t tau = st->tau;
    const uint32_t want = st->ties_take;
    if (emitted + want != kb) {
        if (threadIdx.x == 0) atomicOr(b.status, 1u);
        return;
    }
    const int64_t o = t.off[blk];
    const int64_t len = t.off[blk + 1] - o;
    float* e = b.E + (size_t)i * (size_t)t.d + (size_t)o;
    const size_t slot0 = (size_t)i * (size_t)b.K + (size_t)b.seg_off[blk];
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
            const int64_t r0 = t.tile_r0[tb + q];
            const int64_t rs = r0 + (int64_t)threadIdx.x * 32;
            uint32_t mine = 0;
            for (int k = 0; k < 32; ++k) {
                const int64_t r = rs + k;
                if (r < len && mag_key(e[r]) == tau) mine |= 1u << k;
            }
            uint32_t tile_tot;
            const uint32_t rank0 = block_inclusive_scan((uint32_t)__popc(mine), scratch, &tile_tot) - __popc(mine);
            uint32_t rank = rank0;
            while (mine && rank < take) {
                const int k = __ffs(mine) - 1;
                mine &= mine - 1;
                const int64_t r = rs + k;
                const uint32_t pos = emitted + before + rank;
                if (pos < kb) {
                    b.idx[slot0 + pos] = (int32_t)(o + r);
                    b.val[slot0 + pos] = e[r];
                }
                ++rank;
            }
            __syncthreads();
        }
        taken += batch_total;
        __syncthreads();
    }
    if (threadIdx.x == 0 && taken < want) atomicOr(b.status, 1u);
}

// ------------------------------------------------------------------------------------------
// small blocks: the whole selection inside one CTA's shared memory

__global__ void __launch_bounds__(kThreads) topk_small_kernel(Tables t, TopkBuffers b, const float* __restrict__ G) {
    __shared__ uint32_t xs[kSmallMax];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t scratch[kWarps];
    __shared__ uint32_t sh_prefix, sh_krem, sh_cnt, sh_rlast;
    const int blk = b.small_blk[blockIdx.x];
    const int i = blockIdx.y;
    const int64_t o = t.off[blk];
    const int len = (int)(t.off[blk + 1] - o);
    const uint32_t kb = (uint32_t)(b.seg_off[blk + 1] - b.seg_off[blk]);
    const float* g = G + (size_t)i * (size_t)t.d + (size_t)o;
    float* e = b.E + (size_t)i * (size_t)t.d + (size_t)o;
    for (int r = threadIdx.x; r < len; r += kThreads) xs[r] = __float_as_uint(__fadd_rn(__ldcs(g + r), e[r]));

    // radix select over the 31-bit key: digits of 8, 8, 8 and 7 bits from the top
    uint32_t prefix = 0, k_rem = kb;
    int shift = 31;       // bits below `shift` are still undecided
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
    // Algorithm 2, line 8: e = x - g~ (0 where kept, x elsewhere)
    for (int r = threadIdx.x; r < len; r += kThreads) e[r] = kept(r) ? 0.0f : __uint_as_float(xs[r]);
}

// ------------------------------------------------------------------------------------------
// scatter: acc[j] += x_ij over all kept (i, j); binary64 atomics, exact hence order-independent.
// The same walk zeroes e at the kept coordinates (they were left holding x by the sweep).

__global__ void __launch_bounds__(kThreads) topk_scatter_kernel(int64_t K, int64_t d, int32_t n,
                                                                const int32_t* __restrict__ idx,
                                                                const float* __restrict__ val,
                                                                double* __restrict__ acc, float* __restrict__ E) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int i = 0; i < n; ++i) {
        const int32_t* ix = idx + (size_t)i * (size_t)K;
        const float* vx = val + (size_t)i * (size_t)K;
        float* e = E + (size_t)i * (size_t)d;
        for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < K; p += stride) {
            const int32_t j = ix[p];
            atomicAdd(acc + j, (double)vx[p]);
            e[j] = 0.0f;
        }
    }
}

// ------------------------------------------------------------------------------------------

static int persistent_grid(const compams_context* c, int64_t items, int ctas_per_sm) {
    int64_t cap = (int64_t)c->num_sms * ctas_per_sm;
    if (items < 1) items = 1;
    return (int)(items < cap ? items : cap);
}

cudaError_t launch_topk_small(compams_context* c, const float* grads) {
    dim3 grid((unsigned)c->tk.nsmall, (unsigned)c->n);
    topk_small_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk, grads);
    return cudaGetLastError();
}

cudaError_t launch_topk_sweep(compams_context* c, const float* grads) {
    dim3 grid((unsigned)c->tab.ntiles, (unsigned)c->n);
    topk_sweep_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk, grads);
    return cudaGetLastError();
}

cudaError_t launch_topk_find(compams_context* c, int pass) {
    const unsigned grid = (unsigned)((int64_t)c->n * c->tab.nseg);
    if (pass == 1)
        topk_find_kernel<kBins1, 11, 1><<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    else if (pass == 2)
        topk_find_kernel<kBins23, 10, 2><<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    else
        topk_find_kernel<kBins23, 10, 3><<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    return cudaGetLastError();
}

cudaError_t launch_topk_hist(compams_context* c, int pass) {
    const int grid = persistent_grid(c, (int64_t)c->n * c->tab.ntiles, 8);
    if (pass == 2)
        topk_hist_kernel<2><<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    else
        topk_hist_kernel<3><<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    return cudaGetLastError();
}

cudaError_t launch_topk_collect(compams_context* c) {
    const int grid = persistent_grid(c, (int64_t)c->n * c->tab.ntiles, 6);
    topk_collect_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    return cudaGetLastError();
}

cudaError_t launch_topk_ties(compams_context* c) {
    const unsigned grid = (unsigned)((int64_t)c->n * c->tab.nseg);
    topk_ties_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk);
    return cudaGetLastError();
}

cudaError_t launch_topk_scatter(compams_context* c) {
    const int grid = persistent_grid(c, (c->K + kThreads - 1) / kThreads, 8);
    topk_scatter_kernel<<<grid, kThreads, 0, c->stream>>>(c->K, c->d, c->n, c->tk.idx, c->tk.val, c->tk.acc, c->E);
    return cudaGetLastError();
}

}  // namespace compams

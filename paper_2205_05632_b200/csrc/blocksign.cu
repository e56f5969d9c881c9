// Block-Sign path (Definition 2) of the COMP-AMS step.
//
// bs_sweep   per (worker, tile): x = g + e (Algorithm 2, the corrected-gradient step), x written over E, sign bits
//            packed, sum |x| of the tile in binary64.
// bs_scales  per (worker, block): adds the tile sums in a fixed order and writes the scale
//            ||x_B||_1 / d_B.
// bs_apply   per coordinate: gbar = (1/n) sum_i sign(x_ij) s_{i,b} from the sign bits and
//            scales (the server's average), fused with the AMSGrad update (the moment, maximum and parameter updates).
//
// The residual e = x - sign(x) s (the residual update) needs the scale, which is known only after the whole
// block has been read. Instead of a second pass over [n, d], E keeps x and the subtraction is
// done when E is next read: by the next step's sweep (with the scale of the step that produced
// x) or by bs_materialize when the caller asks for E. Both evaluate the same single fp32
// subtraction, so the values are those of the residual update bit for bit.
#include "context.h"

namespace compams {

// Sign bits of the 4 values of this lane -> the 32-bit word of its 8-lane group (all 8 lanes get it).
__device__ __forceinline__ uint32_t pack_group_word(uint32_t nibble, int lane) {
    uint32_t w = nibble << ((lane & 7) * 4);
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    w |= __shfl_xor_sync(0xffffffffu, w, 4);
    return w;
}

// |x| as a binary64 number without a conversion instruction: for a normal fp32 value the
// binary64 pattern is the same fraction shifted left by 29 bits under an exponent rebiased by 896.
__device__ __forceinline__ double abs_as_double(float x) {
    const uint32_t b = __float_as_uint(x) & 0x7fffffffu;
    if ((b >> 23) == 0u) return (double)__uint_as_float(b);  // zero or subnormal: rare, take the conversion
    return __hiloint2double((int)((b >> 3) + 0x38000000u), (int)(b << 29));
}

// One warp's 1024 consecutive coordinates starting at rw (relative to the block; rw may be negative
// or reach past the block in a tile at either end of it: such coordinates are skipped).
template <bool FULL, typename GT>
__device__ __forceinline__ void bs_sweep_tile(const GT* __restrict__ g, float* __restrict__ e, int len, int rw,
                                              int lane, bool deferred, float sp, double& acc, uint32_t& mymask) {
    const int cg = align_class(g + rw), ce = align_class(e + rw);
    // One iteration (4 coordinates per lane) is worked on while the next one's loads are already in flight
    // (two register buffers that alternate; the loop is fully unrolled). Small batches keep the kernel at
    // 32 registers, eight CTAs per SM: measured 0.329 ms against 0.355 ms for two-iteration batches without
    // prefetch at five CTAs per SM (ResNet-18 shapes, n = 16), the rate of a plain device copy.
    constexpr int NB = 1;
    constexpr int NBT = kIters / NB;
    float4 gbuf[2][NB], ebuf[2][NB];
    auto load_batch = [&](int bt, float4 (&gv)[NB], float4 (&ev)[NB]) {
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int r = rw + (bt * NB + u) * 128 + lane * 4;
            if (FULL || (r >= 0 && r + 3 < len)) {
                gv[u] = load4_stream(g + r, cg);
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
    };
    load_batch(0, gbuf[0], ebuf[0]);
#pragma unroll
    for (int bt = 0; bt < NBT; ++bt) {
        float4 (&gv)[NB] = gbuf[bt & 1];
        float4 (&ev)[NB] = ebuf[bt & 1];
        if (bt + 1 < NBT) load_batch(bt + 1, gbuf[(bt + 1) & 1], ebuf[(bt + 1) & 1]);
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int it = bt * NB + u;
            const int r = rw + it * 128 + lane * 4;
            float xs[4];
            uint32_t nib = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float xo = lane_elem(ev[u], k);
                // deferred residual: e = x_prev - sign(x_prev) * s_prev (Algorithm 2, the residual update)
                float ee = deferred ? __fsub_rn(xo, copysignf(sp, xo)) : xo;
                float x = __fadd_rn(lane_elem(gv[u], k), ee);  // the corrected-gradient step: x = g + e
                xs[k] = x;
                const bool live = FULL || ((unsigned)(r + k) < (unsigned)len);
                if (live) {
                    acc += abs_as_double(x);
                    nib |= (__float_as_uint(x) >> 31) << k;
                }
            }
            if (FULL || (r >= 0 && r + 3 < len)) {
                store4(e + r, ce, make_float4(xs[0], xs[1], xs[2], xs[3]));
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if ((unsigned)(r + k) < (unsigned)len) e[r + k] = xs[k];
            }
            uint32_t w = pack_group_word(nib, lane);
            uint32_t wv = __shfl_sync(0xffffffffu, w, (lane & 3) * 8);
            if ((lane >> 2) == it) mymask = wv;  // lane l ends up holding the sign mask of the warp's l-th 32 coordinates
        }
    }
}

// The same for bfloat16 gradients on a whole tile whose rows of G and E are 16-byte aligned: 8 coordinates per
// lane and iteration, so that the gradient load is 128 bits wide like the two loads and stores of E (with 4
// coordinates per lane the 64-bit gradient loads leave too few bytes in flight: the sweep ran 8 % slower than
// with fp32 gradients although it reads fewer bytes). A warp's 1024 coordinates are 4 chunks of 256.
__device__ __forceinline__ void bs_sweep_tile_bf16x8(const bf16_bits* __restrict__ g, float* __restrict__ e, int rw, int lane,
                                                     bool deferred, float sp, double& acc, uint32_t& mymask) {
    constexpr int NC = kWarpSpan / 256;
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
        uint32_t bits8 = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float xs[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t word = gw[h * 2 + (k >> 1)];
                const float gk = __uint_as_float((k & 1) ? (word & 0xffff0000u) : (word << 16));  // exact widening
                const float xo = lane_elem(ev[h], k);
                // deferred residual: e = x_prev - sign(x_prev) * s_prev (Algorithm 2, the residual update)
                const float ee = deferred ? __fsub_rn(xo, copysignf(sp, xo)) : xo;
                const float x = __fadd_rn(gk, ee);  // the corrected-gradient step: x = g + e
                xs[k] = x;
                acc += abs_as_double(x);
                bits8 |= (__float_as_uint(x) >> 31) << (h * 4 + k);
            }
            *reinterpret_cast<float4*>(e + r + h * 4) = make_float4(xs[0], xs[1], xs[2], xs[3]);
        }
        // 4 lanes make one 32-bit word; word q of the chunk's 8 words sits in lanes 4q .. 4q + 3
        uint32_t w = bits8 << ((lane & 3) * 8);
        w |= __shfl_xor_sync(0xffffffffu, w, 1);
        w |= __shfl_xor_sync(0xffffffffu, w, 2);
        const uint32_t wv = __shfl_sync(0xffffffffu, w, (lane & 7) * 4);
        if ((lane >> 3) == c) mymask = wv;  // lane l ends up holding the sign mask of the warp's l-th 32 coordinates
    }
}

// Tiles are shifted down by s = (i d + o) mod 32, the position of the block's first element within
// a 128-byte line of G and E, so that every warp access covers whole lines (with rows that start
// mid-line a warp's 512 bytes straddle five lines instead of four: measured 7 % slower). The
// sign words stay indexed by coordinate: word q of the block takes its low 32 - s bits from the
// q-th group of 32 shifted coordinates and its high s bits from the next group. The word a tile
// shares with the next tile is put together by bs_scales from the two shares left in `edge`.
#ifndef COMPAMS_BF16_SWEEP_CTAS
#define COMPAMS_BF16_SWEEP_CTAS 5
#endif
template <typename GT>
__global__ void __launch_bounds__(kThreads, sizeof(GT) == 2 ? COMPAMS_BF16_SWEEP_CTAS : 8) bs_sweep_kernel(Tables t, BsBuffers b, const GT* __restrict__ G,
                                                               int deferred, const __grid_constant__ SegParams sp_) {
    __shared__ double red[kWarps];
    __shared__ uint32_t sh_first[kWarps];
    dependency_wait();  // while n d <= kChainMaxElems launched as a programmatic dependent of the step before (whose server
                        // kernel still reads the sign words this kernel is about to overwrite)
    allow_dependents();
    const int tile = blockIdx.x;
    const int i = blockIdx.y;
    const TileInfo ti = sp_.nseg ? find_tile(sp_, tile) : load_tile(t.tiles, tile);
    const int blk = ti.blk;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row0 = (int64_t)i * t.d + ti.o;
    const int s = (int)(row0 & 31);
    const GT* g = G + row0;
    float* e = b.E + row0;
    const float sp = deferred ? b.scales_prev[(size_t)i * t.M + blk] : 0.0f;
    const int r0s = ti.r0 - s;
    const int rw = r0s + warp * kWarpSpan;

    double acc = 0.0;
    uint32_t mymask = 0;
    const bool whole = r0s >= 0 && r0s + kTile <= ti.len;
    bool wide = false;
    if constexpr (sizeof(GT) == 2)
        wide = whole && ((reinterpret_cast<uintptr_t>(g + rw) | reinterpret_cast<uintptr_t>(e + rw)) & 15u) == 0;
    if (wide) {
        if constexpr (sizeof(GT) == 2) bs_sweep_tile_bf16x8(g, e, rw, lane, deferred != 0, sp, acc, mymask);
    } else if (whole) {
        bs_sweep_tile<true>(g, e, ti.len, rw, lane, deferred != 0, sp, acc, mymask);
    } else {
        bs_sweep_tile<false>(g, e, ti.len, rw, lane, deferred != 0, sp, acc, mymask);
    }

    // tile sum in binary64 (fixed shuffle tree); bs_scales adds the tile sums of a block in a fixed order
    if (lane == 0) sh_first[warp] = mymask;
    const double sum = block_sum_double(acc, red);  // its barriers also publish sh_first
    if (threadIdx.x == 0) b.tile_sum[(size_t)i * t.ntiles + tile] = sum;

    uint32_t next = __shfl_down_sync(0xffffffffu, mymask, 1);
    const bool last = warp == kWarps - 1 && lane == 31;
    if (lane == 31) next = last ? 0u : sh_first[warp + 1];
    const uint32_t word = __funnelshift_r(mymask, next, (uint32_t)s);  // s = 0: the mask itself
    const int q = (ti.r0 >> 5) + warp * 32 + lane;  // word of the block this lane completes
    const int wb = (ti.len + 31) >> 5;
    const int64_t wofs = sp_.nseg ? (int64_t)sp_.wofs[ti.seg] : b.word_off[blk];
    if (!last && q < wb) b.bits[(size_t)i * (size_t)b.W + (size_t)wofs + (size_t)q] = word;
    // shares of the two words in common with the neighbouring tiles: the high bits of the word before
    // this tile's first, the low bits of its last
    if (threadIdx.x == 0 || last) {
        uint32_t* ed = reinterpret_cast<uint32_t*>(b.edge + (size_t)i * t.ntiles + tile);
        if (last) ed[1] = word;
        else ed[0] = s ? (mymask << (32 - s)) : 0u;
    }
}

// One CTA per (worker, block): scale = ||x_B||_1 / d_B from the tile sums (Definition 2). Built for 256 threads
// (many blocks of a few tiles) and for 1024 with four tile sums requested at a time (a whole-vector block has
// thousands of tiles and only n CTAs to add them: 256 threads took 33 us at d = 2^26, n = 8, most of it waiting
// for one load after the other). The order of the additions is fixed by the tile count and the thread count,
// and every handle of a sharded run makes the same choice, so equal inputs give equal bits.
template <int NT>
__global__ void __launch_bounds__(NT) bs_scales_kernel(Tables t, BsBuffers b) {
    __shared__ double red[NT / 32];
    allow_dependents();
    dependency_wait();  // the sweep's tile sums and word shares
    const int blk = blockIdx.x, i = blockIdx.y;
    const SegInfo* si = t.segs + blk;
    const double* ts = b.tile_sum + (size_t)i * t.ntiles + si->tile0;
    const int nt = si->ntile_b;
    double part = 0.0;
    int k = threadIdx.x;
    for (; k + 3 * NT < nt; k += 4 * NT) {
        const double s0 = ts[k], s1 = ts[k + NT], s2 = ts[k + 2 * NT], s3 = ts[k + 3 * NT];
        part += s0;
        part += s1;
        part += s2;
        part += s3;
    }
    for (; k < nt; k += NT) part += ts[k];
    // the sign word two neighbouring tiles have in common: one share from each
    {
        const uint2* ed = b.edge + (size_t)i * t.ntiles + si->tile0;
        const int wb = (si->len + 31) >> 5;
        uint32_t* words = b.bits + (size_t)i * (size_t)b.W + (size_t)b.word_off[blk];
#pragma unroll 4
        for (int j = threadIdx.x; j < nt; j += NT) {
            const int q = (j + 1) * (kTile / 32) - 1;
            if (q < wb) words[q] = ed[j].y | (j + 1 < nt ? ed[j + 1].x : 0u);
        }
    }
    const double S = block_sum_double<NT / 32>(part, red);
    // one division in binary64, one rounding to fp32
    if (threadIdx.x == 0) b.scales_cur[(size_t)i * t.M + blk] = __double2float_rn(S / (double)si->len);
}

// E holds x; turn it into e = x - sign(x) * s in place (Algorithm 2, the residual update).
__global__ void __launch_bounds__(kThreads) bs_materialize_kernel(Tables t, float* __restrict__ E,
                                                                  const float* __restrict__ scales) {
    const int i = blockIdx.y;
    const TileInfo ti = load_tile(t.tiles, blockIdx.x);
    const int blk = ti.blk;
    const int64_t o = ti.o;
    const int64_t len = ti.len;
    const int64_t r0 = ti.r0;
    const float s = scales[(size_t)i * t.M + blk];
    float* e = E + (size_t)i * (size_t)t.d + (size_t)o;
    const int64_t end = (r0 + kTile < len) ? r0 + kTile : len;
    for (int64_t r = r0 + threadIdx.x; r < end; r += kThreads) {
        float x = e[r];
        e[r] = __fsub_rn(x, copysignf(s, x));
    }
}

constexpr int kApplyChunk = 32;  // workers whose sign words are staged (and transposed) at a time: one per lane
#ifndef COMPAMS_APPLY_TABLES_FROM
#define COMPAMS_APPLY_TABLES_FROM 20
#endif
constexpr int kApplyTablesFrom = COMPAMS_APPLY_TABLES_FROM;  // workers from which the table form of bs_apply is used

// Transposes four 32 x 32 bit matrices held across a warp: on entry lane i holds x[q] = row i of matrix q
// (bit c = element (i, c)); on return lane c holds column c (bit i = element (i, c)). Five rounds of the
// usual block swap: in round j a lane exchanges with lane ^ j the half of its bits whose position differs
// from its own index in bit j. Shifting the partner's word by +-j and keeping only the positions that
// change is a rotation followed by a bitwise select.
__device__ __forceinline__ void transpose32x4(uint32_t (&x)[4], int lane) {
#pragma unroll
    for (int j = 16; j >= 1; j >>= 1) {
        const uint32_t m = j == 16 ? 0x0000ffffu : j == 8 ? 0x00ff00ffu : j == 4 ? 0x0f0f0f0fu : j == 2 ? 0x33333333u : 0x55555555u;
        const bool up = (lane & j) != 0;
        const uint32_t keep = up ? ~m : m;          // positions whose bit j equals the lane's stay
        const uint32_t rot = up ? 32u - j : (uint32_t)j;  // the partner's bits move down (up) by j
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t y = __shfl_xor_sync(0xffffffffu, x[q], j);
            x[q] = (x[q] & keep) | (__funnelshift_l(y, y, rot) & ~keep);
        }
    }
}

// Server side of Block-Sign (Algorithm 2, the server's average and update): one CTA per 1024 consecutive
// coordinates of a block, one float4 group per thread. The tile's block comes from the constant bank, so the
// sign words, the scales and the optimizer state are all requested at once.
//
// Per coordinate the sum over workers of +-s_i is (sum of all s_i) - 2 (sum of the s_i whose bit is set).
// TABLES = false (few workers): one predicated binary64 add per worker and coordinate.
// TABLES = true: the second sum depends only on the coordinate's pattern of sign bits over the workers, and all
// 1024 coordinates of the CTA share the workers' scales: for every 4 workers a 16-entry table holds the sum of
// each subset of their scales (exact in binary64 wherever the plain sum is), and a coordinate adds one table entry
// per 4 workers instead of testing one bit per worker. The patterns come from transposing the sign words in the
// warp: lane i reads worker i's four words of the warp's 128 coordinates, transpose32x4 turns them into one word
// per coordinate, and 16 shuffles hand every lane the patterns of its own 4 coordinates. Up to 32 workers per
// round. The kernel is bound by instruction issue: the fixed cost of the transposition (36 shuffles per round)
// pays from about two dozen workers up (n = 32, d = 2^27: step 9.23 -> 8.87 ms; n = 16: no change; n = 8: 3 %
// slower, hence the two forms).
template <bool TABLES, bool RECORD>
__global__ void __launch_bounds__(kThreads, 5) bs_apply_kernel(Tables t, BsBuffers b, float* __restrict__ theta,
                                                               HyperParams hp,
                                                               const __grid_constant__ SegParams sp_) {
    __shared__ uint32_t sh_bits[kApplyChunk][33];        // [worker][word], rows padded against bank conflicts
    __shared__ double sh_tab[kApplyChunk / 4][16];       // TABLES: [group of 4 workers][subset] sum of the subset's
                                                         // scales; else: the workers' scales
    const int tile = blockIdx.x >> 3;
    const TileInfo ti = sp_.nseg ? find_tile(sp_, tile) : load_tile(t.tiles, tile);
    const int blk = ti.blk;
    const int len = ti.len;
    const int rs = ti.r0 + (int)(blockIdx.x & 7) * kWarpSpan;  // first coordinate of this CTA, relative to the block
    if (rs >= len) return;
    const int r = rs + (int)threadIdx.x * 4;
    const int64_t o = ti.o;
    float* gbar = b.gbar + o;
    float* m = b.m + o;
    float* v = b.v + o;
    float* vh = b.vhat + o;
    float* th = theta + o;
    const int cls = align_class(m);  // all five vectors are 16-byte aligned at coordinate 0
    const bool full = r + 3 < len;
    float4 mm = make_float4(0.f, 0.f, 0.f, 0.f), vv = mm, hh = mm, tt = mm;
    if (full) {
        mm = load4(m + r, cls);
        vv = load4(v + r, cls);
        hh = load4(vh + r, cls);
        tt = load4(th + r, cls);
    }
    dependency_wait();  // the state above was last written a step ago; sign words and scales are this step's
    const size_t wbase = (size_t)(sp_.nseg ? (int64_t)sp_.wofs[ti.seg] : b.word_off[blk]) + (size_t)(rs >> 5);
    const int lane = threadIdx.x & 31, wr = threadIdx.x >> 5;  // warp wr owns coordinates 128 wr ... of the CTA's 1024
    const bool word_live = rs + lane * 32 < len;
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0, all = 0.0;
    for (int i0 = 0; i0 < t.n; i0 += kApplyChunk) {
        const int nc = (t.n - i0 < kApplyChunk) ? t.n - i0 : kApplyChunk;
        __syncthreads();
        // warp wr stages the words of workers wr, wr + 8, ...: 32 consecutive words each, one per lane
        for (int c = wr; c < nc; c += kWarps)
            sh_bits[c][lane] = word_live ? __ldg(b.bits + (size_t)(i0 + c) * (size_t)b.W + wbase + lane) : 0u;
        if constexpr (TABLES) {
            const int ng = (nc + 3) >> 2;  // groups of 4 workers in this round
            if (threadIdx.x < ng * 16) {   // one table entry per thread: the scales of the subset's members
                const int gq = threadIdx.x >> 4, sub = threadIdx.x & 15;
                double e = 0.0;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (((sub >> j) & 1) && gq * 4 + j < nc)
                        e += (double)b.scales_cur[(size_t)(i0 + gq * 4 + j) * t.M + blk];
                sh_tab[gq][sub] = e;
            }
            __syncthreads();
            // lane i: worker i's words of this warp's coordinates -> lane c: the workers' bits of coordinate 32 q + c
            uint32_t x[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) x[q] = lane < nc ? sh_bits[lane][wr * 4 + q] : 0u;
            transpose32x4(x, lane);
            // this thread's coordinates 4 lane + k lie in word q = lane / 8 at bit 4 (lane % 8) + k: their patterns
            // sit in lane 4 (lane % 8) + k, matrix lane / 8 (a trip through shared memory instead of these 16
            // shuffles was slower)
            uint4 pat = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t y0 = __shfl_sync(0xffffffffu, x[q], (lane & 7) * 4 + 0);
                const uint32_t y1 = __shfl_sync(0xffffffffu, x[q], (lane & 7) * 4 + 1);
                const uint32_t y2 = __shfl_sync(0xffffffffu, x[q], (lane & 7) * 4 + 2);
                const uint32_t y3 = __shfl_sync(0xffffffffu, x[q], (lane & 7) * 4 + 3);
                if ((lane >> 3) == q) pat = make_uint4(y0, y1, y2, y3);
            }
#pragma unroll
            for (int gq = 0; gq < kApplyChunk / 4; ++gq) {
                if (gq < ng) {  // the same for every thread of the CTA
                    all += sh_tab[gq][15];
                    a0 += sh_tab[gq][(pat.x >> (4 * gq)) & 15u];
                    a1 += sh_tab[gq][(pat.y >> (4 * gq)) & 15u];
                    a2 += sh_tab[gq][(pat.z >> (4 * gq)) & 15u];
                    a3 += sh_tab[gq][(pat.w >> (4 * gq)) & 15u];
                }
            }
        } else {
            double* sh_s = &sh_tab[0][0];
            if (threadIdx.x < nc) sh_s[threadIdx.x] = (double)b.scales_cur[(size_t)(i0 + threadIdx.x) * t.M + blk];
            __syncthreads();
            const int wsel = threadIdx.x >> 3, nsh = (threadIdx.x & 7) * 4;  // this thread's word and its nibble in it
#pragma unroll 4
            for (int c = 0; c < nc; ++c) {
                const double sc = sh_s[c];
                const uint32_t nib = sh_bits[c][wsel] >> nsh;
                all += sc;
                if (nib & 1u) a0 += sc;
                if (nib & 2u) a1 += sc;
                if (nib & 4u) a2 += sc;
                if (nib & 8u) a3 += sc;
            }
        }
    }
    a0 = all - (a0 + a0);
    a1 = all - (a1 + a1);
    a2 = all - (a2 + a2);
    a3 = all - (a3 + a3);
    if (r >= len) return;
    const float gb[4] = {mean_from_acc(a0, hp), mean_from_acc(a1, hp), mean_from_acc(a2, hp),
                         mean_from_acc(a3, hp)};
    if (full) {
        amsgrad_update(gb[0], mm.x, vv.x, hh.x, tt.x, hp);
        amsgrad_update(gb[1], mm.y, vv.y, hh.y, tt.y, hp);
        amsgrad_update(gb[2], mm.z, vv.z, hh.z, tt.z, hp);
        amsgrad_update(gb[3], mm.w, vv.w, hh.w, tt.w, hp);
        if constexpr (RECORD) store4(gbar + r, cls, make_float4(gb[0], gb[1], gb[2], gb[3]));
        store4(m + r, cls, mm);
        store4(v + r, cls, vv);
        store4(vh + r, cls, hh);
        store4(th + r, cls, tt);
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (r + k < len) {
                float m1 = m[r + k], v1 = v[r + k], h1 = vh[r + k], t1 = th[r + k];
                amsgrad_update(gb[k], m1, v1, h1, t1, hp);
                if constexpr (RECORD) gbar[r + k] = gb[k];
                m[r + k] = m1;
                v[r + k] = v1;
                vh[r + k] = h1;
                th[r + k] = t1;
            }
        }
    }
}

// The worker-side kernels see this handle's own rows of the message buffers (sign words, scales);
// the server kernel sees the rows of all n_total workers.
static BsBuffers own_rows(const compams_context* c) {
    BsBuffers b = c->bs;
    const size_t r0 = (size_t)c->row0;
    b.bits = c->bs.bits + r0 * (size_t)c->W;
    b.scales_prev = c->scales[c->scales_cur ^ 1] + r0 * (size_t)c->M;
    b.scales_cur = c->scales[c->scales_cur] + r0 * (size_t)c->M;
    return b;
}

cudaError_t launch_bs_sweep(compams_context* c, const void* grads) {
    dim3 grid((unsigned)c->tab.ntiles, (unsigned)c->n);
    if (c->chain) {  // n d <= kChainMaxElems: the launch overlaps the tail of whatever kernel precedes it on the stream
        if (c->grad_bf16)
            return counted(c, launch_after(bs_sweep_kernel<bf16_bits>, grid, dim3(kThreads), c->stream, c->tab, own_rows(c),
                                (const bf16_bits*)grads, c->e_is_x ? 1 : 0, c->segp));
        return counted(c, launch_after(bs_sweep_kernel<float>, grid, dim3(kThreads), c->stream, c->tab, own_rows(c),
                            (const float*)grads, c->e_is_x ? 1 : 0, c->segp));
    }
    if (c->grad_bf16)
        bs_sweep_kernel<bf16_bits><<<grid, kThreads, 0, c->stream>>>(c->tab, own_rows(c), (const bf16_bits*)grads,
                                                                     c->e_is_x ? 1 : 0, c->segp);
    else
        bs_sweep_kernel<float><<<grid, kThreads, 0, c->stream>>>(c->tab, own_rows(c), (const float*)grads,
                                                                 c->e_is_x ? 1 : 0, c->segp);
    return counted(c, cudaGetLastError());
}

cudaError_t launch_bs_scales(compams_context* c) {
    dim3 grid((unsigned)c->M, (unsigned)c->n);
    if (c->tab.ntiles > 256 * (int64_t)c->M)  // on average more than 256 tiles to a block
        return counted(c, launch_after(bs_scales_kernel<1024>, grid, dim3(1024), c->stream, c->tab, own_rows(c)));
    return counted(c, launch_after(bs_scales_kernel<kThreads>, grid, dim3(kThreads), c->stream, c->tab, own_rows(c)));
}

cudaError_t launch_bs_apply(compams_context* c, float* theta) {
    BsBuffers b = c->bs;
    b.scales_cur = c->scales[c->scales_cur];
    Tables t = c->tab;
    t.n = c->n_total;  // the average runs over every worker's message
    const dim3 grid((unsigned)c->tab.ntiles * kWarps);
    const bool tables = c->n_total >= kApplyTablesFrom;
    // four builds: the inner sum by tables or worker by worker; gbar stored or not (a run-time branch around the
    // store slowed the kernel by a tenth)
    void (*kernel)(Tables, BsBuffers, float*, HyperParams, const SegParams) =
        tables ? (b.gbar ? bs_apply_kernel<true, true> : bs_apply_kernel<true, false>)
               : (b.gbar ? bs_apply_kernel<false, true> : bs_apply_kernel<false, false>);
    if (c->n == c->n_total) return counted(c, launch_after(kernel, grid, dim3(kThreads), c->stream, t, b, theta, c->hp, c->segp));
    // sharded workers: the other workers' messages were written by the caller's exchange, which is
    // ordered on the stream like any kernel; a plain launch waits for it
    kernel<<<grid, dim3(kThreads), 0, c->stream>>>(t, b, theta, c->hp, c->segp);
    return counted(c, cudaGetLastError());
}

cudaError_t launch_bs_materialize(compams_context* c) {
    dim3 grid((unsigned)c->tab.ntiles, (unsigned)c->n);
    bs_materialize_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->E, c->scales[c->scales_cur] + (size_t)c->row0 * (size_t)c->M);
    return counted(c, cudaGetLastError());
}

}  // namespace compams

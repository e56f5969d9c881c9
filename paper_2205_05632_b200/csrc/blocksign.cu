// Block-Sign path (Definition 2) of the COMP-AMS step.
//
// bs_sweep   per (worker, tile): x = g + e (Algorithm 2, line 7), x written over E, sign bits
//            packed, sum |x| of the tile in binary64.
// bs_scales  per (worker, block): adds the tile sums in a fixed order and writes the scale
//            ||x_B||_1 / d_B.
// bs_apply   per coordinate: gbar = (1/n) sum_i sign(x_ij) s_{i,b} from the sign bits and
//            scales (line 12), fused with the AMSGrad update (lines 13-16).
//
// The residual e = x - sign(x) s (line 8) needs the scale, which is known only after the whole
// block has been read. Instead of a second pass over [n, d], E keeps x and the subtraction is
// done when E is next read: by the next step's sweep (with the scale of the step that produced
// x) or by bs_materialize when the caller asks for E. Both evaluate the same single fp32
// subtraction, so the values are those of line 8 bit for bit.
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

template <bool FULL>
__device__ __forceinline__ void bs_sweep_tile(const float* __restrict__ g, float* __restrict__ e, int len, int rw,
                                              int lane, bool deferred, float sp, double& acc, uint32_t& myword) {
    const int cg = align_class(g), ce = align_class(e);
#pragma unroll
    for (int bt = 0; bt < kIters / 2; ++bt) {
        float4 gv[2], ev[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int r = rw + (bt * 2 + u) * 128 + lane * 4;
            if (FULL || r + 3 < len) {
                gv[u] = load4_stream(g + r, cg);
                ev[u] = load4(e + r, ce);
            } else {
                float gt[4], et[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    gt[k] = (r + k < len) ? __ldg(g + r + k) : 0.0f;
                    et[k] = (r + k < len) ? e[r + k] : 0.0f;
                }
                gv[u] = make_float4(gt[0], gt[1], gt[2], gt[3]);
                ev[u] = make_float4(et[0], et[1], et[2], et[3]);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int it = bt * 2 + u;
            const int r = rw + it * 128 + lane * 4;
            float xs[4];
            uint32_t nib = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float xo = lane_elem(ev[u], k);
                // deferred residual: e = x_prev - sign(x_prev) * s_prev (Algorithm 2, line 8)
                float ee = deferred ? __fsub_rn(xo, copysignf(sp, xo)) : xo;
                float x = __fadd_rn(lane_elem(gv[u], k), ee);  // line 7: x = g + e
                xs[k] = x;
                const bool live = FULL || (r + k < len);
                if (live) {
                    acc += abs_as_double(x);
                    nib |= (__float_as_uint(x) >> 31) << k;
                }
            }
            if (FULL || r + 3 < len) {
                store4(e + r, ce, make_float4(xs[0], xs[1], xs[2], xs[3]));
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (r + k < len) e[r + k] = xs[k];
            }
            uint32_t w = pack_group_word(nib, lane);
            uint32_t wv = __shfl_sync(0xffffffffu, w, (lane & 3) * 8);
            if ((lane >> 2) == it) myword = wv;  // lane l ends up holding word l of the warp's 32 words
        }
    }
}

__global__ void __launch_bounds__(kThreads, 5) bs_sweep_kernel(Tables t, BsBuffers b, const float* __restrict__ G,
                                                               int deferred, const __grid_constant__ SegParams sp_) {
    __shared__ double red[kWarps];
    const int tile = blockIdx.x;
    const int i = blockIdx.y;
    const TileInfo ti = sp_.nseg ? find_tile(sp_, tile) : load_tile(t.tiles, tile);
    const int blk = ti.blk;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* g = G + (size_t)i * (size_t)t.d + (size_t)ti.o;
    float* e = b.E + (size_t)i * (size_t)t.d + (size_t)ti.o;
    const float sp = deferred ? b.scales_prev[(size_t)i * t.M + blk] : 0.0f;
    const int rw = ti.r0 + warp * kWarpSpan;

    double acc = 0.0;
    uint32_t myword = 0;
    if (ti.r0 + kTile <= ti.len)
        bs_sweep_tile<true>(g, e, ti.len, rw, lane, deferred != 0, sp, acc, myword);
    else
        bs_sweep_tile<false>(g, e, ti.len, rw, lane, deferred != 0, sp, acc, myword);

    if (rw + lane * 32 < ti.len)
        b.bits[(size_t)i * (size_t)b.W + (size_t)b.word_off[blk] + (size_t)(rw >> 5) + lane] = myword;

    // tile sum in binary64 (fixed shuffle tree); bs_scales adds the tile sums of a block in a fixed order
    double s = block_sum_double(acc, red);
    if (threadIdx.x == 0) b.tile_sum[(size_t)i * t.ntiles + tile] = s;
}

// One CTA per (worker, block): scale = ||x_B||_1 / d_B from the tile sums (Definition 2).
__global__ void __launch_bounds__(kThreads) bs_scales_kernel(Tables t, BsBuffers b) {
    __shared__ double red[kWarps];
    const int blk = blockIdx.x, i = blockIdx.y;
    const SegInfo* si = t.segs + blk;
    const double* ts = b.tile_sum + (size_t)i * t.ntiles + si->tile0;
    double part = 0.0;
    for (int k = threadIdx.x; k < si->ntile_b; k += kThreads) part += ts[k];
    const double S = block_sum_double(part, red);
    // one division in binary64, one rounding to fp32
    if (threadIdx.x == 0) b.scales_cur[(size_t)i * t.M + blk] = __double2float_rn(S / (double)si->len);
}

// E holds x; turn it into e = x - sign(x) * s in place (Algorithm 2, line 8).
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

constexpr int kApplyChunk = 64;  // workers whose sign words are staged in shared memory at a time

// One CTA per 1024 consecutive coordinates of a block (one float4 group per thread).
__global__ void __launch_bounds__(kThreads, 6) bs_apply_kernel(Tables t, BsBuffers b, float* __restrict__ theta,
                                                               HyperParams hp) {
    __shared__ uint32_t sh_bits[kApplyChunk][32];
    __shared__ double sh_s[kApplyChunk];
    const TileInfo ti = load_tile(t.tiles, blockIdx.x >> 3);
    const int blk = ti.blk;
    const int len = ti.len;
    const int rs = ti.r0 + (int)(blockIdx.x & 7) * kWarpSpan;  // first coordinate of this CTA, relative to the block
    if (rs >= len) return;
    const int r = rs + (int)threadIdx.x * 4;
    const int wsel = threadIdx.x >> 3, nsh = (threadIdx.x & 7) * 4;

    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    const size_t wbase = (size_t)b.word_off[blk] + (size_t)(rs >> 5);
    const int wl = threadIdx.x & 31, wr = threadIdx.x >> 5;  // word and worker this thread stages
    const bool word_live = rs + wl * 32 < len;
    for (int i0 = 0; i0 < t.n; i0 += kApplyChunk) {
        const int nc = (t.n - i0 < kApplyChunk) ? t.n - i0 : kApplyChunk;
        __syncthreads();
        for (int c = wr; c < nc; c += kWarps)
            sh_bits[c][wl] = word_live ? __ldg(b.bits + (size_t)(i0 + c) * (size_t)b.W + wbase + wl) : 0u;
        if (threadIdx.x < nc) sh_s[threadIdx.x] = (double)b.scales_cur[(size_t)(i0 + threadIdx.x) * t.M + blk];
        __syncthreads();
#pragma unroll 4
        for (int c = 0; c < nc; ++c) {
            const double s = sh_s[c];
            const double ns = -s;
            const uint32_t nib = sh_bits[c][wsel] >> nsh;
            a0 += (nib & 1u) ? ns : s;
            a1 += (nib & 2u) ? ns : s;
            a2 += (nib & 4u) ? ns : s;
            a3 += (nib & 8u) ? ns : s;
        }
    }
    if (r >= len) return;
    const int64_t o = ti.o;
    float* gbar = b.gbar + o;
    float* m = b.m + o;
    float* v = b.v + o;
    float* vh = b.vhat + o;
    float* th = theta + o;
    const int cls = align_class(m);  // all five vectors are 16-byte aligned at coordinate 0
    const float gb[4] = {mean_from_acc(a0, hp.nf), mean_from_acc(a1, hp.nf), mean_from_acc(a2, hp.nf),
                         mean_from_acc(a3, hp.nf)};
    if (r + 3 < len) {
        float4 mm = load4(m + r, cls), vv = load4(v + r, cls), hh = load4(vh + r, cls), tt = load4(th + r, cls);
        amsgrad_update(gb[0], mm.x, vv.x, hh.x, tt.x, hp);
        amsgrad_update(gb[1], mm.y, vv.y, hh.y, tt.y, hp);
        amsgrad_update(gb[2], mm.z, vv.z, hh.z, tt.z, hp);
        amsgrad_update(gb[3], mm.w, vv.w, hh.w, tt.w, hp);
        store4(gbar + r, cls, make_float4(gb[0], gb[1], gb[2], gb[3]));
        store4(m + r, cls, mm);
        store4(v + r, cls, vv);
        store4(vh + r, cls, hh);
        store4(th + r, cls, tt);
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (r + k < len) {
                float mm = m[r + k], vv = v[r + k], hh = vh[r + k], tt = th[r + k];
                amsgrad_update(gb[k], mm, vv, hh, tt, hp);
                gbar[r + k] = gb[k];
                m[r + k] = mm;
                v[r + k] = vv;
                vh[r + k] = hh;
                th[r + k] = tt;
            }
        }
    }
}

cudaError_t launch_bs_sweep(compams_context* c, const float* grads) {
    dim3 grid((unsigned)c->tab.ntiles, (unsigned)c->n);
    BsBuffers b = c->bs;
    b.scales_prev = c->scales[c->scales_cur ^ 1];
    b.scales_cur = c->scales[c->scales_cur];
    bs_sweep_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, b, grads, c->e_is_x ? 1 : 0, c->segp);
    return cudaGetLastError();
}

cudaError_t launch_bs_scales(compams_context* c) {
    dim3 grid((unsigned)c->M, (unsigned)c->n);
    BsBuffers b = c->bs;
    b.scales_cur = c->scales[c->scales_cur];
    bs_scales_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, b);
    return cudaGetLastError();
}

cudaError_t launch_bs_apply(compams_context* c, float* theta) {
    BsBuffers b = c->bs;
    b.scales_cur = c->scales[c->scales_cur];
    bs_apply_kernel<<<(unsigned)c->tab.ntiles * kWarps, kThreads, 0, c->stream>>>(c->tab, b, theta, c->hp);
    return cudaGetLastError();
}

cudaError_t launch_bs_materialize(compams_context* c) {
    dim3 grid((unsigned)c->tab.ntiles, (unsigned)c->n);
    bs_materialize_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->E, c->scales[c->scales_cur]);
    return cudaGetLastError();
}

}  // namespace compams

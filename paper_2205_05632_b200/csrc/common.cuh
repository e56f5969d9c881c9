// Device helpers shared by the COMP-AMS kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace compams {

constexpr int kThreads = 256;          // threads per CTA of every tiled kernel
constexpr int kWarps = kThreads / 32;
constexpr int kTile = 8192;            // coordinates per tile: 8 warps x 8 iterations x 32 lanes x 4
constexpr int kWarpSpan = kTile / kWarps;  // 1024 consecutive coordinates per warp
constexpr int kIters = kWarpSpan / 128;    // 8 iterations of one float4 per lane

// One tile: kTile consecutive coordinates of one block (the last tile of a block may be shorter).
struct __align__(16) TileInfo {
    int64_t o;        // first coordinate of the block inside [0, d)
    int32_t len;      // block length d_b
    int32_t r0;       // first coordinate of the tile, relative to the block
    int32_t blk;      // block index b
    int32_t seg;      // index of the block among the tiled blocks
    int32_t tile0;    // first tile of the block
    int32_t ntile_b;  // number of tiles of the block
};

// One tiled block as the kernels see it (the Top-k fields are 0 for Block-Sign).
struct __align__(16) SegInfo {
    int64_t o;         // first coordinate of the block
    int64_t slot0;     // first message slot of the block inside a worker's row of K entries
    int64_t cand_off;  // first candidate slot of the block inside a worker's row of candidate slots
    int32_t len;       // block length d_b
    int32_t blk;       // block index b
    int32_t tile0;     // first tile
    int32_t ntile_b;   // number of tiles
    uint32_t kb;       // entries to keep
    uint32_t cap;      // candidate capacity (0: this block never uses the candidate path)
};

// The tiled blocks again, small enough to travel as a kernel argument: a CTA of a sweep finds its
// tile's block in the constant bank instead of waiting for a global-memory table before it can
// issue its first data load. nseg = 0 when there are too many blocks (the tile table is used).
constexpr int kParamSegs = 168;
struct SegParams {
    int32_t nseg;
    int32_t tile0[kParamSegs + 1];  // first tile of each tiled block, then the total
    int32_t len[kParamSegs];
    int32_t blk[kParamSegs];
    int32_t wofs[kParamSegs];  // Block-Sign: first sign word of the block within a worker's row of words
    int64_t o[kParamSegs];
};

// AMSGrad hyper-parameters as the fp32 numbers every kernel uses (Algorithm 1).
struct HyperParams {
    float lr, beta1, beta2, omb1, omb2, eps, nf;  // omb = 1 - beta (fp32), nf = (float)n
    float inv_nf;  // 1 / n when n is a power of two (then x * inv_nf == x / n bit for bit), else 0
};

// One AMSGrad coordinate update (Algorithm 2, the moment, maximum and parameter updates). Every operation is a separately
// rounded fp32 operation: no fused multiply-add, IEEE square root and division.
__device__ __forceinline__ void amsgrad_update(float g, float& m, float& v, float& vh, float& th,
                                               const HyperParams& hp) {
    m = __fadd_rn(__fmul_rn(hp.beta1, m), __fmul_rn(hp.omb1, g));
    v = __fadd_rn(__fmul_rn(hp.beta2, v), __fmul_rn(hp.omb2, __fmul_rn(g, g)));
    vh = fmaxf(vh, v);
    th = __fsub_rn(th, __fdiv_rn(__fmul_rn(hp.lr, m), __fsqrt_rn(__fadd_rn(vh, hp.eps))));
}

// gbar = (float)(sum over workers, accumulated in binary64) / (float)n  (Algorithm 2, the server's average).
// For n a power of two the division is a multiplication by the exactly representable 1 / n: both
// round the same real number once, so the bits agree (subnormal results included) and the
// multi-instruction IEEE division is saved.
__device__ __forceinline__ float mean_from_acc(double acc, const HyperParams& hp) {
    const float s = __double2float_rn(acc);
    return hp.inv_nf != 0.0f ? __fmul_rn(s, hp.inv_nf) : __fdiv_rn(s, hp.nf);
}

// Magnitude key: fp32 bits with the sign cleared; unsigned order == order of |x| for finite x.
__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// Alignment class of a float pointer: its address in floats modulo 4. Class 0 allows 128-bit
// accesses, class 2 64-bit ones, odd classes 32-bit ones. Rows of a packed [n, d] buffer start
// in different classes when d is not a multiple of 4.
__device__ __forceinline__ int align_class(const void* p) { return (int)((reinterpret_cast<uintptr_t>(p) >> 2) & 3u); }

// Read-only load of 4 consecutive floats at p, whose alignment class is cls. Deliberately NOT an
// evict-first load: when rows are not 128-byte aligned, neighbouring warps share cache lines, and
// an evict-first policy makes the second warp fetch the shared line again (measured: 3.9 TB/s
// against 6.7 TB/s for this access pattern).
__device__ __forceinline__ float4 load4_stream(const float* p, int cls) {
    float4 r;
    if (cls == 0) {
        r = __ldg(reinterpret_cast<const float4*>(p));
    } else if (cls == 2) {
        float2 a = __ldg(reinterpret_cast<const float2*>(p));
        float2 b = __ldg(reinterpret_cast<const float2*>(p + 2));
        r = make_float4(a.x, a.y, b.x, b.y);
    } else {
        r = make_float4(__ldg(p), __ldg(p + 1), __ldg(p + 2), __ldg(p + 3));
    }
    return r;
}

// Gradients may also arrive as bfloat16, passed as their 16-bit patterns: widening to fp32 is exact
// (the pattern shifted left by 16), so x = g + e is the same fp32 addition as with fp32 gradients
// of those values. The class of a bfloat16 pointer is its address in elements modulo 4: class 0
// allows one 64-bit access for 4 elements, class 2 two 32-bit ones, odd classes four 16-bit ones.
typedef uint16_t bf16_bits;
__device__ __forceinline__ int align_class(const bf16_bits* p) { return (int)((reinterpret_cast<uintptr_t>(p) >> 1) & 3u); }
__device__ __forceinline__ float widen(bf16_bits h) { return __uint_as_float((uint32_t)h << 16); }
__device__ __forceinline__ float load1_stream(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load1_stream(const bf16_bits* p) { return widen(__ldg(p)); }
__device__ __forceinline__ float4 load4_stream(const bf16_bits* p, int cls) {
    uint32_t lo, hi;
    if (cls == 0) {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
        lo = v.x;
        hi = v.y;
    } else if (cls == 2) {
        lo = __ldg(reinterpret_cast<const uint32_t*>(p));
        hi = __ldg(reinterpret_cast<const uint32_t*>(p + 2));
    } else {
        lo = (uint32_t)__ldg(p) | ((uint32_t)__ldg(p + 1) << 16);
        hi = (uint32_t)__ldg(p + 2) | ((uint32_t)__ldg(p + 3) << 16);
    }
    return make_float4(__uint_as_float(lo << 16), __uint_as_float(lo & 0xffff0000u), __uint_as_float(hi << 16),
                       __uint_as_float(hi & 0xffff0000u));
}

// Plain (cached) load of 4 consecutive floats.
__device__ __forceinline__ float4 load4(const float* p, int cls) {
    float4 r;
    if (cls == 0) {
        r = *reinterpret_cast<const float4*>(p);
    } else if (cls == 2) {
        float2 a = *reinterpret_cast<const float2*>(p);
        float2 b = *reinterpret_cast<const float2*>(p + 2);
        r = make_float4(a.x, a.y, b.x, b.y);
    } else {
        r = make_float4(p[0], p[1], p[2], p[3]);
    }
    return r;
}

__device__ __forceinline__ void store4(float* p, int cls, float4 v) {
    if (cls == 0) {
        *reinterpret_cast<float4*>(p) = v;
    } else if (cls == 2) {
        *reinterpret_cast<float2*>(p) = make_float2(v.x, v.y);
        *reinterpret_cast<float2*>(p + 2) = make_float2(v.z, v.w);
    } else {
        p[0] = v.x; p[1] = v.y; p[2] = v.z; p[3] = v.w;
    }
}

__device__ __forceinline__ float lane_elem(const float4& v, int k) {
    return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w;
}

// Tile record `tile` of a table, fetched with two 128-bit read-only loads.
__device__ __forceinline__ TileInfo load_tile(const TileInfo* tiles, int tile) {
    const int4* p = reinterpret_cast<const int4*>(tiles + tile);
    const int4 a = __ldg(p), b = __ldg(p + 1);
    TileInfo ti;
    ti.o = ((int64_t)(uint32_t)a.y << 32) | (uint32_t)a.x;
    ti.len = a.z;
    ti.r0 = a.w;
    ti.blk = b.x;
    ti.seg = b.y;
    ti.tile0 = b.z;
    ti.ntile_b = b.w;
    return ti;
}

// The same record from the kernel-argument copy of the block list (binary search over tile0).
__device__ __forceinline__ TileInfo find_tile(const SegParams& sp, int tile) {
    int lo = 0, hi = sp.nseg - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (sp.tile0[mid] <= tile) lo = mid; else hi = mid - 1;
    }
    TileInfo ti;
    ti.o = sp.o[lo];
    ti.len = sp.len[lo];
    ti.r0 = (tile - sp.tile0[lo]) * kTile;
    ti.blk = sp.blk[lo];
    ti.seg = lo;
    ti.tile0 = sp.tile0[lo];
    ti.ntile_b = sp.tile0[lo + 1] - sp.tile0[lo];
    return ti;
}

// Programmatic dependent launch: a kernel launched with launch_after() may start while the kernel
// before it on the stream is still draining. It may touch nothing that kernel (or any earlier one it
// has not been ordered after) writes until dependency_wait() has returned; what it reads before that
// - here: optimizer state that only the previous step wrote - overlaps the predecessor's tail.
// allow_dependents() in the predecessor lets the successor's CTAs in as soon as all of its own have
// started. Both are no-ops in a plainly launched kernel.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Inclusive scan of one unsigned value per thread across a CTA of kThreads threads.
// `scratch` holds NWARPS words (the CTA has NWARPS warps). Returns the inclusive prefix; *total receives the CTA sum.
template <int NWARPS = kWarps>
__device__ __forceinline__ uint32_t block_inclusive_scan(uint32_t x, uint32_t* scratch, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t s = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xffffffffu, s, o);
        if (lane >= o) s += y;
    }
    __syncthreads();  // scratch may still be read from an earlier call
    if (lane == 31) scratch[warp] = s;
    __syncthreads();
    uint32_t base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) {
        uint32_t c = scratch[w];
        if (w < warp) base += c;
        tot += c;
    }
    *total = tot;
    return s + base;
}

// Deterministic CTA sum of one double per thread (fixed shuffle tree, then warps in order).
// Result valid in thread 0. `scratch` holds one double per warp of the CTA (WARPS of them).
template <int WARPS = kWarps>
__device__ __forceinline__ double block_sum_double(double x, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    __syncthreads();
    if (lane == 0) scratch[warp] = x;
    __syncthreads();
    double s = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < WARPS; ++w) s += scratch[w];
    }
    return s;
}

}  // namespace compams

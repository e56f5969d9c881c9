// compams_blocksign_sweep_static: the Block-Sign sweep for callers that cannot allocate.
//
// Some callers run where device allocation is off the table: inside a framework's allocator
// callback, in a process whose memory was sized and handed out up front, or at a point of a
// serving loop where a cudaMalloc (which synchronises the device) would stall every other stream.
// The handle-based API allocates its state and scratch in compams_create; this entry point takes
// every input and output from the caller and keeps its only scratch - the per-tile partial sums
// of |x| and the per-row arrival counters - in one fixed array that lives in the library's device
// image. It calls no cudaMalloc / cudaFree and no allocating library routine.
//
// The array has a fixed size, so the problem size is capped (see the limits below); it is shared
// by every call in the process and keeps whatever the last call left in it, so the part that
// must start at zero is cleared at the start of each call, and two calls whose device work
// overlaps in time (different streams, or different host threads) race on it.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/compams.h"
#include "common.cuh"

namespace {

using namespace compams;

constexpr int64_t kStaticMaxRows = 1024;    // workers
constexpr int64_t kStaticMaxTiles = 65536;  // n * ceil(d / 8192), e.g. n = 16 with d up to 33.5 M
constexpr size_t kSumsBytes = (size_t)kStaticMaxTiles * sizeof(double);
constexpr size_t kScratchBytes = kSumsBytes + (size_t)kStaticMaxRows * sizeof(uint32_t);

// 516 KiB held by every GPU that loads the library, until the process exits.
// Layout: kStaticMaxTiles doubles (tile sums), then kStaticMaxRows arrival counters.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// In host code g_static_scratch is only a handle for the runtime, not a device address: the
// address a kernel can use comes from cudaGetSymbolAddress, once per device.
constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};

// X is read and then overwritten by the same thread: it is read with plain loads (the read-only data path
// is defined only for memory the kernel never writes) and carries no __restrict__.
__global__ void __launch_bounds__(kThreads) bs_sweep_static_kernel(const float* __restrict__ G, float* X,
                                                                   const float* __restrict__ scales_prev,
                                                                   float* __restrict__ scales_out,
                                                                   uint32_t* __restrict__ bits, int64_t d,
                                                                   int64_t words_per_row, int tiles_per_row,
                                                                   int deferred, double* __restrict__ tile_sum,
                                                                   uint32_t* __restrict__ arrivals) {
    __shared__ double red[kWarps];
    __shared__ int is_last;
    const int tile = blockIdx.x, i = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* g = G + (size_t)i * (size_t)d;
    float* x = X + (size_t)i * (size_t)d;
    const int cg = align_class(g), cx = align_class(x);
    const float sp = deferred ? scales_prev[i] : 0.0f;
    const int64_t rw = (int64_t)tile * kTile + (int64_t)warp * kWarpSpan;
    double acc = 0.0;
    uint32_t myword = 0;
    for (int it = 0; it < kIters; ++it) {
        const int64_t r = rw + it * 128 + lane * 4;
        float gv[4], xv[4];
        if (r + 3 < d) {
            float4 a = load4_stream(g + r, cg), b = load4(x + r, cx);
            gv[0] = a.x; gv[1] = a.y; gv[2] = a.z; gv[3] = a.w;
            xv[0] = b.x; xv[1] = b.y; xv[2] = b.z; xv[3] = b.w;
        } else {
            for (int k = 0; k < 4; ++k) {
                gv[k] = (r + k < d) ? __ldg(g + r + k) : 0.0f;
                xv[k] = (r + k < d) ? x[r + k] : 0.0f;
            }
        }
        uint32_t nib = 0;
        for (int k = 0; k < 4; ++k) {
            // the residual of the previous step, e = x_prev - sign(x_prev) * s_prev, then x = g + e
            const float e = deferred ? __fsub_rn(xv[k], copysignf(sp, xv[k])) : xv[k];
            xv[k] = __fadd_rn(gv[k], e);
            if (r + k < d) {
                acc += (double)fabsf(xv[k]);
                nib |= (__float_as_uint(xv[k]) >> 31) << k;
            }
        }
        if (r + 3 < d) {
            store4(x + r, cx, make_float4(xv[0], xv[1], xv[2], xv[3]));
        } else {
            for (int k = 0; k < 4; ++k)
                if (r + k < d) x[r + k] = xv[k];
        }
        uint32_t w = nib << ((lane & 7) * 4);
        w |= __shfl_xor_sync(0xffffffffu, w, 1);
        w |= __shfl_xor_sync(0xffffffffu, w, 2);
        w |= __shfl_xor_sync(0xffffffffu, w, 4);
        const uint32_t wv = __shfl_sync(0xffffffffu, w, (lane & 3) * 8);
        if ((lane >> 2) == it) myword = wv;
    }
    if (rw + (int64_t)lane * 32 < d) bits[(size_t)i * (size_t)words_per_row + (size_t)(rw >> 5) + lane] = myword;

    const double s = block_sum_double(acc, red);
    if (threadIdx.x == 0) {
        tile_sum[(size_t)i * tiles_per_row + tile] = s;
        __threadfence();
        is_last = (atomicAdd(&arrivals[i], 1u) == (uint32_t)(tiles_per_row - 1));
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double part = 0.0;
    for (int k = threadIdx.x; k < tiles_per_row; k += kThreads) part += __ldcg(tile_sum + (size_t)i * tiles_per_row + k);
    const double S = block_sum_double(part, red);
    if (threadIdx.x == 0) scales_out[i] = __double2float_rn(S / (double)d);
}

}  // namespace

extern "C" int compams_blocksign_sweep_static(const float* grads, float* x_state, const float* scales_prev,
                                              float* scales_out, uint32_t* sign_bits, int32_t n, int64_t d,
                                              int32_t deferred, void* cuda_stream) {
    if (!grads || !x_state || !scales_out || !sign_bits || (deferred && !scales_prev)) return COMPAMS_ERR_INVALID_ARG;
    if (n < 1 || d < 1 || d >= ((int64_t)1 << 31)) return COMPAMS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(grads) & 3u) || (reinterpret_cast<uintptr_t>(x_state) & 3u))
        return COMPAMS_ERR_INVALID_ARG;
    const int64_t tiles_per_row = (d + kTile - 1) / kTile;
    if (n > kStaticMaxRows || (int64_t)n * tiles_per_row > kStaticMaxTiles) return COMPAMS_ERR_TOO_LARGE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return COMPAMS_ERR_CUDA;
    if (!g_scratch_addr[dev]) {
        // one-time set-up for this device (it is the current one): resolve the array's device address
        unsigned char* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_static_scratch) != cudaSuccess || !p) return COMPAMS_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    unsigned char* base = g_scratch_addr[dev];
    double* tile_sum = reinterpret_cast<double*>(base);
    uint32_t* arrivals = reinterpret_cast<uint32_t*>(base + kSumsBytes);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the arrival counters must start at zero whatever an earlier call left behind
    if (cudaMemsetAsync(arrivals, 0, (size_t)n * sizeof(uint32_t), stream) != cudaSuccess) return COMPAMS_ERR_CUDA;
    dim3 grid((unsigned)tiles_per_row, (unsigned)n);
    bs_sweep_static_kernel<<<grid, kThreads, 0, stream>>>(grads, x_state, scales_prev, scales_out, sign_bits, d,
                                                          (d + 31) / 32, (int)tiles_per_row, deferred ? 1 : 0,
                                                          tile_sum, arrivals);
    return cudaGetLastError() == cudaSuccess ? COMPAMS_OK : COMPAMS_ERR_CUDA;
}

extern "C" int compams_blocksign_sweep_static_limits(int64_t* max_workers, int64_t* max_tiles) {
    if (!max_workers || !max_tiles) return COMPAMS_ERR_INVALID_ARG;
    *max_workers = kStaticMaxRows;
    *max_tiles = kStaticMaxTiles;
    return COMPAMS_OK;
}

// Random-k path of the COMP-AMS step: every (worker, block) keeps k_b coordinates drawn uniformly at random,
// whatever their values (Section 2.1 lists Random-k beside Top-k among the deterministic sparsifiers; with
// error feedback the dropped coordinates wait in e until they are drawn).
//
// The kept set of (step t, worker i, block b) is { pi(r) : r = 0 .. k_b - 1 }, pi a keyed pseudorandom
// permutation of the block's coordinates: a balanced Feistel network of six rounds over the smallest even
// number of bits that covers d_b, with cycle walking back into [0, d_b). The six 32-bit round keys are the
// halves of the first three words of one Philox4x64-10 block (Salmon, Moraes, Dror, Shaw, SC 2011) at counter
// (0, 0, b, i) under key (seed, t); the round function is the 32-bit finalizer of MurmurHash3 applied to
// (right half xor round key). Being the image of k_b distinct inputs under a bijection, the set has exactly k_b
// members and needs no selection pass: the sweep is the Top-k sweep without candidates (x = g + e written over
// E), then one thread per message slot computes its coordinate, fetches x there, zeroes it (the residual of a
// kept coordinate) and hands the pair to the server.
#include "context.h"
#include "scatter.cuh"

namespace compams {

struct RoundKeys {
    uint32_t k[6];
};

__device__ __forceinline__ RoundKeys randk_round_keys(uint64_t seed, uint64_t step, uint64_t worker, uint64_t block) {
    const uint64_t M0 = 0xD2E7470EE14C6C93ull, M1 = 0xCA5A826395121157ull;
    const uint64_t W0 = 0x9E3779B97F4A7C15ull, W1 = 0xBB67AE8584CAA73Bull;
    uint64_t c0 = 0, c1 = 0, c2 = block, c3 = worker, k0 = seed, k1 = step;
#pragma unroll 1
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += W0;
            k1 += W1;
        }
        const uint64_t hi0 = __umul64hi(M0, c0), lo0 = M0 * c0;
        const uint64_t hi1 = __umul64hi(M1, c2), lo1 = M1 * c2;
        const uint64_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0;
        c1 = lo1;
        c2 = n2;
        c3 = lo0;
    }
    RoundKeys out;
    out.k[0] = (uint32_t)c0;
    out.k[1] = (uint32_t)(c0 >> 32);
    out.k[2] = (uint32_t)c1;
    out.k[3] = (uint32_t)(c1 >> 32);
    out.k[4] = (uint32_t)c2;
    out.k[5] = (uint32_t)(c2 >> 32);
    return out;
}

__device__ __forceinline__ uint32_t fmix32(uint32_t h) {
    h ^= h >> 16;
    h *= 0x85ebca6bu;
    h ^= h >> 13;
    h *= 0xc2b2ae35u;
    h ^= h >> 16;
    return h;
}

// Image of r under the permutation of {0, ..., m - 1} with the given round keys; m < 2^32.
__device__ __forceinline__ uint32_t randk_permute(uint32_t m, uint32_t r, const uint32_t* keys) {
    int bits = 2;
    while (bits < 32 && (1u << bits) < m) bits += 2;
    const int w = bits >> 1;
    const uint32_t mask = (1u << w) - 1u;
    uint32_t k[6];
#pragma unroll
    for (int i = 0; i < 6; ++i) k[i] = keys[i];
    uint32_t x = r;
    do {
        uint32_t L = x >> w, R = x & mask;
#pragma unroll
        for (int round = 0; round < 6; ++round) {
            const uint32_t nR = L ^ (fmix32(R ^ k[round]) & mask);
            L = R;
            R = nR;
        }
        x = (L << w) | R;
    } while (x >= m);  // at most a few rounds on average: the domain is less than four times m
    return x;
}

// One thread per message slot of this handle's t.n workers (worker il of the handle is worker row0 + il of the
// job). The slots of one (worker, block) are consecutive, so within a CTA the thread holding a block's first slot
// (or thread 0, for a block begun in the CTA before) derives the round keys once and the others read them from
// shared memory.
__global__ void __launch_bounds__(kThreads) randk_emit_kernel(Tables t, TopkBuffers b, int32_t row0, uint64_t seed,
                                                              uint64_t step, int deliver) {
    __shared__ uint32_t keys[kThreads][6];
    const int tid = threadIdx.x;
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + tid;
    const bool valid = p < (int64_t)t.n * b.K;
    int64_t il = 0, q = 0, o = 0;
    int lo = 0;
    uint32_t len = 1, r = 0;
    if (valid) {
        il = p / b.K;
        q = p % b.K;  // slot within the worker's row; its block by bisection of the slot offsets
        int hi = t.M - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (__ldg(b.seg_off + mid) <= q) lo = mid; else hi = mid - 1;
        }
        o = __ldg(t.off + lo);
        len = (uint32_t)(__ldg(t.off + lo + 1) - o);
        r = (uint32_t)(q - __ldg(b.seg_off + lo));
        if (tid == 0 || r == 0) {
            const RoundKeys rk = randk_round_keys(seed, step, (uint64_t)(row0 + il), (uint64_t)lo);
#pragma unroll
            for (int i = 0; i < 6; ++i) keys[tid][i] = rk.k[i];
        }
    }
    __syncthreads();
    int32_t j = 0;
    uint32_t xbits = 0;
    if (valid) {
        const int leader = r < (uint32_t)tid ? tid - (int)r : 0;
        j = (int32_t)(o + randk_permute(len, r, keys[leader]));
        float* ex = b.E + (size_t)il * (size_t)t.d + (size_t)j;
        xbits = __float_as_uint(*ex);  // the sweep left x = g + e there
        *ex = 0.0f;                    // the residual update at a kept coordinate: e = x - x
        const size_t slot = (size_t)(row0 + il) * (size_t)b.K + (size_t)q;
        b.idx[slot] = j;
        b.val[slot] = __uint_as_float(xbits);
    }
    if (deliver) scatter_warp(b, valid, j, xbits);
}

cudaError_t launch_randk_emit(compams_context* c, bool deliver) {
    const int64_t count = (int64_t)c->n * c->K;
    const unsigned grid = (unsigned)((count + kThreads - 1) / kThreads);
    randk_emit_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk, c->row0, c->seed, c->iter, deliver ? 1 : 0);
    return counted(c, cudaGetLastError());
}

}  // namespace compams

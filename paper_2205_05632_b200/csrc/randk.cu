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

struct Drawn {
    bool valid;
    int32_t il;  // worker within the handle
    int64_t q;   // slot within the worker's message row
    int32_t j;   // the drawn coordinate
};

// A CTA covers kThreads consecutive message slots of one worker; every thread computes the coordinate of its
// slot. The slots of one block are consecutive, so the thread holding a block's first slot (or thread 0, for a
// block begun in the CTA before) derives the round keys once and the others read them from shared memory.
// Called by all threads of the CTA.
__device__ __forceinline__ Drawn randk_draw(const Tables& t, const TopkBuffers& b, int32_t row0, uint64_t seed,
                                            uint64_t step, uint32_t (*keys)[6]) {
    const uint32_t per_worker = (uint32_t)((b.K + kThreads - 1) / kThreads);
    const int tid = threadIdx.x;
    Drawn dr;
    dr.il = (int32_t)(blockIdx.x / per_worker);
    dr.q = (int64_t)(blockIdx.x % per_worker) * kThreads + tid;
    dr.valid = dr.q < b.K;
    dr.j = 0;
    int64_t o = 0;
    uint32_t len = 1, r = 0;
    if (dr.valid) {
        int lo = 0, hi = t.M - 1;  // the slot's block, by bisection of the slot offsets
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (__ldg(b.seg_off + mid) <= dr.q) lo = mid; else hi = mid - 1;
        }
        o = __ldg(t.off + lo);
        len = (uint32_t)(__ldg(t.off + lo + 1) - o);
        r = (uint32_t)(dr.q - __ldg(b.seg_off + lo));
        if (tid == 0 || r == 0) {
            const RoundKeys rk = randk_round_keys(seed, step, (uint64_t)(row0 + dr.il), (uint64_t)lo);
#pragma unroll
            for (int i = 0; i < 6; ++i) keys[tid][i] = rk.k[i];
        }
    }
    __syncthreads();
    if (dr.valid) {
        const int leader = r < (uint32_t)tid ? tid - (int)r : 0;
        dr.j = (int32_t)(o + randk_permute(len, r, keys[leader]));
    }
    return dr;
}

// Worker il keeps coordinate j in message slot q: x goes to the message, its residual is zero.
__device__ __forceinline__ uint32_t randk_take(const Tables& t, const TopkBuffers& b, int32_t row0, int32_t il, int64_t q,
                                               int32_t j) {
    // the sweep left x = g + e there; the residual of a kept coordinate is e = x - x = 0. One exchange at the L2
    // fetches the one and leaves the other (a load followed by a store to the same scattered word made this
    // kernel six times slower).
    uint32_t* ex = reinterpret_cast<uint32_t*>(b.E + (size_t)il * (size_t)t.d + (size_t)j);
    const uint32_t xbits = atomicExch(ex, 0u);
    const size_t slot = (size_t)(row0 + il) * (size_t)b.K + (size_t)q;
    b.idx[slot] = j;
    b.val[slot] = __uint_as_float(xbits);
    return xbits;
}

// One thread per message slot draws its coordinate and takes it.
__global__ void __launch_bounds__(kThreads) randk_emit_kernel(Tables t, TopkBuffers b, int32_t row0, uint64_t seed,
                                                              uint64_t step, int deliver) {
    __shared__ uint32_t keys[kThreads][6];
    const Drawn dr = randk_draw(t, b, row0, seed, step, keys);
    uint32_t xbits = 0;
    if (dr.valid) xbits = randk_take(t, b, row0, dr.il, dr.q, dr.j);
    if (deliver) scatter_warp(b, dr.valid, dr.j, xbits);
}

cudaError_t launch_randk_emit(compams_context* c, bool deliver) {
    const int64_t per_worker = (c->K + kThreads - 1) / kThreads;
    const unsigned grid = (unsigned)(per_worker * c->n);
    randk_emit_kernel<<<grid, kThreads, 0, c->stream>>>(c->tab, c->tk, c->row0, c->seed, c->iter, deliver ? 1 : 0);
    return counted(c, cudaGetLastError());
}

}  // namespace compams

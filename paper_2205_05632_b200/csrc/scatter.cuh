// Delivery of kept (coordinate, value) pairs to the server: shared by the Top-k and the Random-k kernels.
#pragma once

#include "context.h"

namespace compams {

// A kept (coordinate, value) pair reaches the server: it joins the bucket of its coordinate range at position
// `pos` or, when the bucket is full, the binary64 accumulator.
__device__ __forceinline__ void deliver_pair(const TopkBuffers& b, uint32_t T, uint32_t pos, int32_t j, uint32_t xbits) {
    if (pos < (uint32_t)b.bucket_cap) {
        b.bucket[(size_t)T * (size_t)b.bucket_cap + pos] = make_uint2((uint32_t)j % (uint32_t)kBucketSpan, xbits);
    } else {  // a coordinate range kept by far more entries than average: binary64 atomics instead
        atomicAdd(b.acc + j, (double)__uint_as_float(xbits));
        b.bdirty[T] = 1u;
    }
}

// One pair per thread, the whole warp together: the lanes whose pairs fall into the same bucket get their
// slots with one atomic.
__device__ __forceinline__ void scatter_warp(const TopkBuffers& b, bool valid, int32_t j, uint32_t xbits) {
    const uint32_t T = valid ? (uint32_t)j / (uint32_t)kBucketSpan : 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const unsigned peers = __match_any_sync(0xffffffffu, T);
    uint32_t base = 0;
    const int leader = __ffs(peers) - 1;
    if (valid && lane == leader) base = atomicAdd(b.bcount + T, (uint32_t)__popc(peers));
    base = __shfl_sync(0xffffffffu, base, leader);
    if (!valid) return;
    deliver_pair(b, T, base + (uint32_t)__popc(peers & ((1u << lane) - 1u)), j, xbits);
}

}  // namespace compams

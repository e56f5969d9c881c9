// Uncompressed mode (k = d, q = 0 in Assumption 1) and the stand-alone AMSGrad update.
//
// dense_mean_amsgrad: gbar = mean over workers of g_i (Algorithm 2, the server's average with C = identity,
// so e stays 0), fused with the AMSGrad update (the moment, maximum and parameter updates). One pass over G [n, d] and the
// four state vectors: (4n + 32) bytes per coordinate, plus 4 for gbar while the caller has asked for it to be recorded
// (a null gbar: not written).
//
// amsgrad_bucket: the server update of the Top-k path. The scatter kernel has grouped the kept
// (coordinate, value) entries of all workers by coordinate range; one CTA per range sums them in
// binary64 in shared memory, rounds, divides by n and applies the moment, maximum and parameter updates.
#include "context.h"

namespace compams {

// One CTA per 1024 coordinates: one float4 group per thread, the workers' rows read one after another.
// Two builds: eight CTAs per SM (32 registers, a few spilled words) beat six (40 registers) once there are
// rows enough to wait for - 0.187 against 0.200 ms on ResNet-18 shapes, n = 16 - and lose to them when the
// optimizer state is most of the traffic (d = 2^26: n = 1 0.427 against 0.395 ms, n = 4 0.531 against 0.522 ms,
// n = 8 0.677 against 0.707 ms). Requesting the state ahead of the rows costs registers and is slower.
template <typename GT, int CTAS_PER_SM>
__global__ void __launch_bounds__(kThreads, CTAS_PER_SM) dense_mean_amsgrad_kernel(int32_t n, int64_t d, const GT* __restrict__ G,
                                                                         float* __restrict__ gbar, float* __restrict__ m,
                                                                         float* __restrict__ v, float* __restrict__ vhat,
                                                                         float* __restrict__ theta, HyperParams hp) {
    const int64_t groups = d >> 2;
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q < groups) {
        const int64_t j = q << 2;
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
        const GT* p = G + j;
#pragma unroll 4
        for (int32_t i = 0; i < n; ++i) {
            const GT* pi = p + (size_t)i * (size_t)d;
            float4 g = load4_stream(pi, align_class(pi));
            a0 += (double)g.x;
            a1 += (double)g.y;
            a2 += (double)g.z;
            a3 += (double)g.w;
        }
        float4 gb = make_float4(mean_from_acc(a0, hp), mean_from_acc(a1, hp), mean_from_acc(a2, hp),
                                mean_from_acc(a3, hp));
        float4 mm = *reinterpret_cast<const float4*>(m + j);
        float4 vv = *reinterpret_cast<const float4*>(v + j);
        float4 vh = *reinterpret_cast<const float4*>(vhat + j);
        float4 th = *reinterpret_cast<const float4*>(theta + j);
        amsgrad_update(gb.x, mm.x, vv.x, vh.x, th.x, hp);
        amsgrad_update(gb.y, mm.y, vv.y, vh.y, th.y, hp);
        amsgrad_update(gb.z, mm.z, vv.z, vh.z, th.z, hp);
        amsgrad_update(gb.w, mm.w, vv.w, vh.w, th.w, hp);
        if (gbar) *reinterpret_cast<float4*>(gbar + j) = gb;
        *reinterpret_cast<float4*>(m + j) = mm;
        *reinterpret_cast<float4*>(v + j) = vv;
        *reinterpret_cast<float4*>(vhat + j) = vh;
        *reinterpret_cast<float4*>(theta + j) = th;
    }
    // the last d % 4 coordinates
    if (blockIdx.x == 0 && threadIdx.x < (d & 3)) {
        const int64_t j = (groups << 2) + threadIdx.x;
        double a = 0.0;
        for (int32_t i = 0; i < n; ++i) a += (double)load1_stream(G + (size_t)i * (size_t)d + (size_t)j);
        float gb = mean_from_acc(a, hp);
        float mm = m[j], vv = v[j], vh = vhat[j], th = theta[j];
        amsgrad_update(gb, mm, vv, vh, th, hp);
        if (gbar) gbar[j] = gb;
        m[j] = mm;
        v[j] = vv;
        vhat[j] = vh;
        theta[j] = th;
    }
}

// Server update of the Top-k path, one CTA per bucket of kBucketSpan coordinates: the bucket's kept
// entries (all workers) are summed in binary64 in shared memory, in the order the atomics arrive, then
// gbar = (float)sum / n and Algorithm 2, the moment, maximum and parameter updates. The binary64 sum of the
// fp32 terms of one coordinate is exact - and then the order cannot matter - as long as 24 + (the spread of
// the terms' exponents) + log2 n <= 53, i.e. the magnitudes kept at one coordinate lie within 2^24 of one
// another at n = 32. Wider spreads (one worker keeps 1e-12 where another keeps 1) can round differently from
// run to run in the last bit of gbar, which stays inside the tolerance the step is specified to. Entries
// that did not fit their bucket were added to acc[] by the scatter kernel and are folded in (and acc
// cleared) here.
template <bool RECORD>
__global__ void __launch_bounds__(kThreads, 5) amsgrad_bucket_kernel(int64_t d, TopkBuffers b, float* __restrict__ theta,
                                                                     HyperParams hp) {
    static_assert(kBucketSpan == 4 * kThreads, "one float4 group per thread");
    __shared__ double sacc[kBucketSpan];
    const uint32_t T = blockIdx.x;
    const int loc = (int)threadIdx.x * 4;
    const int64_t j = (int64_t)T * kBucketSpan + loc;
    const bool full = j + 3 < d;
    // the state of this thread's four coordinates is requested first, so that it is in flight
    // while the bucket's entries are summed
    float4 mm = make_float4(0.f, 0.f, 0.f, 0.f), vv = mm, vh = mm, th = mm;
    if (full) {
        mm = *reinterpret_cast<const float4*>(b.m + j);
        vv = *reinterpret_cast<const float4*>(b.v + j);
        vh = *reinterpret_cast<const float4*>(b.vhat + j);
        th = *reinterpret_cast<const float4*>(theta + j);
    }
    dependency_wait();  // everything below is this step's: the scatter kernel's buckets
    // the bucket's first round of entries is requested before its fill count is known (the slots
    // exist whatever they hold; an entry is used only if the count covers it)
    const uint2* ent = b.bucket + (size_t)T * (size_t)b.bucket_cap;
    uint2 first = make_uint2(0u, 0u);
    if (threadIdx.x < (uint32_t)b.bucket_cap) first = ent[threadIdx.x];
    const uint32_t appended = b.bcount[T];
    const uint32_t cnt = appended < (uint32_t)b.bucket_cap ? appended : (uint32_t)b.bucket_cap;
    const bool dirty = b.bdirty[T] != 0u;
    sacc[loc] = 0.0;
    sacc[loc + 1] = 0.0;
    sacc[loc + 2] = 0.0;
    sacc[loc + 3] = 0.0;
    __syncthreads();
    if (threadIdx.x < cnt) atomicAdd(&sacc[first.x], (double)__uint_as_float(first.y));
    for (uint32_t e = threadIdx.x + kThreads; e < cnt; e += kThreads) {
        const uint2 cv = ent[e];
        atomicAdd(&sacc[cv.x], (double)__uint_as_float(cv.y));
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        b.bcount[T] = 0u;
        b.bdirty[T] = 0u;
    }
    if (j >= d) return;
    double a[4] = {sacc[loc], sacc[loc + 1], sacc[loc + 2], sacc[loc + 3]};
    if (full) {
        if (dirty) {
            const double2 x01 = *reinterpret_cast<const double2*>(b.acc + j);
            const double2 x23 = *reinterpret_cast<const double2*>(b.acc + j + 2);
            a[0] += x01.x; a[1] += x01.y; a[2] += x23.x; a[3] += x23.y;
            *reinterpret_cast<double2*>(b.acc + j) = make_double2(0.0, 0.0);
            *reinterpret_cast<double2*>(b.acc + j + 2) = make_double2(0.0, 0.0);
        }
        float4 gb = make_float4(mean_from_acc(a[0], hp), mean_from_acc(a[1], hp), mean_from_acc(a[2], hp),
                                mean_from_acc(a[3], hp));
        amsgrad_update(gb.x, mm.x, vv.x, vh.x, th.x, hp);
        amsgrad_update(gb.y, mm.y, vv.y, vh.y, th.y, hp);
        amsgrad_update(gb.z, mm.z, vv.z, vh.z, th.z, hp);
        amsgrad_update(gb.w, mm.w, vv.w, vh.w, th.w, hp);
        if constexpr (RECORD) *reinterpret_cast<float4*>(b.gbar + j) = gb;
        *reinterpret_cast<float4*>(b.m + j) = mm;
        *reinterpret_cast<float4*>(b.v + j) = vv;
        *reinterpret_cast<float4*>(b.vhat + j) = vh;
        *reinterpret_cast<float4*>(theta + j) = th;
    } else {
        for (int k = 0; k < 4 && j + k < d; ++k) {
            double ak = a[k];
            if (dirty) {
                ak += b.acc[j + k];
                b.acc[j + k] = 0.0;
            }
            const float gb = mean_from_acc(ak, hp);
            float m1 = b.m[j + k], v1 = b.v[j + k], h1 = b.vhat[j + k], t1 = theta[j + k];
            amsgrad_update(gb, m1, v1, h1, t1, hp);
            if constexpr (RECORD) b.gbar[j + k] = gb;
            b.m[j + k] = m1;
            b.v[j + k] = v1;
            b.vhat[j + k] = h1;
            theta[j + k] = t1;
        }
    }
}

// gbar stored or not: a null pointer here (as a template parameter this kernel ran 4 % slower), a template
// parameter in amsgrad_bucket and bs_apply (where the run-time branch around the store cost up to a tenth).
template <typename GT>
static void launch_dense_typed(compams_context* c, const GT* g, float* theta, int grid) {
    float* gbar = c->record_gbar ? c->gbar : nullptr;
    if (c->n >= 6)
        dense_mean_amsgrad_kernel<GT, 8><<<grid, kThreads, 0, c->stream>>>(c->n, c->d, g, gbar, c->m, c->v, c->vhat, theta, c->hp);
    else
        dense_mean_amsgrad_kernel<GT, 6><<<grid, kThreads, 0, c->stream>>>(c->n, c->d, g, gbar, c->m, c->v, c->vhat, theta, c->hp);
}

cudaError_t launch_dense_mean_amsgrad(compams_context* c, const void* grads, float* theta) {
    int64_t groups = c->d >> 2;
    int grid = (int)((groups + kThreads - 1) / kThreads);
    if (grid < 1) grid = 1;
    if (c->grad_bf16) launch_dense_typed(c, (const bf16_bits*)grads, theta, grid);
    else launch_dense_typed(c, (const float*)grads, theta, grid);
    return counted(c, cudaGetLastError());
}

cudaError_t launch_amsgrad(compams_context* c, float* theta) {
    const dim3 grid((unsigned)c->tk.nbucket);
    return counted(c, c->tk.gbar ? launch_after(amsgrad_bucket_kernel<true>, grid, dim3(kThreads), c->stream, c->d, c->tk, theta, c->hp)
                                 : launch_after(amsgrad_bucket_kernel<false>, grid, dim3(kThreads), c->stream, c->d, c->tk, theta, c->hp));
}

}  // namespace compams

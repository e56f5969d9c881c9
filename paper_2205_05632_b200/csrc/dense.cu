// Uncompressed mode (k = d, q = 0 in Assumption 1) and the stand-alone AMSGrad update.
//
// dense_mean_amsgrad: gbar = mean over workers of g_i (Algorithm 2, line 12 with C = identity,
// so e stays 0), fused with the AMSGrad update (lines 13-16). One pass over G [n, d] and the
// four state vectors: (4n + 32) bytes per coordinate plus 4 for gbar.
//
// amsgrad_from_acc: the server update of the Top-k path. The scatter kernel has accumulated
// sum_i g~_i in a binary64 buffer; this kernel rounds it, divides by n, clears the buffer for
// the next step and applies lines 13-16.
#include "context.h"

namespace compams {

// One CTA per 1024 coordinates: one float4 group per thread, the workers' rows read one after another.
__global__ void __launch_bounds__(kThreads, 6) dense_mean_amsgrad_kernel(int32_t n, int64_t d, const float* __restrict__ G,
                                                                         float* __restrict__ gbar, float* __restrict__ m,
                                                                         float* __restrict__ v, float* __restrict__ vhat,
                                                                         float* __restrict__ theta, HyperParams hp) {
    const int64_t groups = d >> 2;
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q < groups) {
        const int64_t j = q << 2;
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
        const float* p = G + j;
#pragma unroll 4
        for (int32_t i = 0; i < n; ++i) {
            const float* pi = p + (size_t)i * (size_t)d;
            float4 g = load4_stream(pi, align_class(pi));
            a0 += (double)g.x;
            a1 += (double)g.y;
            a2 += (double)g.z;
            a3 += (double)g.w;
        }
        float4 gb = make_float4(mean_from_acc(a0, hp.nf), mean_from_acc(a1, hp.nf), mean_from_acc(a2, hp.nf),
                                mean_from_acc(a3, hp.nf));
        float4 mm = *reinterpret_cast<const float4*>(m + j);
        float4 vv = *reinterpret_cast<const float4*>(v + j);
        float4 vh = *reinterpret_cast<const float4*>(vhat + j);
        float4 th = *reinterpret_cast<const float4*>(theta + j);
        amsgrad_update(gb.x, mm.x, vv.x, vh.x, th.x, hp);
        amsgrad_update(gb.y, mm.y, vv.y, vh.y, th.y, hp);
        amsgrad_update(gb.z, mm.z, vv.z, vh.z, th.z, hp);
        amsgrad_update(gb.w, mm.w, vv.w, vh.w, th.w, hp);
        *reinterpret_cast<float4*>(gbar + j) = gb;
        *reinterpret_cast<float4*>(m + j) = mm;
        *reinterpret_cast<float4*>(v + j) = vv;
        *reinterpret_cast<float4*>(vhat + j) = vh;
        *reinterpret_cast<float4*>(theta + j) = th;
    }
    // the last d % 4 coordinates
    if (blockIdx.x == 0 && threadIdx.x < (d & 3)) {
        const int64_t j = (groups << 2) + threadIdx.x;
        double a = 0.0;
        for (int32_t i = 0; i < n; ++i) a += (double)G[(size_t)i * (size_t)d + (size_t)j];
        float gb = mean_from_acc(a, hp.nf);
        float mm = m[j], vv = v[j], vh = vhat[j], th = theta[j];
        amsgrad_update(gb, mm, vv, vh, th, hp);
        gbar[j] = gb;
        m[j] = mm;
        v[j] = vv;
        vhat[j] = vh;
        theta[j] = th;
    }
}

// One float4 group per thread.
__global__ void __launch_bounds__(kThreads, 6) amsgrad_from_acc_kernel(int64_t d, double* __restrict__ acc,
                                                                       float* __restrict__ gbar, float* __restrict__ m,
                                                                       float* __restrict__ v, float* __restrict__ vhat,
                                                                       float* __restrict__ theta, HyperParams hp) {
    const int64_t groups = d >> 2;
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q < groups) {
        const int64_t j = q << 2;
        double2 a01 = *reinterpret_cast<const double2*>(acc + j);
        double2 a23 = *reinterpret_cast<const double2*>(acc + j + 2);
        float4 mm = *reinterpret_cast<const float4*>(m + j);
        float4 vv = *reinterpret_cast<const float4*>(v + j);
        float4 vh = *reinterpret_cast<const float4*>(vhat + j);
        float4 th = *reinterpret_cast<const float4*>(theta + j);
        float4 gb = make_float4(mean_from_acc(a01.x, hp.nf), mean_from_acc(a01.y, hp.nf), mean_from_acc(a23.x, hp.nf),
                                mean_from_acc(a23.y, hp.nf));
        amsgrad_update(gb.x, mm.x, vv.x, vh.x, th.x, hp);
        amsgrad_update(gb.y, mm.y, vv.y, vh.y, th.y, hp);
        amsgrad_update(gb.z, mm.z, vv.z, vh.z, th.z, hp);
        amsgrad_update(gb.w, mm.w, vv.w, vh.w, th.w, hp);
        *reinterpret_cast<double2*>(acc + j) = make_double2(0.0, 0.0);
        *reinterpret_cast<double2*>(acc + j + 2) = make_double2(0.0, 0.0);
        *reinterpret_cast<float4*>(gbar + j) = gb;
        *reinterpret_cast<float4*>(m + j) = mm;
        *reinterpret_cast<float4*>(v + j) = vv;
        *reinterpret_cast<float4*>(vhat + j) = vh;
        *reinterpret_cast<float4*>(theta + j) = th;
    }
    if (blockIdx.x == 0 && threadIdx.x < (d & 3)) {
        const int64_t j = (groups << 2) + threadIdx.x;
        float gb = mean_from_acc(acc[j], hp.nf);
        acc[j] = 0.0;
        float mm = m[j], vv = v[j], vh = vhat[j], th = theta[j];
        amsgrad_update(gb, mm, vv, vh, th, hp);
        gbar[j] = gb;
        m[j] = mm;
        v[j] = vv;
        vhat[j] = vh;
        theta[j] = th;
    }
}

cudaError_t launch_dense_mean_amsgrad(compams_context* c, const float* grads, float* theta) {
    int64_t groups = c->d >> 2;
    int grid = (int)((groups + kThreads - 1) / kThreads);
    if (grid < 1) grid = 1;
    dense_mean_amsgrad_kernel<<<grid, kThreads, 0, c->stream>>>(c->n, c->d, grads, c->gbar, c->m, c->v, c->vhat, theta,
                                                                c->hp);
    return cudaGetLastError();
}

cudaError_t launch_amsgrad(compams_context* c, float* theta) {
    int64_t groups = c->d >> 2;
    int grid = (int)((groups + kThreads - 1) / kThreads);
    if (grid < 1) grid = 1;
    amsgrad_from_acc_kernel<<<grid, kThreads, 0, c->stream>>>(c->d, c->tk.acc, c->gbar, c->m, c->v, c->vhat, theta,
                                                              c->hp);
    return cudaGetLastError();
}

}  // namespace compams

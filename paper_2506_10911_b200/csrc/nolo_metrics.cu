// Replica divergence: how far the W workers' slow weights have drifted apart (the quantity of
// Fig. 3b: the standard deviation of the model weights across the data-parallel replicas).
//
// For every parameter p the population variance of phi[0..W-1][p] across the workers is computed
// with Welford's update in float32 (stable when the replicas are close, as they are), and the
// per-parameter standard deviation and variance are summed over all parameters in float64: first
// inside each CTA, then over the CTAs by a second kernel, both in a fixed order, so the result is
// reproducible.  A read-only pass: 4 bytes per worker-parameter.
#include "nolo_internal.h"

namespace nolo {

namespace {

constexpr int kThreads = 256;
constexpr int kItems = 4;     // quads per thread
constexpr int kUnroll = 4;    // worker rows in flight per thread

struct Welford4 {
    float4 mean, m2;
    __device__ __forceinline__ void init() {
        mean = make_float4(0.f, 0.f, 0.f, 0.f);
        m2 = mean;
    }
    __device__ __forceinline__ void push(float4 x, float inv_k) {
        float d;
        d = x.x - mean.x; mean.x += d * inv_k; m2.x += d * (x.x - mean.x);
        d = x.y - mean.y; mean.y += d * inv_k; m2.y += d * (x.y - mean.y);
        d = x.z - mean.z; mean.z += d * inv_k; m2.z += d * (x.z - mean.z);
        d = x.w - mean.w; mean.w += d * inv_k; m2.w += d * (x.w - mean.w);
    }
};

__global__ void __launch_bounds__(kThreads)
divergence_partial_kernel(const float* __restrict__ phi, int W, int64_t stride, int64_t P,
                          double2* __restrict__ partial) {
    const int64_t full_quads = P >> 2;
    const int64_t q0 = (int64_t)blockIdx.x * (kThreads * kItems) + threadIdx.x;
    const float inv_W = 1.0f / (float)W;
    double sum_std = 0.0, sum_var = 0.0;

    Welford4 acc[kItems];
#pragma unroll
    for (int it = 0; it < kItems; ++it) acc[it].init();
    bool ok[kItems];
#pragma unroll
    for (int it = 0; it < kItems; ++it) ok[it] = q0 + (int64_t)it * kThreads < full_quads;
#pragma unroll kUnroll
    for (int w = 0; w < W; ++w) {
        const float4* row = reinterpret_cast<const float4*>(phi + (int64_t)w * stride);
        const float inv_k = __frcp_rn((float)(w + 1));
        float4 x[kItems];
#pragma unroll
        for (int it = 0; it < kItems; ++it)
            if (ok[it]) x[it] = __ldcs(row + q0 + (int64_t)it * kThreads);
#pragma unroll
        for (int it = 0; it < kItems; ++it)
            if (ok[it]) acc[it].push(x[it], inv_k);
    }
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
        if (!ok[it]) continue;
        const float4 v = make_float4(acc[it].m2.x * inv_W, acc[it].m2.y * inv_W, acc[it].m2.z * inv_W,
                                     acc[it].m2.w * inv_W);
        sum_var += (double)v.x + (double)v.y + (double)v.z + (double)v.w;
        sum_std += (double)sqrtf(v.x) + (double)sqrtf(v.y) + (double)sqrtf(v.z) + (double)sqrtf(v.w);
    }
    // ragged tail (P mod 4 columns): one thread of the last CTA
    if ((P & 3) && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
        for (int64_t c = P & ~int64_t(3); c < P; ++c) {
            float mean = 0.f, m2 = 0.f;
            for (int w = 0; w < W; ++w) {
                const float x = phi[(int64_t)w * stride + c];
                const float d = x - mean;
                mean += d * __frcp_rn((float)(w + 1));
                m2 += d * (x - mean);
            }
            const float v = m2 * inv_W;
            sum_var += (double)v;
            sum_std += (double)sqrtf(v);
        }
    }
    // CTA reduction in a fixed order: lanes by shuffle tree, then warps in order
    __shared__ double2 warp_part[kThreads / 32];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        sum_std += __shfl_down_sync(0xffffffffu, sum_std, off);
        sum_var += __shfl_down_sync(0xffffffffu, sum_var, off);
    }
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = make_double2(sum_std, sum_var);
    __syncthreads();
    if (threadIdx.x == 0) {
        double2 t = warp_part[0];
        for (int w = 1; w < kThreads / 32; ++w) { t.x += warp_part[w].x; t.y += warp_part[w].y; }
        partial[blockIdx.x] = t;
    }
}

// One CTA adds the per-CTA partial sums: each thread a strided slice, then a fixed-order tree.
__global__ void __launch_bounds__(1024)
divergence_final_kernel(const double2* __restrict__ partial, int64_t count, double inv_P,
                        double* __restrict__ out) {
    __shared__ double2 sm[1024];
    double2 t = make_double2(0.0, 0.0);
    for (int64_t i = threadIdx.x; i < count; i += 1024) { t.x += partial[i].x; t.y += partial[i].y; }
    sm[threadIdx.x] = t;
    __syncthreads();
    for (int s = 512; s > 0; s >>= 1) {
        if (threadIdx.x < s) { sm[threadIdx.x].x += sm[threadIdx.x + s].x; sm[threadIdx.x].y += sm[threadIdx.x + s].y; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        out[0] = sm[0].x * inv_P;            // mean over parameters of the across-worker std
        out[1] = sqrt(sm[0].y * inv_P);      // root of the mean across-worker variance
    }
}

}  // namespace

int64_t divergence_partials(int64_t P) {
    const int64_t quads = (P + 3) >> 2;
    const int64_t per_cta = (int64_t)kThreads * kItems;
    return (quads + per_cta - 1) / per_cta;
}

cudaError_t launch_divergence(const float* phi, int W, int64_t stride, int64_t P, void* partials,
                              double* out2, cudaStream_t stream) {
    const int64_t ctas = divergence_partials(P);
    if (ctas > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    divergence_partial_kernel<<<(unsigned)ctas, kThreads, 0, stream>>>(phi, W, stride, P,
                                                                       static_cast<double2*>(partials));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    divergence_final_kernel<<<1, 1024, 0, stream>>>(static_cast<const double2*>(partials), ctas,
                                                    1.0 / (double)P, out2);
    return cudaGetLastError();
}

}  // namespace nolo

// Fused NoLoCo outer step (Section 3.2, Eq. 1-3) for W workers resident in one GPU's memory.
//
// Work decomposition: one CTA owns one subgroup x one tile of parameters.  Every member's
// phi / theta / delta element is loaded from HBM exactly once (128-bit coalesced, streaming
// cache policy) and every output element stored exactly once; the pseudo-gradients, their sum
// and the subgroup mean of phi exist only in registers.  The path is bandwidth bound
// (about 10 flops per 20-24 bytes), so there is no tensor-core work here.
//
//   Delta_j  = phi_j - theta_j                                            (Eq. 1)
//   delta_i' = alpha*delta_i - (beta/n) sum_j Delta_j - gamma*(phi_i - (1/n) sum_j phi_j)   (Eq. 2)
//   phi_i'   = phi_i + delta_i'                                           (Eq. 3)
//   theta_i' = phi_i'   (start of the next inner phase)
#include "nolo_internal.h"

#include <cuda_bf16.h>

namespace nolo {

namespace {

constexpr int kThreads = 256;

struct KArgs {
    float* phi;
    void* theta;
    float* delta;
    const int32_t* perm;
    int64_t stride;
    int64_t P;
    int n;
    float alpha, beta_over_n, gamma, inv_n;
};

// ---- theta access: 4 consecutive parameters as float4, fp32 or bf16 storage -------------

__device__ __forceinline__ float4 load_theta4(const float* row, int64_t q) {
    return __ldcs(reinterpret_cast<const float4*>(row) + q);
}
__device__ __forceinline__ float4 load_theta4(const __nv_bfloat16* row, int64_t q) {
    const uint2 v = __ldcs(reinterpret_cast<const uint2*>(row) + q);
    float4 r;
    r.x = __uint_as_float(v.x << 16);
    r.y = __uint_as_float(v.x & 0xffff0000u);
    r.z = __uint_as_float(v.y << 16);
    r.w = __uint_as_float(v.y & 0xffff0000u);
    return r;
}
__device__ __forceinline__ void store_theta4(float* row, int64_t q, float4 v) {
    __stcs(reinterpret_cast<float4*>(row) + q, v);
}
__device__ __forceinline__ void store_theta4(__nv_bfloat16* row, int64_t q, float4 v) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);   // round to nearest even
    const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    __stcs(reinterpret_cast<uint2*>(row) + q, u);
}
__device__ __forceinline__ float load_theta1(const float* row, int64_t c) { return row[c]; }
__device__ __forceinline__ float load_theta1(const __nv_bfloat16* row, int64_t c) {
    return __bfloat162float(row[c]);
}
__device__ __forceinline__ void store_theta1(float* row, int64_t c, float v) { row[c] = v; }
__device__ __forceinline__ void store_theta1(__nv_bfloat16* row, int64_t c, float v) {
    row[c] = __float2bfloat16_rn(v);
}

__device__ __forceinline__ float update1(float phi, float delta, float sum_Delta, float mean_phi,
                                         const KArgs& a, float* delta_out) {
    const float d = a.alpha * delta - a.beta_over_n * sum_Delta - a.gamma * (phi - mean_phi);
    *delta_out = d;
    return phi + d;
}

// Columns P - (P % 4) .. P-1 of one subgroup, element by element (rows are only guaranteed to be
// padded to a multiple of 8, and padding must not be written).
template <typename ThetaT>
__device__ void scalar_tail(const KArgs& a, int g) {
    const int n = a.n;
    for (int64_t c = a.P & ~int64_t(3); c < a.P; ++c) {
        float sD = 0.f, sP = 0.f;
        for (int j = 0; j < n; ++j) {
            const int64_t row = (int64_t)a.perm[g * n + j] * a.stride;
            const float p = a.phi[row + c];
            sD += p - load_theta1(static_cast<const ThetaT*>(a.theta) + row, c);
            sP += p;
        }
        const float mP = sP * a.inv_n;
        for (int j = 0; j < n; ++j) {
            const int64_t row = (int64_t)a.perm[g * n + j] * a.stride;
            float d;
            const float p = update1(a.phi[row + c], a.delta[row + c], sD, mP, a, &d);
            a.phi[row + c] = p;
            a.delta[row + c] = d;
            store_theta1(static_cast<ThetaT*>(a.theta) + row, c, p);
        }
    }
}

// ---- register-resident path: subgroup size N known at compile time ----------------------
//
// Each thread handles ITEMS quads (4 consecutive parameters) of the tile, 256 quads apart, for all
// N members: phi_j stays in registers between the reduction and the update, so nothing is read
// twice.  All loads of a thread are issued before the first use to keep many bytes in flight.
template <int N, typename ThetaT, int ITEMS>
__global__ void __launch_bounds__(kThreads)
outer_step_reg_kernel(const KArgs a) {
    const int g = blockIdx.y;
    const int64_t full_quads = a.P >> 2;
    const int64_t q0 = (int64_t)blockIdx.x * (kThreads * ITEMS) + threadIdx.x;

    int row[N];
#pragma unroll
    for (int j = 0; j < N; ++j) row[j] = __ldg(a.perm + g * N + j);
    auto phi_row = [&](int j) { return a.phi + (int64_t)row[j] * a.stride; };
    auto delta_row = [&](int j) { return a.delta + (int64_t)row[j] * a.stride; };
    auto theta_row = [&](int j) { return static_cast<ThetaT*>(a.theta) + (int64_t)row[j] * a.stride; };

    float4 phi[ITEMS][N], dlt[ITEMS][N], the[ITEMS][N];
    bool ok[ITEMS];
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const int64_t q = q0 + (int64_t)it * kThreads;
        ok[it] = q < full_quads;
        if (ok[it]) {
#pragma unroll
            for (int j = 0; j < N; ++j) {
                phi[it][j] = __ldcs(reinterpret_cast<const float4*>(phi_row(j)) + q);
                the[it][j] = load_theta4(theta_row(j), q);
            }
#pragma unroll
            for (int j = 0; j < N; ++j)
                dlt[it][j] = __ldcs(reinterpret_cast<const float4*>(delta_row(j)) + q);
        }
    }
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        if (!ok[it]) continue;
        const int64_t q = q0 + (int64_t)it * kThreads;
        float4 sD = make_float4(0.f, 0.f, 0.f, 0.f), sP = sD;
#pragma unroll
        for (int j = 0; j < N; ++j) {          // fixed member order: deterministic sums
            sD.x += phi[it][j].x - the[it][j].x;  sP.x += phi[it][j].x;
            sD.y += phi[it][j].y - the[it][j].y;  sP.y += phi[it][j].y;
            sD.z += phi[it][j].z - the[it][j].z;  sP.z += phi[it][j].z;
            sD.w += phi[it][j].w - the[it][j].w;  sP.w += phi[it][j].w;
        }
        const float4 mP = make_float4(sP.x * a.inv_n, sP.y * a.inv_n, sP.z * a.inv_n, sP.w * a.inv_n);
#pragma unroll
        for (int j = 0; j < N; ++j) {
            float4 d, p;
            p.x = update1(phi[it][j].x, dlt[it][j].x, sD.x, mP.x, a, &d.x);
            p.y = update1(phi[it][j].y, dlt[it][j].y, sD.y, mP.y, a, &d.y);
            p.z = update1(phi[it][j].z, dlt[it][j].z, sD.z, mP.z, a, &d.z);
            p.w = update1(phi[it][j].w, dlt[it][j].w, sD.w, mP.w, a, &d.w);
            __stcs(reinterpret_cast<float4*>(phi_row(j)) + q, p);
            __stcs(reinterpret_cast<float4*>(delta_row(j)) + q, d);
            store_theta4(theta_row(j), q, p);
        }
    }
    if ((a.P & 3) && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) scalar_tail<ThetaT>(a, g);
}

// ---- any subgroup size: two passes over the members -------------------------------------
//
// Pass 1 accumulates the two sums; pass 2 re-reads phi_i (the tile was just touched, so this is
// normally an L2 hit) together with delta_i and writes the update.  Costs at most 4 extra bytes
// of reads per parameter when the re-read misses L2.
template <typename ThetaT>
__global__ void __launch_bounds__(kThreads)
outer_step_any_kernel(const KArgs a) {
    const int g = blockIdx.y;
    const int n = a.n;
    const int64_t full_quads = a.P >> 2;
    const int64_t q = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const int32_t* members = a.perm + (int64_t)g * n;
    if (q < full_quads) {
        float4 sD = make_float4(0.f, 0.f, 0.f, 0.f), sP = sD;
#pragma unroll 4
        for (int j = 0; j < n; ++j) {
            const int64_t row = (int64_t)__ldg(members + j) * a.stride;
            const float4 p = __ldg(reinterpret_cast<const float4*>(a.phi + row) + q);
            const float4 t = load_theta4(static_cast<const ThetaT*>(a.theta) + row, q);
            sD.x += p.x - t.x;  sP.x += p.x;
            sD.y += p.y - t.y;  sP.y += p.y;
            sD.z += p.z - t.z;  sP.z += p.z;
            sD.w += p.w - t.w;  sP.w += p.w;
        }
        const float4 mP = make_float4(sP.x * a.inv_n, sP.y * a.inv_n, sP.z * a.inv_n, sP.w * a.inv_n);
#pragma unroll 4
        for (int j = 0; j < n; ++j) {
            const int64_t row = (int64_t)__ldg(members + j) * a.stride;
            const float4 p0 = __ldcs(reinterpret_cast<const float4*>(a.phi + row) + q);
            const float4 d0 = __ldcs(reinterpret_cast<const float4*>(a.delta + row) + q);
            float4 d, p;
            p.x = update1(p0.x, d0.x, sD.x, mP.x, a, &d.x);
            p.y = update1(p0.y, d0.y, sD.y, mP.y, a, &d.y);
            p.z = update1(p0.z, d0.z, sD.z, mP.z, a, &d.z);
            p.w = update1(p0.w, d0.w, sD.w, mP.w, a, &d.w);
            __stcs(reinterpret_cast<float4*>(a.phi + row) + q, p);
            __stcs(reinterpret_cast<float4*>(a.delta + row) + q, d);
            store_theta4(static_cast<ThetaT*>(a.theta) + row, q, p);
        }
    }
    if ((a.P & 3) && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) scalar_tail<ThetaT>(a, g);
}

template <int N, typename ThetaT, int ITEMS>
cudaError_t launch_reg(const KArgs& k, int groups, cudaStream_t stream) {
    const int64_t quads = (k.P + 3) >> 2;   // a trailing partial quad still needs a CTA for the tail
    const int64_t per_cta = (int64_t)kThreads * ITEMS;
    const int64_t tiles = (quads + per_cta - 1) / per_cta;
    if (tiles > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)tiles, (unsigned)groups);
    outer_step_reg_kernel<N, ThetaT, ITEMS><<<grid, kThreads, 0, stream>>>(k);
    return cudaGetLastError();
}

template <typename ThetaT>
cudaError_t launch_any(const KArgs& k, int groups, cudaStream_t stream) {
    const int64_t quads = (k.P + 3) >> 2;
    const int64_t tiles = (quads + kThreads - 1) / kThreads;
    if (tiles > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)tiles, (unsigned)groups);
    outer_step_any_kernel<ThetaT><<<grid, kThreads, 0, stream>>>(k);
    return cudaGetLastError();
}

template <typename ThetaT>
cudaError_t dispatch(const KArgs& k, int groups, cudaStream_t stream) {
    switch (k.n) {
        case 1:  return launch_reg<1, ThetaT, 4>(k, groups, stream);
        case 2:  return launch_reg<2, ThetaT, 2>(k, groups, stream);
        case 4:  return launch_reg<4, ThetaT, 1>(k, groups, stream);
        case 8:  return launch_reg<8, ThetaT, 1>(k, groups, stream);
        default: return launch_any<ThetaT>(k, groups, stream);
    }
}

}  // namespace

cudaError_t launch_outer(const OuterArgs& a, cudaStream_t stream) {
    if (a.P <= 0 || a.W <= 0) return cudaSuccess;
    KArgs k;
    k.phi = a.phi; k.theta = a.theta; k.delta = a.delta; k.perm = a.perm;
    k.stride = a.stride; k.P = a.P; k.n = a.n;
    k.alpha = a.alpha; k.gamma = a.gamma;
    k.beta_over_n = a.beta / (float)a.n;
    k.inv_n = 1.0f / (float)a.n;
    const int groups = a.W / a.n;
    if (groups > 65535) return cudaErrorInvalidConfiguration;
    return a.theta_bf16 ? dispatch<__nv_bfloat16>(k, groups, stream)
                        : dispatch<float>(k, groups, stream);
}

}  // namespace nolo

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

#include <cooperative_groups.h>
#include <cuda_bf16.h>

namespace cg = cooperative_groups;

namespace nolo {

namespace {

// Launch shape.  One CTA = kThreads threads; a thread of the register-resident kernel handles
// ITEMS quads for all members of its subgroup.  The defaults were chosen by measurement on B200.
#ifndef NOLO_THREADS
#define NOLO_THREADS 256
#endif
#ifndef NOLO_MIN_BLOCKS
#define NOLO_MIN_BLOCKS 1
#endif
#ifndef NOLO_ITEMS_N1
#define NOLO_ITEMS_N1 4
#endif
#ifndef NOLO_ITEMS_N2
#define NOLO_ITEMS_N2 2
#endif
#ifndef NOLO_ITEMS_N4
#define NOLO_ITEMS_N4 1
#endif
#ifndef NOLO_ITEMS_N8
#define NOLO_ITEMS_N8 1
#endif
constexpr int kThreads = NOLO_THREADS;

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
// Raw (unconverted) loads, so that the conversion sits with the arithmetic and never between loads.
__device__ __forceinline__ float4 load_theta_raw(const float* row, int64_t q) {
    return __ldcs(reinterpret_cast<const float4*>(row) + q);
}
__device__ __forceinline__ uint2 load_theta_raw(const __nv_bfloat16* row, int64_t q) {
    return __ldcs(reinterpret_cast<const uint2*>(row) + q);
}
__device__ __forceinline__ float4 widen(float4 v) { return v; }
__device__ __forceinline__ float4 widen(uint2 v) {
    float4 r;
    r.x = __uint_as_float(v.x << 16);
    r.y = __uint_as_float(v.x & 0xffff0000u);
    r.z = __uint_as_float(v.y << 16);
    r.w = __uint_as_float(v.y & 0xffff0000u);
    return r;
}
template <typename ThetaT> struct ThetaRaw { using type = float4; };
template <> struct ThetaRaw<__nv_bfloat16> { using type = uint2; };

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
__global__ void __launch_bounds__(kThreads, NOLO_MIN_BLOCKS)
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

// ---- large subgroups (8 < n <= 64, 192 < n <= 256): members split across warps, CTAs and a cluster
//
// Holding phi of every member of a tile in registers costs n x 512 bytes per 32 quads, and the
// kernel only streams at full bandwidth while more than one CTA fits on an SM (one CTA's loads
// must overlap another's barrier and stores).  So a CTA takes at most 64 members: warp w of its
// G <= 8 warps holds up to 8 members, w*MPW .. w*MPW+MPW-1 of the CTA's share, for the same 32
// quads (each member row is read in coalesced 512-byte segments), and a larger subgroup is spread
// over a thread-block cluster of C = 2 or 4 CTAs that work on the same tile.  Partial sums meet
// in shared memory (warps of a CTA) and then in distributed shared memory (CTAs of the cluster);
// both are added in a fixed order, so the result is deterministic and identical in every CTA.
// As in the small-n kernel every element is read once and written once.  The CTA shape (64
// members, 8 per warp) measured best on B200 among 32/64/128 members and 4/8 per warp.
#ifndef NOLO_SPLIT_CTA_MEMBERS
#define NOLO_SPLIT_CTA_MEMBERS 64     // members one CTA holds (larger subgroups use a cluster)
#endif
#ifndef NOLO_SPLIT_PREF
#define NOLO_SPLIT_PREF 8             // members per warp aimed at when a CTA has more than 16 members
#endif
constexpr int kSplitMaxCluster = 4;    // larger clusters measured slower than the two-pass kernel
constexpr int kSplitMembersPerCta = NOLO_SPLIT_CTA_MEMBERS;
constexpr int kSplitMaxWarps = 16;

// Launch bounds: MAXW warps per CTA; registers per thread capped so that several CTAs fit an SM.
template <int MPW, int MAXW>
struct SplitShape {
    static constexpr int kRegs = MPW <= 4 ? 80 : 128;
    static constexpr int kMinBlocks = (65536 / (MAXW * 32 * kRegs)) > 0 ? (65536 / (MAXW * 32 * kRegs)) : 1;
};

template <int MPW, typename ThetaT, bool CLUSTER, int MAXW>
__global__ void __launch_bounds__(MAXW * 32, SplitShape<MPW, MAXW>::kMinBlocks)
outer_step_split_kernel(const KArgs a, int members_per_cta) {
    __shared__ float4 part_D[MAXW][32];
    __shared__ float4 part_P[MAXW][32];
    __shared__ float4 cta_D[32];
    __shared__ float4 cta_P[32];
    const int G = blockDim.x >> 5;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.y;
    const int n = a.n;
    int C = 1, rank = 0;
    if (CLUSTER) {
        cg::cluster_group cluster = cg::this_cluster();
        C = (int)cluster.num_blocks();
        rank = (int)cluster.block_rank();
    }
    const int64_t tile = CLUSTER ? (int64_t)(blockIdx.x / C) : (int64_t)blockIdx.x;
    const int64_t q = tile * 32 + lane;
    const bool ok = q < (a.P >> 2);
    const int j_begin = rank * members_per_cta;
    const int j_end = min(n, j_begin + members_per_cta);
    const int j0 = j_begin + warp * MPW;

    int row[MPW];
#pragma unroll
    for (int m = 0; m < MPW; ++m) row[m] = (j0 + m < j_end) ? __ldg(a.perm + g * n + j0 + m) : -1;

    float4 phi[MPW], dlt[MPW];
    float4 sD = make_float4(0.f, 0.f, 0.f, 0.f), sP = sD;
    if (ok) {
        typename ThetaRaw<ThetaT>::type raw[MPW];
#pragma unroll
        for (int m = 0; m < MPW; ++m) {
            if (row[m] >= 0) {
                const int64_t off = (int64_t)row[m] * a.stride;
                phi[m] = __ldcs(reinterpret_cast<const float4*>(a.phi + off) + q);
                raw[m] = load_theta_raw(static_cast<const ThetaT*>(a.theta) + off, q);
            }
        }
#pragma unroll
        for (int m = 0; m < MPW; ++m) {
            if (row[m] >= 0)
                dlt[m] = __ldcs(reinterpret_cast<const float4*>(a.delta + (int64_t)row[m] * a.stride) + q);
        }
#pragma unroll
        for (int m = 0; m < MPW; ++m) {
            if (row[m] >= 0) {
                const float4 t = widen(raw[m]);
                sD.x += phi[m].x - t.x;  sP.x += phi[m].x;
                sD.y += phi[m].y - t.y;  sP.y += phi[m].y;
                sD.z += phi[m].z - t.z;  sP.z += phi[m].z;
                sD.w += phi[m].w - t.w;  sP.w += phi[m].w;
            }
        }
    }
    part_D[warp][lane] = sD;
    part_P[warp][lane] = sP;
    __syncthreads();
    // sum over the warps of this CTA, in warp order
    sD = part_D[0][lane];
    sP = part_P[0][lane];
    for (int w = 1; w < G; ++w) {
        const float4 d = part_D[w][lane], p = part_P[w][lane];
        sD.x += d.x; sD.y += d.y; sD.z += d.z; sD.w += d.w;
        sP.x += p.x; sP.y += p.y; sP.z += p.z; sP.w += p.w;
    }
    if (CLUSTER) {
        cg::cluster_group cluster = cg::this_cluster();
        if (warp == 0) {
            cta_D[lane] = sD;
            cta_P[lane] = sP;
        }
        cluster.sync();                       // every CTA's sums are published
        // sum over the CTAs of the cluster, in rank order, through distributed shared memory
        const float4* rD = cluster.map_shared_rank(cta_D, 0);
        const float4* rP = cluster.map_shared_rank(cta_P, 0);
        sD = rD[lane];
        sP = rP[lane];
        for (int c = 1; c < C; ++c) {
            rD = cluster.map_shared_rank(cta_D, c);
            rP = cluster.map_shared_rank(cta_P, c);
            const float4 d = rD[lane], p = rP[lane];
            sD.x += d.x; sD.y += d.y; sD.z += d.z; sD.w += d.w;
            sP.x += p.x; sP.y += p.y; sP.z += p.z; sP.w += p.w;
        }
        cluster.barrier_arrive();             // this CTA no longer reads its peers' shared memory
    }
    if (ok) {
        const float4 mP = make_float4(sP.x * a.inv_n, sP.y * a.inv_n, sP.z * a.inv_n, sP.w * a.inv_n);
#pragma unroll
        for (int m = 0; m < MPW; ++m) {
            if (row[m] >= 0) {
                const int64_t off = (int64_t)row[m] * a.stride;
                float4 d, p;
                p.x = update1(phi[m].x, dlt[m].x, sD.x, mP.x, a, &d.x);
                p.y = update1(phi[m].y, dlt[m].y, sD.y, mP.y, a, &d.y);
                p.z = update1(phi[m].z, dlt[m].z, sD.z, mP.z, a, &d.z);
                p.w = update1(phi[m].w, dlt[m].w, sD.w, mP.w, a, &d.w);
                __stcs(reinterpret_cast<float4*>(a.phi + off) + q, p);
                __stcs(reinterpret_cast<float4*>(a.delta + off) + q, d);
                store_theta4(static_cast<ThetaT*>(a.theta) + off, q, p);
            }
        }
    }
    if ((a.P & 3) && rank == 0 && tile == (int64_t)(gridDim.x / C) - 1 && threadIdx.x == 0)
        scalar_tail<ThetaT>(a, g);
    if (CLUSTER) cg::this_cluster().barrier_wait();   // peers may still be reading this CTA's sums
}

// ---- 64 < n <= 192: phi staged in shared memory by bulk-async copies ------------------------
//
// One CTA of 8 warps (16 above 112 members) owns one subgroup x 32 quads, for all n members.  The members' phi segments
// (512 bytes each) are brought into shared memory by cp.async.bulk copies that complete on one
// mbarrier, so phi needs no registers while it waits for the reduction; meanwhile every warp
// streams the theta segments of its own members through registers and sums them.  After the
// mbarrier and one CTA barrier each warp updates its own members: phi from shared memory, delta
// from global memory.  sum_Delta is formed as sum(phi) - sum(theta), both in a fixed order.
// Still one read and one write per element; n x 512 bytes of shared memory per CTA, 3 CTAs per SM
// at n = 128, 2 at n = 192.  Measured 2 to 19 % faster than spreading such a subgroup over a cluster
// of CTAs; from about 256 members on the cluster kernel below is the faster one again.
// The wait on the mbarrier is bounded: if it ever ran out, the CTA would leave its
// tile untouched and raise the status word instead of hanging.
#ifndef NOLO_STAGED
#define NOLO_STAGED 1
#endif
#ifndef NOLO_STAGED_MAX_N
#define NOLO_STAGED_MAX_N 192
#endif
#ifndef NOLO_STAGED_SPLIT
#define NOLO_STAGED_SPLIT 112      // up to here 8 warps, above 16 (8 to 14 members per warp)
#endif
constexpr int kStagedChunk = 4;      // member rows in flight per thread
constexpr int kStagedWaitLimit = 1 << 20;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

template <typename ThetaT, int kStagedWarps>
__global__ void __launch_bounds__(kStagedWarps * 32, kStagedWarps <= 8 ? 3 : 2)
outer_step_staged_kernel(const KArgs a, int32_t* __restrict__ status) {
    extern __shared__ __align__(128) unsigned char staged_smem[];
    float4* phi_s = reinterpret_cast<float4*>(staged_smem);          // [n][32] quads
    __shared__ float4 part_T[kStagedWarps][32];
    __shared__ float4 part_P[kStagedWarps][32];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int timed_out;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.y;
    const int n = a.n;
    const int32_t* members = a.perm + (int64_t)g * n;
    const int64_t full_quads = a.P >> 2;
    const int64_t q0 = (int64_t)blockIdx.x * 32;
    const int tile_quads = (int)(full_quads - q0 < 32 ? (full_quads - q0 > 0 ? full_quads - q0 : 0) : 32);
    const uint32_t row_bytes = (uint32_t)tile_quads * 16u;
    const uint32_t bar_addr = smem_u32(&bar);

    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        timed_out = 0;
    }
    __syncthreads();
    if (warp == 0 && tile_quads > 0) {
        if (lane == 0)
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr),
                         "r"((uint32_t)n * row_bytes)
                         : "memory");
        __syncwarp();
        for (int j = lane; j < n; j += 32) {
            const float* src = a.phi + (int64_t)__ldg(members + j) * a.stride + q0 * 4;
            asm volatile(
                "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                    smem_u32(phi_s + (size_t)j * 32)),
                "l"(src), "r"(row_bytes), "r"(bar_addr)
                : "memory");
        }
    }

    // theta of this warp's members, through registers
    const int mpw = (n + kStagedWarps - 1) / kStagedWarps;
    const int j_begin = warp * mpw;
    const int j_end = min(n, j_begin + mpw);
    const bool ok = lane < tile_quads;
    const int64_t q = q0 + lane;
    float4 sT = make_float4(0.f, 0.f, 0.f, 0.f), sP = sT;
    if (ok) {
        for (int j = j_begin; j < j_end; j += kStagedChunk) {
            typename ThetaRaw<ThetaT>::type raw[kStagedChunk];
#pragma unroll
            for (int i = 0; i < kStagedChunk; ++i)
                if (j + i < j_end)
                    raw[i] = load_theta_raw(
                        static_cast<const ThetaT*>(a.theta) + (int64_t)__ldg(members + j + i) * a.stride, q);
#pragma unroll
            for (int i = 0; i < kStagedChunk; ++i)
                if (j + i < j_end) {
                    const float4 t = widen(raw[i]);
                    sT.x += t.x; sT.y += t.y; sT.z += t.z; sT.w += t.w;
                }
        }
    }
    if (tile_quads > 0) {                     // bounded wait for the phi segments
        bool done = false;
        for (int it = 0; it < kStagedWaitLimit && !done; ++it) {
            uint32_t ready;
            asm volatile(
                "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n selp.u32 %0, 1, 0, p;\n}\n"
                : "=r"(ready)
                : "r"(bar_addr)
                : "memory");
            done = ready != 0;
        }
        if (!done) timed_out = 1;
    }
    if (ok && !timed_out) {
        for (int j = j_begin; j < j_end; ++j) {
            const float4 p = phi_s[(size_t)j * 32 + lane];
            sP.x += p.x; sP.y += p.y; sP.z += p.z; sP.w += p.w;
        }
    }
    part_T[warp][lane] = sT;
    part_P[warp][lane] = sP;
    __syncthreads();
    if (timed_out) {                           // same value in every thread after the barrier
        if (threadIdx.x == 0 && status) atomicExch(status, 1);
        return;
    }
    if (ok) {
        float4 tT = part_T[0][lane], tP = part_P[0][lane];
#pragma unroll
        for (int w = 1; w < kStagedWarps; ++w) {
            const float4 t = part_T[w][lane], p = part_P[w][lane];
            tT.x += t.x; tT.y += t.y; tT.z += t.z; tT.w += t.w;
            tP.x += p.x; tP.y += p.y; tP.z += p.z; tP.w += p.w;
        }
        const float4 sD = make_float4(tP.x - tT.x, tP.y - tT.y, tP.z - tT.z, tP.w - tT.w);
        const float4 mP = make_float4(tP.x * a.inv_n, tP.y * a.inv_n, tP.z * a.inv_n, tP.w * a.inv_n);
        for (int j = j_begin; j < j_end; j += kStagedChunk) {
            float4 dl[kStagedChunk];
            int64_t off[kStagedChunk];
#pragma unroll
            for (int i = 0; i < kStagedChunk; ++i)
                if (j + i < j_end) {
                    off[i] = (int64_t)__ldg(members + j + i) * a.stride;
                    dl[i] = __ldcs(reinterpret_cast<const float4*>(a.delta + off[i]) + q);
                }
#pragma unroll
            for (int i = 0; i < kStagedChunk; ++i)
                if (j + i < j_end) {
                    const float4 p0 = phi_s[(size_t)(j + i) * 32 + lane];
                    float4 d, p;
                    p.x = update1(p0.x, dl[i].x, sD.x, mP.x, a, &d.x);
                    p.y = update1(p0.y, dl[i].y, sD.y, mP.y, a, &d.y);
                    p.z = update1(p0.z, dl[i].z, sD.z, mP.z, a, &d.z);
                    p.w = update1(p0.w, dl[i].w, sD.w, mP.w, a, &d.w);
                    __stcs(reinterpret_cast<float4*>(a.phi + off[i]) + q, p);
                    __stcs(reinterpret_cast<float4*>(a.delta + off[i]) + q, d);
                    store_theta4(static_cast<ThetaT*>(a.theta) + off[i], q, p);
                }
        }
    }
    if ((a.P & 3) && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) scalar_tail<ThetaT>(a, g);
}

// ---- any subgroup size (used above 256 members): two passes over the members ---------------
//
// Pass 1 accumulates the two sums; pass 2 re-reads phi_i together with delta_i and writes the
// update.  The re-read hits L2 only for small subgroups; for the large ones it is used for it costs
// 4 extra bytes of DRAM reads per parameter (28 instead of 24 bytes), and the kernel still sustains
// a flat 5.3-5.4 TB/s of algorithmic bytes for any n, which beats clusters of 8 CTAs.
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

template <int MPW, typename ThetaT, int MAXW>
cudaError_t launch_split(const KArgs& k, int groups, int warps, int cluster, int members_per_cta,
                         cudaStream_t stream) {
    const int64_t quads = (k.P + 3) >> 2;
    const int64_t tiles = (quads + 31) / 32;
    if (tiles * cluster > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    if (cluster == 1) {
        dim3 grid((unsigned)tiles, (unsigned)groups);
        outer_step_split_kernel<MPW, ThetaT, false, MAXW><<<grid, warps * 32, 0, stream>>>(k, members_per_cta);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles * cluster), (unsigned)groups);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = cluster;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, outer_step_split_kernel<MPW, ThetaT, true, MAXW>, k, members_per_cta);
}

template <typename ThetaT, int WARPS>
cudaError_t launch_staged(const KArgs& k, int groups, int32_t* status, cudaStream_t stream) {
    const int64_t quads = (k.P + 3) >> 2;
    const int64_t tiles = (quads + 31) / 32;
    if (tiles > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)k.n * 32 * sizeof(float4);
    cudaError_t e = cudaFuncSetAttribute(outer_step_staged_kernel<ThetaT, WARPS>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)tiles, (unsigned)groups);
    outer_step_staged_kernel<ThetaT, WARPS><<<grid, WARPS * 32, smem, stream>>>(k, status);
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
cudaError_t dispatch(const KArgs& k, int groups, int32_t* status, cudaStream_t stream) {
    switch (k.n) {
        case 1:  return launch_reg<1, ThetaT, NOLO_ITEMS_N1>(k, groups, stream);
        // pairs: 2 quads per thread with fp32 theta, 1 with bf16 theta measured best (+0.7 %)
        case 2:  return launch_reg<2, ThetaT, (sizeof(ThetaT) == 4) ? NOLO_ITEMS_N2 : 1>(k, groups, stream);
        case 3:  return launch_reg<3, ThetaT, 1>(k, groups, stream);
        case 4:  return launch_reg<4, ThetaT, NOLO_ITEMS_N4>(k, groups, stream);
        case 5:  return launch_reg<5, ThetaT, 1>(k, groups, stream);
        case 6:  return launch_reg<6, ThetaT, 1>(k, groups, stream);
        case 7:  return launch_reg<7, ThetaT, 1>(k, groups, stream);
        case 8:  return launch_reg<8, ThetaT, NOLO_ITEMS_N8>(k, groups, stream);
        default: break;
    }
    if (NOLO_STAGED && k.n > kSplitMembersPerCta && k.n <= NOLO_STAGED_MAX_N) {
        if (k.n <= NOLO_STAGED_SPLIT) return launch_staged<ThetaT, 8>(k, groups, status, stream);
        return launch_staged<ThetaT, 16>(k, groups, status, stream);
    }
    if (k.n <= kSplitMembersPerCta * kSplitMaxCluster) {
        int cluster = 1;
        while (cluster * kSplitMembersPerCta < k.n) cluster *= 2;          // 1, 2 or 4 CTAs
        const int per_cta = (k.n + cluster - 1) / cluster;                 // members per CTA
        const int pref = per_cta > 16 ? NOLO_SPLIT_PREF : 4;               // members per warp aimed at
        const int G = (per_cta + pref - 1) / pref;
        const int mpw = (per_cta + G - 1) / G;
        constexpr int MAXW = (kSplitMembersPerCta + NOLO_SPLIT_PREF - 1) / NOLO_SPLIT_PREF;
        static_assert(MAXW <= kSplitMaxWarps && MAXW >= 4, "CTA shape out of range");
        switch (mpw) {
#define NOLO_SPLIT_CASE(M) \
    case M: return launch_split<M, ThetaT, MAXW>(k, groups, G, cluster, per_cta, stream);
            NOLO_SPLIT_CASE(1) NOLO_SPLIT_CASE(2) NOLO_SPLIT_CASE(3) NOLO_SPLIT_CASE(4)
            NOLO_SPLIT_CASE(5) NOLO_SPLIT_CASE(6) NOLO_SPLIT_CASE(7) NOLO_SPLIT_CASE(8)
#undef NOLO_SPLIT_CASE
            default: break;
        }
    }
    return launch_any<ThetaT>(k, groups, stream);            // n > 256
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
    return a.theta_bf16 ? dispatch<__nv_bfloat16>(k, groups, a.status, stream)
                        : dispatch<float>(k, groups, a.status, stream);
}

}  // namespace nolo

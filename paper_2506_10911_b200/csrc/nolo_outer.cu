// Fused NoLoCo outer step (Section 3.2, Eq. 1-3) for W workers resident in one GPU's memory.
//
// Work decomposition: one CTA owns one subgroup x one tile of parameters.  Every member's
// phi / theta / delta element is fetched from HBM exactly once (128-bit coalesced, streaming
// cache policy) and every output element stored exactly once; the pseudo-gradients, their sum
// and the subgroup mean of phi exist only on chip.  The path is bandwidth bound (about 15 flops
// per 20-24 bytes), so there is no tensor-core work here.
//
//   Delta_j  = phi_j - theta_j                                            (Eq. 1)
//   delta_i' = alpha*delta_i - (beta/n) sum_j Delta_j - gamma*(phi_i - (1/n) sum_j phi_j)   (Eq. 2)
//   phi_i'   = phi_i + delta_i'                                           (Eq. 3)
//   theta_i' = phi_i'   (start of the next inner phase)
//
// Two kernels cover the subgroup sizes:
//   n <= 8        register-resident: one thread holds its quad of every member;
//   n > 8         two passes over the members, the second read of phi served by L1/L2.
//
// Arithmetic.  Delta_j is formed per member and summed in float32 in short fixed-order partial
// sums.  gamma * (phi_i - mean phi) is a small number formed from large ones: a mean rounded to
// float32 would pass half an ulp of |phi| straight into delta', whose tolerance does not grow
// with |phi|.  So the mean is carried as an unevaluated float32 pair hi + lo (about 46 bits):
// the register kernel refines a float32 mean by the mean of the residuals phi_j - mean, the
// two-pass kernel sums phi with error-free additions (Knuth's two-sum: the rounding error of every
// addition is recovered exactly and kept in lo).  Float64 accumulators would do the same, but
// the float32 <-> float64 conversions they need run at 16 per clock per SM on B200 and cost
// the wide-subgroup kernels 20-35 % of their bandwidth when measured.
#include "nolo_internal.h"

#include <cuda_bf16.h>

namespace nolo {

namespace {

constexpr int kThreads = 256;   // CTA size of the register-resident kernel and of the helpers

struct KArgs {
    float* phi;
    void* theta;
    float* delta;
    const int32_t* perm;
    const double* mean_phi;   // subgroup means of phi prepared in advance, [groups][mean_stride]; or NULL
    int64_t mean_stride;
    int64_t stride;
    int64_t P;
    int n;
    float alpha, beta_over_n, gamma, inv_n, n_f;
    double inv_n_d;
};

__device__ __forceinline__ void f4_add(float4& s, const float4 v) {
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
}
__device__ __forceinline__ float4 f4_sub(const float4 a, const float4 b) {
    return make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w);
}
__device__ __forceinline__ float4 f4_scale(const float4 a, const float s) {
    return make_float4(a.x * s, a.y * s, a.z * s, a.w * s);
}
__device__ __forceinline__ float4 f4_zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }

// ---- the mean of phi as a float32 pair ----------------------------------------------------

// hi + x with the rounding error of the addition added to lo (error-free: hi_new + error == hi + x).
__device__ __forceinline__ void two_sum(float& hi, float& lo, const float x) {
    const float s = hi + x;
    const float bb = s - hi;
    lo += (hi - (s - bb)) + (x - bb);
    hi = s;
}

// Running sum of the phi quads of some members, later the mean: value = hi + lo.
struct PairSum {
    float4 hi, lo;
    __device__ __forceinline__ void clear() { hi = f4_zero(); lo = f4_zero(); }
    __device__ __forceinline__ void add(const float4 v) {
        two_sum(hi.x, lo.x, v.x); two_sum(hi.y, lo.y, v.y); two_sum(hi.z, lo.z, v.z); two_sum(hi.w, lo.w, v.w);
    }
    __device__ __forceinline__ void add(const PairSum& o) { add(o.hi); f4_add(lo, o.lo); }
    // sum -> sum / n.  m = fl(hi / n) leaves hi - m*n, which the fused multiply-add returns exactly.
    static __device__ __forceinline__ void divide1(float& h, float& l, const float inv_n, const float n_f) {
        const float m = h * inv_n;
        const float r = fmaf(-m, n_f, h);
        l = (r + l) * inv_n;
        h = m;
    }
    __device__ __forceinline__ void divide(const KArgs& a) {
        divide1(hi.x, lo.x, a.inv_n, a.n_f); divide1(hi.y, lo.y, a.inv_n, a.n_f);
        divide1(hi.z, lo.z, a.inv_n, a.n_f); divide1(hi.w, lo.w, a.inv_n, a.n_f);
    }
    // phi - mean
    __device__ __forceinline__ float4 deviation(const float4 phi) const { return f4_sub(f4_sub(phi, hi), lo); }
};

// The mean of subgroup g for quad q prepared in advance (float64 in memory), split into hi + lo.
__device__ __forceinline__ PairSum load_prepared_mean(const KArgs& a, int g, int64_t q) {
    const double2* m = reinterpret_cast<const double2*>(a.mean_phi + (int64_t)g * a.mean_stride) + 2 * q;
    const double2 u = __ldg(m), v = __ldg(m + 1);
    PairSum p;
    p.hi = make_float4((float)u.x, (float)u.y, (float)v.x, (float)v.y);
    p.lo = make_float4((float)(u.x - (double)p.hi.x), (float)(u.y - (double)p.hi.y),
                       (float)(v.x - (double)p.hi.z), (float)(v.y - (double)p.hi.w));
    return p;
}

// ---- theta access: 4 consecutive parameters as float4, fp32 or bf16 storage -------------

__device__ __forceinline__ float4 widen(float4 v) { return v; }
__device__ __forceinline__ float4 widen(uint2 v) {
    float4 r;
    r.x = __uint_as_float(v.x << 16);
    r.y = __uint_as_float(v.x & 0xffff0000u);
    r.z = __uint_as_float(v.y << 16);
    r.w = __uint_as_float(v.y & 0xffff0000u);
    return r;
}
// Raw (unconverted) loads, so that the conversion sits with the arithmetic and never between loads
// (a conversion placed between the loads serialised them when measured).
__device__ __forceinline__ float4 load_theta_raw(const float* row, int64_t q) {
    return __ldcs(reinterpret_cast<const float4*>(row) + q);
}
__device__ __forceinline__ uint2 load_theta_raw(const __nv_bfloat16* row, int64_t q) {
    return __ldcs(reinterpret_cast<const uint2*>(row) + q);
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

// Eq. 2 and Eq. 3 for one parameter; dev = phi_i - mean phi.
__device__ __forceinline__ float update1(float phi, float dev, float delta, float sum_Delta,
                                         const KArgs& a, float* delta_out) {
    const float d = a.alpha * delta - a.beta_over_n * sum_Delta - a.gamma * dev;
    *delta_out = d;
    return phi + d;
}
__device__ __forceinline__ float4 update4(const float4 phi, const float4 dev, const float4 delta,
                                          const float4 sum_Delta, const KArgs& a, float4* delta_out) {
    float4 p;
    p.x = update1(phi.x, dev.x, delta.x, sum_Delta.x, a, &delta_out->x);
    p.y = update1(phi.y, dev.y, delta.y, sum_Delta.y, a, &delta_out->y);
    p.z = update1(phi.z, dev.z, delta.z, sum_Delta.z, a, &delta_out->z);
    p.w = update1(phi.w, dev.w, delta.w, sum_Delta.w, a, &delta_out->w);
    return p;
}
// update and store one member's quad
template <typename ThetaT>
__device__ __forceinline__ void update_store(const KArgs& a, int64_t row_off, int64_t q, const float4 phi,
                                             const float4 dev, const float4 delta, const float4 sum_Delta) {
    float4 d;
    const float4 p = update4(phi, dev, delta, sum_Delta, a, &d);
    __stcs(reinterpret_cast<float4*>(a.phi + row_off) + q, p);
    __stcs(reinterpret_cast<float4*>(a.delta + row_off) + q, d);
    store_theta4(static_cast<ThetaT*>(a.theta) + row_off, q, p);
}

// Columns P - (P % 4) .. P-1 of one subgroup, element by element in float64 (rows are only
// guaranteed to be padded to a multiple of 8, and padding must not be written).
template <typename ThetaT>
__device__ void scalar_tail(const KArgs& a, int g) {
    const int n = a.n;
    for (int64_t c = a.P & ~int64_t(3); c < a.P; ++c) {
        double sD = 0.0, sP = 0.0;
        for (int j = 0; j < n; ++j) {
            const int64_t row = (int64_t)a.perm[g * n + j] * a.stride;
            const float p = a.phi[row + c];
            sD += (double)(p - load_theta1(static_cast<const ThetaT*>(a.theta) + row, c));
            sP += (double)p;
        }
        const double mP = a.mean_phi ? a.mean_phi[(int64_t)g * a.mean_stride + c] : sP * a.inv_n_d;
        for (int j = 0; j < n; ++j) {
            const int64_t row = (int64_t)a.perm[g * n + j] * a.stride;
            float d;
            const float p0 = a.phi[row + c];
            const float p = update1(p0, (float)((double)p0 - mP), a.delta[row + c], (float)sD, a, &d);
            a.phi[row + c] = p;
            a.delta[row + c] = d;
            store_theta1(static_cast<ThetaT*>(a.theta) + row, c, p);
        }
    }
}

// ---- n <= 8: register-resident, subgroup size N known at compile time --------------------
//
// Each thread handles ITEMS quads (4 consecutive parameters) of the tile, 256 quads apart, for all
// N members: phi_j stays in registers between the reduction and the update, so nothing is read
// twice.  All loads of a thread are issued before the first use to keep many bytes in flight.
// ITEMS = 4 for n = 1, 2 for pairs with float32 theta, 1 otherwise (chosen by measurement).
template <int N, typename ThetaT, int ITEMS, bool PREPARED>
__global__ void __launch_bounds__(kThreads, 1)
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

    float4 phi[ITEMS][N], dlt[ITEMS][N];
    typename ThetaRaw<ThetaT>::type the[ITEMS][N];
    bool ok[ITEMS];
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const int64_t q = q0 + (int64_t)it * kThreads;
        ok[it] = q < full_quads;
        if (ok[it]) {
#pragma unroll
            for (int j = 0; j < N; ++j) {
                phi[it][j] = __ldcs(reinterpret_cast<const float4*>(phi_row(j)) + q);
                the[it][j] = load_theta_raw(theta_row(j), q);
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
        // Sums in the fixed member order (deterministic).  The mean of phi is formed in two
        // passes over the registers: a plain float32 mean, then the mean of the residuals
        // phi_j - mean, so that hi + lo keeps the precision of the spread of the replicas.
        float4 sD = f4_zero(), s0 = f4_zero();
#pragma unroll
        for (int j = 0; j < N; ++j) {
            f4_add(sD, f4_sub(phi[it][j], widen(the[it][j])));          // Eq. 1
            f4_add(s0, phi[it][j]);
        }
        PairSum mean;
        if (PREPARED) {
            mean = load_prepared_mean(a, g, q);
        } else {
            mean.hi = f4_scale(s0, a.inv_n);
            float4 sR = f4_zero();
#pragma unroll
            for (int j = 0; j < N; ++j) f4_add(sR, f4_sub(phi[it][j], mean.hi));
            mean.lo = f4_scale(sR, a.inv_n);
        }
#pragma unroll
        for (int j = 0; j < N; ++j)
            update_store<ThetaT>(a, (int64_t)row[j] * a.stride, q, phi[it][j], mean.deviation(phi[it][j]),
                                 dlt[it][j], sD);
    }
    if ((a.P & 3) && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) scalar_tail<ThetaT>(a, g);
}

// ---- n > 8: two passes over the members, the second read of phi served by L1 / L2 ----------
//
// One CTA owns one subgroup x ROWQ quads.  Its THREADS threads form THREADS/ROWQ slots of ROWQ
// consecutive quads; slot s walks members s, s + SLOTS, ... in chunks of U rows in flight.  Pass 1
// reads phi and theta and accumulates the two sums; the slots' partial sums meet in shared memory;
// pass 2 reads phi again together with delta and writes the update.  Between the two reads of a
// phi element lie only the other rows of the same CTA's tile (n x ROWQ x 16 bytes), so the second
// read is served by L1 or L2 as long as the tiles of all resident CTAs fit there: profiled DRAM
// traffic equals the algorithmic 24 / 20 bytes per worker-parameter, and nothing has to be parked
// in registers or shared memory, whatever n is.  The first chunk of pass 2 depends on no sum, so
// its loads are issued before the partial sums meet and are in flight across the CTA barrier.
// No bulk copies, no clusters and no waits other than that one barrier (none at all with one slot).
//
// The shape trades three things: bytes in flight (threads x U), the width of the piece of a row
// that one CTA streams (ROWQ x 16 bytes: DRAM likes 1-2 KB pieces better than 512-byte ones, and
// 256-byte ones least) and the L2 footprint of the resident tiles
// (CTAs per SM x n x ROWQ x 16 bytes x 148 SMs), which must stay well below the 126 MB of L2 or
// the re-read goes to DRAM.  Small subgroups therefore take wide pieces and few slots, large
// ones narrow pieces; the best shapes have SLOTS x U close to n, so that a slot walks its rows
// in one to four chunks.  Measured on B200 as a fraction of a plain copy (float32 / bfloat16
// theta): 0.96-0.97 / 0.94-0.96 up to 48 members, 0.95 / 0.94 at 64 and at 96, 0.93 at 128,
// 0.92 up to 224, 0.93-0.88 up to 640, 0.89 / 0.84 at 1024.
//
// Tried and measured slower on this access pattern: members held in registers by the warps of a
// CTA, one pass (0.94 for 9-64 members: 512-byte pieces); rings of asynchronous copies (cp.async)
// that keep several chunks in flight per thread (same rate: the kernel is not short of loads in
// flight); phi parked in shared memory; phi parked in tensor memory (tcgen05.st / tcgen05.ld;
// exact, but two CTAs of eight warps per SM are too few warps: 0.78-0.85); a persistent grid
// (0.5-0.7: all CTAs in the same phase at once).  With the re-read of phi left out altogether
// the 512-byte-piece loops reach only 0.92 / 0.91 / 0.89 of a plain copy at n = 128 / 256 / 1024:
// what is lost is lost to streaming n x 3 rows in narrow pieces, not to the second read.
template <typename ThetaT, int THREADS, int ROWQ, int U, int MINB>
__global__ void __launch_bounds__(THREADS, MINB)
outer_step_twopass_kernel(const KArgs a) {
    static_assert(THREADS % 32 == 0 && THREADS % ROWQ == 0, "slots tile the CTA");
    static_assert(ROWQ >= 32 ? ROWQ % 32 == 0 : 32 % ROWQ == 0, "a slot is whole warps or a whole fraction of one");
    constexpr int SLOTS = THREADS / ROWQ;
    constexpr int WARPS = THREADS / 32;
    // Partial sums that meet in shared memory: one per slot when slots are whole warps, one per warp
    // when a warp holds several slots (those are first added by shuffles).
    constexpr int PARTS = ROWQ >= 32 ? SLOTS : WARPS;
    __shared__ float4 part_D[PARTS][ROWQ];
    __shared__ PairSum part_P[PARTS][ROWQ];
    const int lane = threadIdx.x & 31;
    const int ql = threadIdx.x % ROWQ;
    const int slot = threadIdx.x / ROWQ;
    const int part = ROWQ >= 32 ? slot : (threadIdx.x >> 5);
    const int g = blockIdx.y;
    const int n = a.n;
    const int32_t* members = a.perm + (int64_t)g * n;
    const int64_t q = (int64_t)blockIdx.x * ROWQ + ql;
    const bool ok = q < (a.P >> 2);

    float4 sD = f4_zero();
    PairSum sP;
    sP.clear();
    if (ok) {
        for (int j = slot; j < n; j += SLOTS * U) {
            float4 p[U];
            typename ThetaRaw<ThetaT>::type t[U];
#pragma unroll
            for (int i = 0; i < U; ++i) {
                const int jj = j + i * SLOTS;
                if (jj < n) {
                    const int64_t off = (int64_t)__ldg(members + jj) * a.stride;
                    p[i] = reinterpret_cast<const float4*>(a.phi + off)[q];     // default policy: stays cached for pass 2
                    t[i] = load_theta_raw(static_cast<const ThetaT*>(a.theta) + off, q);
                }
            }
#pragma unroll
            for (int i = 0; i < U; ++i) {
                if (j + i * SLOTS < n) {
                    f4_add(sD, f4_sub(p[i], widen(t[i])));              // Eq. 1
                    sP.add(p[i]);
                }
            }
        }
    }
    // pass 2, chunk by chunk: phi (from L1 / L2) and delta of U rows
    float4 p2[U], d2[U];
    int64_t off2[U];
    auto load_chunk = [&](int j) {
#pragma unroll
        for (int i = 0; i < U; ++i) {
            const int jj = j + i * SLOTS;
            if (jj < n) {
                off2[i] = (int64_t)__ldg(members + jj) * a.stride;
                p2[i] = __ldcs(reinterpret_cast<const float4*>(a.phi + off2[i]) + q);
                d2[i] = __ldcs(reinterpret_cast<const float4*>(a.delta + off2[i]) + q);
            }
        }
    };
    if (ok) load_chunk(slot);      // in flight while the partial sums meet
    if constexpr (ROWQ < 32) {
        // the slots of one warp that share a quad, in a fixed order
#pragma unroll
        for (int o = ROWQ; o < 32; o <<= 1) {
            PairSum t;
            float4 d;
            d.x = __shfl_xor_sync(0xffffffffu, sD.x, o); d.y = __shfl_xor_sync(0xffffffffu, sD.y, o);
            d.z = __shfl_xor_sync(0xffffffffu, sD.z, o); d.w = __shfl_xor_sync(0xffffffffu, sD.w, o);
            t.hi.x = __shfl_xor_sync(0xffffffffu, sP.hi.x, o); t.hi.y = __shfl_xor_sync(0xffffffffu, sP.hi.y, o);
            t.hi.z = __shfl_xor_sync(0xffffffffu, sP.hi.z, o); t.hi.w = __shfl_xor_sync(0xffffffffu, sP.hi.w, o);
            t.lo.x = __shfl_xor_sync(0xffffffffu, sP.lo.x, o); t.lo.y = __shfl_xor_sync(0xffffffffu, sP.lo.y, o);
            t.lo.z = __shfl_xor_sync(0xffffffffu, sP.lo.z, o); t.lo.w = __shfl_xor_sync(0xffffffffu, sP.lo.w, o);
            // both partners add (lower slot) + (higher slot) in that order, so they agree bit for bit
            if (lane & o) {
                PairSum mine = sP;
                sP = t;
                sP.add(mine);
                d.x += sD.x; d.y += sD.y; d.z += sD.z; d.w += sD.w;
                sD = d;
            } else {
                sP.add(t);
                f4_add(sD, d);
            }
        }
    }
    if constexpr (PARTS > 1) {
        // the partial sums of the slots (or warps) meet in shared memory
        if (ROWQ >= 32 || lane < ROWQ) {
            part_D[part][ql] = sD;
            part_P[part][ql] = sP;
        }
        __syncthreads();
    }
    if (ok) {
        if constexpr (PARTS > 1) {          // added in index order: the same result in every slot
            sD = part_D[0][ql];
            sP = part_P[0][ql];
#pragma unroll
            for (int w = 1; w < PARTS; ++w) {
                f4_add(sD, part_D[w][ql]);
                sP.add(part_P[w][ql]);
            }
        }
        if (a.mean_phi) sP = load_prepared_mean(a, g, q);
        else sP.divide(a);
        for (int j = slot; j < n; j += SLOTS * U) {
            if (j != slot) load_chunk(j);
#pragma unroll
            for (int i = 0; i < U; ++i) {
                if (j + i * SLOTS < n) update_store<ThetaT>(a, off2[i], q, p2[i], sP.deviation(p2[i]), d2[i], sD);
            }
        }
    }
    if ((a.P & 3) && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) scalar_tail<ThetaT>(a, g);
}

// ---- subgroup means of phi alone (first half of the split-phase step) ------------------------
//
// mean[g][p] = (1/n) sum_{j in subgroup g} phi_j[p], stored as float64.  Section 3.2 notes that
// the slow weights of the partners are known as soon as the previous outer step has finished, so
// this part of Eq. 2 can be exchanged early; only the pseudo-gradients have to wait for the inner
// phase.  Read-only on phi: 4 bytes read per worker-parameter, 8/n bytes written.
constexpr int kMeanUnroll = 4;   // member rows in flight per quad

// Four consecutive float64 means with one 256-bit store (one whole 32-byte sector per lane) where
// the row is 32-byte aligned, else as two 128-bit stores.
template <bool WIDE>
__device__ __forceinline__ void store_mean4(double* out, double a, double b, double c, double d) {
    if (WIDE) {
        asm volatile("st.global.cs.v4.f64 [%0], {%1, %2, %3, %4};" :: "l"(out), "d"(a), "d"(b), "d"(c), "d"(d) : "memory");
    } else {
        __stcs(reinterpret_cast<double2*>(out), make_double2(a, b));
        __stcs(reinterpret_cast<double2*>(out) + 1, make_double2(c, d));
    }
}

// ITEMS quads per thread, 256 quads apart: small subgroups have few rows to keep in flight per
// quad, so each thread takes two quads up to n = 4.
template <int ITEMS, bool WIDE>
__global__ void __launch_bounds__(kThreads)
group_mean_kernel(const float* __restrict__ phi, const int32_t* __restrict__ perm, int n, int64_t stride,
                  int64_t P, double* __restrict__ mean, int64_t mean_stride, double inv_n) {
    const int g = blockIdx.y;
    const int32_t* members = perm + (int64_t)g * n;
    const int64_t q0 = (int64_t)blockIdx.x * (kThreads * ITEMS) + threadIdx.x;
    const int64_t quads = P >> 2;
    PairSum s[ITEMS];
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) s[it].clear();
    for (int j = 0; j < n; j += kMeanUnroll) {
        float4 v[ITEMS][kMeanUnroll];
#pragma unroll
        for (int i = 0; i < kMeanUnroll; ++i) {
            if (j + i < n) {
                const float4* row = reinterpret_cast<const float4*>(phi + (int64_t)__ldg(members + j + i) * stride);
#pragma unroll
                for (int it = 0; it < ITEMS; ++it) {
                    const int64_t q = q0 + (int64_t)it * kThreads;
                    if (q < quads) v[it][i] = __ldcs(row + q);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kMeanUnroll; ++i) {
            if (j + i < n) {
#pragma unroll
                for (int it = 0; it < ITEMS; ++it)
                    if (q0 + (int64_t)it * kThreads < quads) s[it].add(v[it][i]);
            }
        }
    }
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const int64_t q = q0 + (int64_t)it * kThreads;
        if (q < quads) {
            store_mean4<WIDE>(mean + (int64_t)g * mean_stride + 4 * q,
                              ((double)s[it].hi.x + (double)s[it].lo.x) * inv_n, ((double)s[it].hi.y + (double)s[it].lo.y) * inv_n,
                              ((double)s[it].hi.z + (double)s[it].lo.z) * inv_n, ((double)s[it].hi.w + (double)s[it].lo.w) * inv_n);
        }
    }
    if ((P & 3) && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
        for (int64_t c = P & ~int64_t(3); c < P; ++c) {
            double t = 0.0;
            for (int j = 0; j < n; ++j) t += (double)phi[(int64_t)members[j] * stride + c];
            mean[(int64_t)g * mean_stride + c] = t * inv_n;
        }
    }
}

// ---- launches ---------------------------------------------------------------------------

// Tiles of `quads_per_cta` quads; a trailing partial quad still needs a CTA for the scalar tail.
bool tile_grid(const KArgs& k, int64_t quads_per_cta, int groups, dim3* grid) {
    const int64_t quads = (k.P + 3) >> 2;
    const int64_t tiles = (quads + quads_per_cta - 1) / quads_per_cta;
    if (tiles > 0x7fffffffll) return false;
    *grid = dim3((unsigned)tiles, (unsigned)groups);
    return true;
}

template <int N, typename ThetaT, int ITEMS>
cudaError_t launch_reg(const KArgs& k, int groups, cudaStream_t stream) {
    dim3 grid;
    if (!tile_grid(k, (int64_t)kThreads * ITEMS, groups, &grid)) return cudaErrorInvalidConfiguration;
    if (k.mean_phi)
        outer_step_reg_kernel<N, ThetaT, ITEMS, true><<<grid, kThreads, 0, stream>>>(k);
    else
        outer_step_reg_kernel<N, ThetaT, ITEMS, false><<<grid, kThreads, 0, stream>>>(k);
    return cudaGetLastError();
}

template <typename ThetaT, int THREADS, int ROWQ, int U, int MINB>
cudaError_t launch_twopass(const KArgs& k, int groups, cudaStream_t stream) {
    dim3 grid;
    if (!tile_grid(k, ROWQ, groups, &grid)) return cudaErrorInvalidConfiguration;
    outer_step_twopass_kernel<ThetaT, THREADS, ROWQ, U, MINB><<<grid, THREADS, 0, stream>>>(k);
    return cudaGetLastError();
}

// Subgroup sizes up to which each two-pass shape is used (by measurement, see the kernel's comment):
// threads x quads per row piece x rows in flight per slot, CTAs per SM.
constexpr int kTwoPassMaxN1Slot = 12;     // 128 x 128 x 4, 6 CTAs: one slot, no barrier
constexpr int kTwoPassMaxN2Slots = 24;    // 128 x 64 x 8, 4 CTAs
constexpr int kTwoPassMaxN64Quads4 = 64;  // 256 x 64 x 4, 3 CTAs
constexpr int kTwoPassMaxN64Quads8 = 96;  // 256 x 64 x 8, 2 CTAs
constexpr int kTwoPassMaxN4Rows = 128;    // 256 x 32 x 4, 3 CTAs
constexpr int kTwoPassMaxN32Quads = 224;  // 256 x 32 x 8, 2 CTAs
constexpr int kTwoPassMaxN8Warps = 640;   // 256 x 16 x 8, 2 CTAs; above: 512 x 16 x 8, 1 CTA

template <typename ThetaT>
cudaError_t dispatch(const KArgs& k, int groups, cudaStream_t stream) {
    switch (k.n) {
        case 1:  return launch_reg<1, ThetaT, 4>(k, groups, stream);
        // pairs: 2 quads per thread with fp32 theta, 1 with bf16 theta measured best (+0.7 %)
        case 2:  return launch_reg<2, ThetaT, (sizeof(ThetaT) == 4) ? 2 : 1>(k, groups, stream);
        case 3:  return launch_reg<3, ThetaT, 1>(k, groups, stream);
        case 4:  return launch_reg<4, ThetaT, 1>(k, groups, stream);
        case 5:  return launch_reg<5, ThetaT, 1>(k, groups, stream);
        case 6:  return launch_reg<6, ThetaT, 1>(k, groups, stream);
        case 7:  return launch_reg<7, ThetaT, 1>(k, groups, stream);
        case 8:  return launch_reg<8, ThetaT, 1>(k, groups, stream);
        default: break;
    }
    if (k.n <= kTwoPassMaxN1Slot) return launch_twopass<ThetaT, 128, 128, 4, 6>(k, groups, stream);
    if (k.n <= kTwoPassMaxN2Slots) return launch_twopass<ThetaT, 128, 64, 8, 4>(k, groups, stream);
    if (k.n <= kTwoPassMaxN64Quads4) return launch_twopass<ThetaT, 256, 64, 4, 3>(k, groups, stream);
    if (k.n <= kTwoPassMaxN64Quads8) return launch_twopass<ThetaT, 256, 64, 8, 2>(k, groups, stream);
    if (k.n <= kTwoPassMaxN4Rows) return launch_twopass<ThetaT, 256, 32, 4, 3>(k, groups, stream);
    if (k.n <= kTwoPassMaxN32Quads) return launch_twopass<ThetaT, 256, 32, 8, 2>(k, groups, stream);
    if (k.n <= kTwoPassMaxN8Warps) return launch_twopass<ThetaT, 256, 16, 8, 2>(k, groups, stream);
    return launch_twopass<ThetaT, 512, 16, 8, 1>(k, groups, stream);
}

}  // namespace

cudaError_t launch_group_mean(const float* phi, const int32_t* perm, int W, int n, int64_t stride, int64_t P,
                              double* mean, int64_t mean_stride, cudaStream_t stream) {
    if (P <= 0 || W <= 0) return cudaSuccess;
    const int items = n <= 4 ? 2 : 1;
    const int64_t quads = (P + 3) >> 2;
    const int64_t per_cta = (int64_t)kThreads * items;
    const int64_t tiles = (quads + per_cta - 1) / per_cta;
    const int groups = W / n;
    if (tiles > 0x7fffffffll || groups > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)tiles, (unsigned)groups);
    const double inv_n = 1.0 / (double)n;
    // rows of the means are 32-byte aligned when the base is (the stride is a multiple of 64 bytes)
    const bool wide = (reinterpret_cast<uintptr_t>(mean) & 31u) == 0;
    auto launch = [&](auto kernel) { kernel<<<grid, kThreads, 0, stream>>>(phi, perm, n, stride, P, mean, mean_stride, inv_n); };
    if (items == 2) launch(wide ? group_mean_kernel<2, true> : group_mean_kernel<2, false>);
    else launch(wide ? group_mean_kernel<1, true> : group_mean_kernel<1, false>);
    return cudaGetLastError();
}

cudaError_t launch_outer(const OuterArgs& a, cudaStream_t stream) {
    if (a.P <= 0 || a.W <= 0) return cudaSuccess;
    KArgs k;
    k.phi = a.phi; k.theta = a.theta; k.delta = a.delta; k.perm = a.perm;
    k.mean_phi = a.mean_phi; k.mean_stride = a.mean_stride;
    k.stride = a.stride; k.P = a.P; k.n = a.n;
    k.alpha = a.alpha; k.gamma = a.gamma;
    k.beta_over_n = a.beta / (float)a.n;
    k.inv_n = 1.0f / (float)a.n;
    k.n_f = (float)a.n;
    k.inv_n_d = 1.0 / (double)a.n;
    const int groups = a.W / a.n;
    if (groups > 65535) return cudaErrorInvalidConfiguration;
    return a.theta_bf16 ? dispatch<__nv_bfloat16>(k, groups, stream) : dispatch<float>(k, groups, stream);
}

}  // namespace nolo

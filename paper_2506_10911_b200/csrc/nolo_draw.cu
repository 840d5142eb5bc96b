// Random permutations for subgroup draws (Section 3.2) and pipeline routes (Section 3.1).
//
// The paper only asks for random subgroups / random permutations from a seed.  Here element i
// of a draw gets a 64-bit key from the Philox-4x64-10 counter-based generator (Salmon, Moraes,
// Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11) with
// counter = (i, boundary, slot, domain) and key = (seed, step); the permutation lists the
// indices in ascending (key, index) order.  Integer arithmetic only, so the tables are
// reproducible bit for bit on any machine.
#include "nolo_internal.h"

namespace nolo {

namespace {

// Published Philox4x64 multipliers and Weyl key increments.
constexpr uint64_t kM0 = 0xD2E7470EE14C6C93ull;
constexpr uint64_t kM1 = 0xCA5A826395121157ull;
constexpr uint64_t kW0 = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kW1 = 0xBB67AE8584CAA73Bull;

__device__ __forceinline__ uint64_t philox4x64_10_word0(uint64_t c0, uint64_t c1, uint64_t c2,
                                                        uint64_t c3, uint64_t k0, uint64_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t hi0 = __umul64hi(kM0, c0), lo0 = kM0 * c0;
        const uint64_t hi1 = __umul64hi(kM1, c2), lo1 = kM1 * c2;
        const uint64_t n0 = hi1 ^ c1 ^ k0;
        const uint64_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += kW0; k1 += kW1;
    }
    return c0;
}

constexpr int kDrawThreads = 256;

// One CTA per permutation.  Keys live in shared memory; element i's position is the number of
// elements that sort before it (rank by counting: N <= 4096, so N^2 compares are cheap and need
// no sort network).
__global__ void __launch_bounds__(kDrawThreads)
draw_perm_kernel(uint64_t seed, uint64_t step, uint64_t domain, int N, int slots_drawn,
                 int slots_total, int32_t* __restrict__ table) {
    extern __shared__ uint64_t keys[];
    const int b = blockIdx.x / slots_drawn;
    const int s = blockIdx.x % slots_drawn;
    for (int i = threadIdx.x; i < N; i += blockDim.x)
        keys[i] = philox4x64_10_word0((uint64_t)i, (uint64_t)b, (uint64_t)s, domain, seed, step);
    __syncthreads();
    const int k_lo = (slots_drawn == slots_total) ? s : 0;
    const int k_hi = (slots_drawn == slots_total) ? s + 1 : slots_total;
    for (int i = threadIdx.x; i < N; i += blockDim.x) {
        const uint64_t ki = keys[i];
        int rank = 0;
        for (int j = 0; j < N; ++j) {
            const uint64_t kj = keys[j];
            rank += (kj < ki) || (kj == ki && j < i);
        }
        for (int k = k_lo; k < k_hi; ++k)
            table[((int64_t)b * slots_total + k) * N + rank] = i;
    }
}

}  // namespace

cudaError_t launch_draw(uint64_t seed, uint64_t step, int domain, int N, int boundaries,
                        int slots_drawn, int slots_total, int32_t* table, cudaStream_t stream) {
    const int blocks = boundaries * slots_drawn;
    if (blocks <= 0 || N <= 0) return cudaSuccess;
    draw_perm_kernel<<<blocks, kDrawThreads, (size_t)N * sizeof(uint64_t), stream>>>(
        seed, step, (uint64_t)domain, N, slots_drawn, slots_total, table);
    return cudaGetLastError();
}

}  // namespace nolo

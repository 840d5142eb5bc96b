// Random permutations for subgroup draws (Section 3.2) and pipeline routes (Section 3.1).
//
// The paper only asks for random subgroups / random permutations from a seed.  Here element i
// of a draw gets a 64-bit key from the Philox-4x64-10 counter-based generator (Salmon, Moraes,
// Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11) with
// counter = (i, boundary, slot, domain) and key = (seed, step); the permutation lists the
// indices in ascending (key, index) order.  Integer arithmetic only, so the tables are
// reproducible bit for bit on any machine.
#include "nolo_internal.h"
#include "nolo_philox.cuh"

namespace nolo {

namespace {

constexpr int kDrawThreads = 256;

// One CTA per permutation.  Keys live in shared memory; element i's position is the number of
// elements that sort before it (rank by counting: N <= 4096, so N^2 compares are cheap and need
// no sort network).
__global__ void __launch_bounds__(kDrawThreads)
draw_perm_kernel(uint64_t seed, uint64_t step, uint64_t domain, int N, int first_boundary, int slots_drawn,
                 int slots_total, int32_t* __restrict__ table) {
    extern __shared__ uint64_t keys[];
    const int b = first_boundary + blockIdx.x / slots_drawn;
    const int s = blockIdx.x % slots_drawn;
    for (int i = threadIdx.x; i < N; i += blockDim.x)
        keys[i] = draw_key((uint64_t)i, (uint64_t)b, (uint64_t)s, domain, seed, step);
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

cudaError_t launch_draw_range(uint64_t seed, uint64_t step, int domain, int N, int first_boundary,
                              int boundaries, int slots_drawn, int slots_total, int32_t* table,
                              cudaStream_t stream) {
    const int blocks = boundaries * slots_drawn;
    if (blocks <= 0 || N <= 0) return cudaSuccess;
    draw_perm_kernel<<<blocks, kDrawThreads, (size_t)N * sizeof(uint64_t), stream>>>(
        seed, step, (uint64_t)domain, N, first_boundary, slots_drawn, slots_total, table);
    return cudaGetLastError();
}

cudaError_t launch_draw(uint64_t seed, uint64_t step, int domain, int N, int boundaries,
                        int slots_drawn, int slots_total, int32_t* table, cudaStream_t stream) {
    return launch_draw_range(seed, step, domain, N, 0, boundaries, slots_drawn, slots_total, table, stream);
}

}  // namespace nolo

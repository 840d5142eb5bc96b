// Internal launch interfaces between the C ABI layer and the kernels.
// Nothing here is exported.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace nolo {

constexpr int kDomainGroups = 1;  // counter word 3 for subgroup draws
constexpr int kDomainRoute = 2;   // counter word 3 for routing draws

// Draw `blocks` permutations of 0..N-1 into `table`.
// Permutation p (0 <= p < boundaries*slots_drawn) has boundary b = p / slots_drawn and
// slot s = p % slots_drawn, and is written to table[(b*slots_total + k)*N ..] for k = s when
// slots_drawn == slots_total, or for every k in [0, slots_total) when slots_drawn == 1.
cudaError_t launch_draw(uint64_t seed, uint64_t step, int domain, int N, int boundaries,
                        int slots_drawn, int slots_total, int32_t* table, cudaStream_t stream);

// The same for boundaries first_boundary .. first_boundary + boundaries - 1 only (table indexed by the
// absolute boundary).
cudaError_t launch_draw_range(uint64_t seed, uint64_t step, int domain, int N, int first_boundary,
                              int boundaries, int slots_drawn, int slots_total, int32_t* table,
                              cudaStream_t stream);

struct OuterArgs {
    float* phi;          // [W][stride]
    void* theta;         // [W][stride] float or bf16
    float* delta;        // [W][stride]
    const int32_t* perm; // [W]; subgroup g = perm[g*n .. g*n+n-1]
    int64_t stride;      // elements between rows
    int64_t P;           // columns to process, starting at the pointers given
    int W, n;
    int theta_bf16;
    float alpha, beta, gamma;
    // Subgroup means of phi prepared in advance (float64, [W/n][mean_stride], row g for subgroup g of
    // `perm`); NULL = the kernel forms the means itself.
    const double* mean_phi = nullptr;
    int64_t mean_stride = 0;
};

// Fused Eq. 1-3 + theta reset over columns [0, P) of the rows (pointers may be pre-offset by
// a multiple of 8 columns).  One launch.
cudaError_t launch_outer(const OuterArgs& a, cudaStream_t stream);

// mean[g][0..P) = float64 mean of phi over subgroup g of `perm` (the part of Eq. 2 that depends on
// the slow weights only).  One launch.
cudaError_t launch_group_mean(const float* phi, const int32_t* perm, int W, int n, int64_t stride, int64_t P,
                              double* mean, int64_t mean_stride, cudaStream_t stream);

struct RouteArgs {
    const void* in;        // [B][R][K][E]
    void* out;             // [B][R][K][E]
    const int32_t* table;  // [B][K][R]
    int B, R, K;
    int64_t E;
    int elem_size;         // bytes
    int backward;          // 0: out[b][r][k] = in[b][table[b][k][r]][k]; 1: the inverse
};

cudaError_t launch_route(const RouteArgs& a, cudaStream_t stream);

// Plain copy of `bytes` (a multiple of 16): one-shot grid, 128-bit streaming loads and stores.
cudaError_t launch_copy_probe(const void* in, void* out, int64_t bytes, cudaStream_t stream);

// Replica divergence of phi (Fig. 3b): out2[0] = mean over parameters of the across-worker
// population standard deviation, out2[1] = sqrt(mean over parameters of the across-worker variance).
// `partials` is device scratch of divergence_partials(P) * 16 bytes; out2 is device memory.
int64_t divergence_partials(int64_t P);
cudaError_t launch_divergence(const float* phi, int W, int64_t stride, int64_t P, void* partials,
                              double* out2, cudaStream_t stream);

// Latency simulations (Section 4.3).  per_trial: device [trials] resp. [trials][2];
// stats: device, the column means followed by their standard errors.
cudaError_t launch_tree_allreduce(int W, double mu, double sigma, int64_t trials, uint64_t seed,
                                  double* per_trial, double* stats, cudaStream_t stream);
cudaError_t launch_straggler(int W, int n, int H, int T, double mu, double sigma, int64_t trials,
                             uint64_t seed, double* per_trial, double* stats, cudaStream_t stream);

}  // namespace nolo

// Monte-Carlo latency simulations of Section 4.3 and the latency-analysis appendix.
//
//  * tree all-reduce vs pair exchange: message times t ~ LogNormal(mu, sigma^2), i.i.d.; a parent of
//    the binary tree is ready when both children's messages have arrived, the result then descends
//    the same tree; the completion time is the last leaf's arrival.  (Constant t_c gives the paper's
//    2 t_c log2 W; W = 2 is the pair exchange max(t1,t2) + max(t3,t4).)
//  * straggler effect: inner-step times LogNormal(mu, sigma^2); DiLoCo waits at a global barrier
//    after every H inner steps, NoLoCo only for the members of its random subgroup of n.
//
// Random numbers: every Philox-4x64-10 block yields four times.  Words -> u = ((x >> 11) + 0.5) 2^-53;
// Box-Muller on the word pairs (0,1) and (2,3), r = sqrt(-2 ln u_a), gives the normals
// [r01 cos, r01 sin, r23 cos, r23 sin] of the angle 2 pi u_b; t = exp(mu + sigma z).  Sample j of a
// stream is position j % 4 of block j / 4.  float64 throughout.
#include "nolo_internal.h"
#include "nolo_philox.cuh"

namespace nolo {

namespace {

constexpr int kTreeThreads = 128;   // small CTAs: the upper tree levels leave few threads busy
constexpr uint64_t kDomainTree = 3;
constexpr uint64_t kDomainStraggler = 4;

__device__ __forceinline__ double uniform_open(uint64_t x) {
    return ((double)(x >> 11) + 0.5) * 0x1.0p-53;
}

// The two log-normal times of one word pair: cosine first, sine second.
__device__ __forceinline__ void lognormal2(uint64_t wa, uint64_t wb, double mu, double sigma, double& t_cos,
                                           double& t_sin) {
    double s, c;
    const double r = sqrt(-2.0 * log(uniform_open(wa)));
    sincospi(2.0 * uniform_open(wb), &s, &c);
    t_cos = exp(mu + sigma * (r * c));
    t_sin = exp(mu + sigma * (r * s));
}

// The four log-normal times of one block.
__device__ __forceinline__ void lognormal4(const Philox4& b, double mu, double sigma, double (&t)[4]) {
    lognormal2(b.w0, b.w1, mu, sigma, t[0], t[1]);
    lognormal2(b.w2, b.w3, mu, sigma, t[2], t[3]);
}

// Maximum over the CTA, returned to every thread.  Contains two barriers.
__device__ __forceinline__ double block_max(double v, double* scratch /*[32]*/) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, off));
    __syncthreads();                      // scratch may still be read from a previous call
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    const int warps = (blockDim.x + 31) >> 5;
    double m = scratch[0];
    for (int w = 1; w < warps; ++w) m = fmax(m, scratch[w]);
    return m;
}

// One CTA per trial.  node[] holds ready times on the way up and arrival times on the way down,
// indexed like a binary heap: root 1, children of p are 2p and 2p+1, leaves W .. 2W-1.
__global__ void tree_allreduce_kernel(int W, double mu, double sigma, uint64_t seed,
                                      double* __restrict__ out) {
    extern __shared__ double node[];      // [2W]
    __shared__ double scratch[32];
    const uint64_t trial = blockIdx.x;
    for (int i = threadIdx.x; i < 2 * W; i += blockDim.x) node[i] = 0.0;
    __syncthreads();
    // A block serves the four nodes 4q .. 4q+3; two siblings 2p, 2p+1 share one of its word pairs.  One
    // thread per sibling pair: the levels near the root have few nodes, so the work of a block is
    // split over two threads (each recomputes the block's integer rounds) rather than halving the
    // number of busy threads.
    for (int first = W >> 1; first >= 1; first >>= 1) {          // parents of one level: first .. 2*first-1
        for (int p = first + threadIdx.x; p < 2 * first; p += blockDim.x) {
            const Philox4 b = philox4x64_10(p >> 1, trial, 0, kDomainTree, seed, 0);   // children 2p, 2p+1 are in block p/2
            double ta, tb;
            if (p & 1) lognormal2(b.w2, b.w3, mu, sigma, ta, tb);
            else lognormal2(b.w0, b.w1, mu, sigma, ta, tb);
            node[p] = fmax(node[2 * p] + ta, node[2 * p + 1] + tb);
        }
        __syncthreads();
    }
    for (int first = 2; first < 2 * W; first <<= 1) {            // children of one level, top down, in sibling pairs
        for (int c = first + 2 * threadIdx.x; c < 2 * first; c += 2 * blockDim.x) {
            const Philox4 b = philox4x64_10(c >> 2, trial, 1, kDomainTree, seed, 0);
            double ta, tb;
            if (c & 2) lognormal2(b.w2, b.w3, mu, sigma, ta, tb);
            else lognormal2(b.w0, b.w1, mu, sigma, ta, tb);
            const double parent = node[c >> 1];
            node[c] = parent + ta;
            node[c + 1] = parent + tb;
        }
        __syncthreads();
    }
    double m = 0.0;
    for (int leaf = W + threadIdx.x; leaf < 2 * W; leaf += blockDim.x) m = fmax(m, node[leaf]);
    m = block_max(m, scratch);
    if (threadIdx.x == 0) out[trial] = m;
}

// One CTA per trial; thread w (striding) owns worker w.
__global__ void straggler_kernel(int W, int n, int H, int T, double mu, double sigma, uint64_t seed,
                                 double* __restrict__ out /*[trials][2]*/) {
    extern __shared__ unsigned char raw[];
    uint64_t* keys = reinterpret_cast<uint64_t*>(raw);            // [W]
    double* done = reinterpret_cast<double*>(keys + W);           // [W] clock + work of this step
    double* clock = done + W;                                     // [W]
    int* perm = reinterpret_cast<int*>(clock + W);                // [W]
    __shared__ double scratch[32];
    const uint64_t trial = blockIdx.x;
    for (int w = threadIdx.x; w < W; w += blockDim.x) clock[w] = 0.0;
    double barrier_clock = 0.0;
    __syncthreads();
    for (int t = 0; t < T; ++t) {
        double longest = 0.0;
        for (int w = threadIdx.x; w < W; w += blockDim.x) {
            double work = 0.0;
            for (int k0 = 0; k0 < H; k0 += 4) {                   // inner steps k0 .. k0+3 share a block
                double step[4];
                lognormal4(philox4x64_10(k0 >> 2, w, t, kDomainStraggler, seed, trial), mu, sigma, step);
#pragma unroll
                for (int l = 0; l < 4; ++l)
                    if (k0 + l < H) work += step[l];
            }
            longest = fmax(longest, work);
            done[w] = clock[w] + work;
            keys[w] = draw_key(w, trial, 0, kDomainGroups, seed, t);
        }
        barrier_clock += block_max(longest, scratch);             // its barriers also publish done[] and keys[]
        for (int w = threadIdx.x; w < W; w += blockDim.x) {
            const uint64_t kw = keys[w];
            int rank = 0;
            for (int j = 0; j < W; ++j) {
                const uint64_t kj = keys[j];
                rank += (kj < kw) || (kj == kw && j < w);
            }
            perm[rank] = w;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < W; i += blockDim.x) {      // position i of the permutation
            const int g0 = (i / n) * n;
            double m = done[perm[g0]];
            for (int j = 1; j < n; ++j) m = fmax(m, done[perm[g0 + j]]);
            clock[perm[i]] = m;
        }
        __syncthreads();
    }
    double m = 0.0;
    for (int w = threadIdx.x; w < W; w += blockDim.x) m = fmax(m, clock[w]);
    m = block_max(m, scratch);
    if (threadIdx.x == 0) {
        out[2 * trial] = barrier_clock;
        out[2 * trial + 1] = m;
    }
}

// Column means of a [rows][cols] array by one CTA, in a fixed order, to out[c]; the standard error
// of each mean, sqrt(sample variance / rows), to out[cols + c].
__global__ void __launch_bounds__(1024)
column_stats_kernel(const double* __restrict__ x, int64_t rows, int cols, double* __restrict__ out) {
    __shared__ double sm[1024];
    for (int c = 0; c < cols; ++c) {
        double s = 0.0;
        for (int64_t i = threadIdx.x; i < rows; i += 1024) s += x[i * cols + c];
        sm[threadIdx.x] = s;
        __syncthreads();
        for (int k = 512; k > 0; k >>= 1) {
            if (threadIdx.x < k) sm[threadIdx.x] += sm[threadIdx.x + k];
            __syncthreads();
        }
        const double mean = sm[0] / (double)rows;
        __syncthreads();
        double q = 0.0;
        for (int64_t i = threadIdx.x; i < rows; i += 1024) {
            const double d = x[i * cols + c] - mean;
            q += d * d;
        }
        sm[threadIdx.x] = q;
        __syncthreads();
        for (int k = 512; k > 0; k >>= 1) {
            if (threadIdx.x < k) sm[threadIdx.x] += sm[threadIdx.x + k];
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            out[c] = mean;
            out[cols + c] = rows > 1 ? sqrt(sm[0] / (double)(rows - 1) / (double)rows) : 0.0;
        }
        __syncthreads();
    }
}

int round_up_threads(int want) {
    const int t = (want + 31) / 32 * 32;
    return t < 32 ? 32 : (t > 1024 ? 1024 : t);
}

}  // namespace

cudaError_t launch_tree_allreduce(int W, double mu, double sigma, int64_t trials, uint64_t seed,
                                  double* per_trial, double* stats, cudaStream_t stream) {
    const size_t smem = sizeof(double) * 2 * (size_t)W;
    cudaError_t e = cudaFuncSetAttribute(tree_allreduce_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    tree_allreduce_kernel<<<(unsigned)trials, round_up_threads(W / 2 < kTreeThreads ? W / 2 : kTreeThreads), smem, stream>>>(W, mu, sigma, seed,
                                                                                        per_trial);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    column_stats_kernel<<<1, 1024, 0, stream>>>(per_trial, trials, 1, stats);
    return cudaGetLastError();
}

cudaError_t launch_straggler(int W, int n, int H, int T, double mu, double sigma, int64_t trials,
                             uint64_t seed, double* per_trial, double* stats, cudaStream_t stream) {
    const size_t smem = (size_t)W * (8 + 8 + 8 + 4);
    cudaError_t e = cudaFuncSetAttribute(straggler_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    straggler_kernel<<<(unsigned)trials, round_up_threads(W), smem, stream>>>(W, n, H, T, mu, sigma, seed,
                                                                              per_trial);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    column_stats_kernel<<<1, 1024, 0, stream>>>(per_trial, trials, 2, stats);
    return cudaGetLastError();
}

}  // namespace nolo

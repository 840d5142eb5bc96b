/*
 * Second, independent writing of the CPU oracle in plain C.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It restates, element by element and in
 * float64, what the NumPy oracle beside it computes, so that the two can check each other
 * (they must agree to 1e-12 relative) before either judges the CUDA library.  It shares no
 * code, header, table or constant generator with the CUDA library; it is loaded only by the
 * tests and by the benchmark's CPU-baseline leg.
 *
 * What follows the paper (NoLoCo, arXiv 2506.10911):
 *   oc_outer_step      Section 3.2: Eq. 1 (outer gradient), Eq. 2 (modified Nesterov momentum over
 *                      a random subgroup of n workers), Eq. 3 (slow-weight update), then the reset
 *                      of the fast weights to the new slow weights.  Delta = phi - theta: the sign
 *                      under which Eq. 2 as printed moves phi toward theta (Appendix D's recursion).
 *   oc_route           Section 3.1 / Algorithm 1: per stage boundary a permutation of the replicas;
 *                      activations follow it forward, gradients come back along the same path.
 *   oc_divergence      Fig. 3b: spread of the slow weights across the data-parallel replicas.
 * What the paper leaves open and the library defines (hence "parity unpinned" by the paper; pinned
 * in the tests against numpy's own Philox generator and against structural properties):
 *   oc_philox4x64_10   Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3"
 *                      (SC'11): 4 x 64-bit counter, 2 x 64-bit key, 10 rounds.
 *   oc_draw_perm       indices 0..N-1 ordered by (random 64-bit key, index).
 *
 * Loops over parameters are independent; with OpenMP they are shared out over the host cores
 * (oc_set_threads), which changes no result.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef unsigned __int128 u128;

/* Multipliers and Weyl key increments of Philox-4x64 as published (SC'11, Table 2 and Section 3.3). */
static const uint64_t kMul0 = 0xD2E7470EE14C6C93ULL;
static const uint64_t kMul1 = 0xCA5A826395121157ULL;
static const uint64_t kWeyl0 = 0x9E3779B97F4A7C15ULL; /* golden ratio */
static const uint64_t kWeyl1 = 0xBB67AE8584CAA73BULL; /* sqrt(3) - 1 */

int oc_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oc_set_threads(int t) {
#ifdef _OPENMP
    if (t >= 1) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* One block of Philox-4x64-10: out[0..3] from counter ctr[0..3] and key key[0..1]. */
void oc_philox4x64_10(const uint64_t* ctr, const uint64_t* key, uint64_t* out) {
    uint64_t x0 = ctr[0], x1 = ctr[1], x2 = ctr[2], x3 = ctr[3];
    uint64_t ka = key[0], kb = key[1];
    for (int round = 0; round < 10; ++round) {
        const u128 prod_a = (u128)kMul0 * x0; /* feeds words 2 and 3 */
        const u128 prod_b = (u128)kMul1 * x2; /* feeds words 0 and 1 */
        const uint64_t y0 = (uint64_t)(prod_b >> 64) ^ x1 ^ ka;
        const uint64_t y1 = (uint64_t)prod_b;
        const uint64_t y2 = (uint64_t)(prod_a >> 64) ^ x3 ^ kb;
        const uint64_t y3 = (uint64_t)prod_a;
        x0 = y0; x1 = y1; x2 = y2; x3 = y3;
        ka += kWeyl0; /* the key of the next round */
        kb += kWeyl1;
    }
    out[0] = x0; out[1] = x1; out[2] = x2; out[3] = x3;
}

/*
 * Permutation of 0..N-1: element i gets the key word 0 of the block with counter
 * (i, boundary, slot, domain) under key (seed, step); the permutation lists the indices by
 * ascending key, equal keys by ascending index.  Insertion sort: N is at most a few thousand.
 */
int oc_draw_perm(uint64_t seed, uint64_t step, uint64_t domain, uint64_t boundary, uint64_t slot,
                 int N, int32_t* perm) {
    if (N < 0) return -1;
    uint64_t* keys = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(N > 0 ? N : 1));
    if (!keys) return -2;
    const uint64_t key[2] = {seed, step};
    for (int i = 0; i < N; ++i) {
        const uint64_t ctr[4] = {(uint64_t)i, boundary, slot, domain};
        uint64_t blk[4];
        oc_philox4x64_10(ctr, key, blk);
        keys[i] = blk[0];
    }
    for (int i = 0; i < N; ++i) {
        /* indices arrive in ascending order, so inserting after every key <= keys[i] keeps equal
           keys in index order */
        int pos = i;
        while (pos > 0 && keys[perm[pos - 1]] > keys[i]) {
            perm[pos] = perm[pos - 1];
            --pos;
        }
        perm[pos] = i;
    }
    free(keys);
    return 0;
}

static double bf16_to_double(uint16_t b) {
    const uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* float32 -> bfloat16, round to nearest, ties to even; NaN keeps its sign and becomes quiet. */
static uint16_t float_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u) return (uint16_t)((u >> 16) | 0x0040u);
    const uint32_t kept = u >> 16;
    const uint32_t dropped = u & 0xFFFFu;
    uint32_t r = kept;
    if (dropped > 0x8000u || (dropped == 0x8000u && (kept & 1u))) r = kept + 1u; /* carries into the exponent as it should */
    return (uint16_t)r;
}

/*
 * One outer step, out of place.  Rows: phi, delta float32 [W][stride]; theta float32 or bfloat16
 * bits (theta_bf16 != 0) [W][stride]; outputs the same layouts (only columns 0..P-1 are written).
 * perm[W]: subgroup g = perm[g*n .. g*n+n-1].  For every parameter p and subgroup G (Section 3.2):
 *   Delta_j  = phi_j - theta_j                                           Eq. 1
 *   delta_i' = alpha delta_i - (beta/n) sum_G Delta_j - gamma (phi_i - (1/n) sum_G phi_j)   Eq. 2
 *   phi_i'   = phi_i + delta_i'                                          Eq. 3
 *   theta_i' = phi_i' (float32 phi' rounded to bfloat16 when theta is bfloat16)
 * with the sums over all n members and the slow weights from before the update.
 */
int oc_outer_step(const float* phi, const void* theta, const float* delta, const int32_t* perm,
                  int W, int n, int64_t P, int64_t stride, double alpha, double beta, double gamma,
                  int theta_bf16, float* phi_out, float* delta_out, void* theta_out) {
    if (W < 1 || n < 1 || W % n != 0 || P < 0 || stride < P) return -1;
    const int groups = W / n;
    const float* theta_f = (const float*)theta;
    const uint16_t* theta_h = (const uint16_t*)theta;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        for (int g = 0; g < groups; ++g) {
            const int32_t* G = perm + (int64_t)g * n;
            double sum_Delta = 0.0, sum_phi = 0.0;
            for (int j = 0; j < n; ++j) {
                const int64_t at = (int64_t)G[j] * stride + p;
                const double ph = (double)phi[at];
                const double th = theta_bf16 ? bf16_to_double(theta_h[at]) : (double)theta_f[at];
                sum_Delta += ph - th;
                sum_phi += ph;
            }
            const double mean_Delta = sum_Delta / (double)n;
            const double mean_phi = sum_phi / (double)n;
            for (int j = 0; j < n; ++j) {
                const int64_t at = (int64_t)G[j] * stride + p;
                const double ph = (double)phi[at];
                const double d = alpha * (double)delta[at] - beta * mean_Delta - gamma * (ph - mean_phi);
                const float d32 = (float)d;
                const float p32 = (float)(ph + d);
                delta_out[at] = d32;
                phi_out[at] = p32;
                if (theta_bf16) ((uint16_t*)theta_out)[at] = float_to_bf16(p32);
                else ((float*)theta_out)[at] = p32;
            }
        }
    }
    return 0;
}

/* mean[g][p] = (1/n) sum_{j in subgroup g} phi_j[p]: the part of Eq. 2 that needs the slow weights only. */
int oc_subgroup_mean_phi(const float* phi, const int32_t* perm, int W, int n, int64_t P, int64_t stride,
                         double* mean, int64_t mean_stride) {
    if (W < 1 || n < 1 || W % n != 0 || P < 0) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p)
        for (int g = 0; g < W / n; ++g) {
            double s = 0.0;
            for (int j = 0; j < n; ++j) s += (double)phi[(int64_t)perm[(int64_t)g * n + j] * stride + p];
            mean[(int64_t)g * mean_stride + p] = s / (double)n;
        }
    return 0;
}

/*
 * Routing of blocks of `block_bytes` bytes, acts and out laid out [B][R][K][block], table [B][K][R].
 * forward:  out[b][r][k] = acts[b][table[b][k][r]][k];  backward: out[b][table[b][k][r]][k] = acts[b][r][k].
 */
int oc_route(const void* acts, void* out, const int32_t* table, int B, int R, int K, int64_t block_bytes,
             int backward) {
    if (B < 0 || R < 1 || K < 1 || block_bytes < 0) return -1;
    const char* in = (const char*)acts;
    char* o = (char*)out;
#pragma omp parallel for schedule(static) collapse(2)
    for (int b = 0; b < B; ++b)
        for (int r = 0; r < R; ++r)
            for (int k = 0; k < K; ++k) {
                const int s = table[((int64_t)b * K + k) * R + r];
                const int64_t here = (((int64_t)b * R + r) * K + k) * block_bytes;
                const int64_t there = (((int64_t)b * R + s) * K + k) * block_bytes;
                if (backward) memcpy(o + there, in + here, (size_t)block_bytes);
                else memcpy(o + here, in + there, (size_t)block_bytes);
            }
    return 0;
}

/*
 * Fig. 3b: per parameter the population variance of phi across the W replicas (two-pass, float64);
 * out2[0] = mean over parameters of its square root, out2[1] = square root of its mean.
 */
int oc_divergence(const float* phi, int W, int64_t P, int64_t stride, double* out2) {
    if (W < 1 || P < 1) return -1;
    double sum_std = 0.0, sum_var = 0.0;
    for (int64_t p = 0; p < P; ++p) {
        double m = 0.0;
        for (int w = 0; w < W; ++w) m += (double)phi[(int64_t)w * stride + p];
        m /= (double)W;
        double v = 0.0;
        for (int w = 0; w < W; ++w) {
            const double dev = (double)phi[(int64_t)w * stride + p] - m;
            v += dev * dev;
        }
        v /= (double)W;
        sum_std += sqrt(v);
        sum_var += v;
    }
    out2[0] = sum_std / (double)P;
    out2[1] = sqrt(sum_var / (double)P);
    return 0;
}

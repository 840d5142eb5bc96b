/*
 * nolo.h -- C ABI of the NoLoCo outer synchronisation step and random pipeline
 * routing for W simulated data-parallel workers resident in one GPU's memory.
 *
 * The method is that of "NoLoCo: No-all-reduce Low Communication Training
 * Method for Large Models" (arXiv 2506.10911): Section 3.2, Eq. 1-3 (outer
 * step) and Section 3.1 / Algorithm 1 (random pipeline routing).
 *
 * Conventions
 *   - Every function returns an int status: NOLO_OK (0) or a negative NOLO_E*
 *     code.  Nothing throws; nothing aborts.  nolo_strerror() names a code,
 *     nolo_last_error() gives the handle's last detailed message.
 *   - "device" pointers are CUDA device addresses on the device that was
 *     current when nolo_create() ran; "host" pointers are ordinary (ideally
 *     page-locked) host addresses.  The library never frees or reallocates a
 *     caller's buffer; it owns only its small index tables.
 *   - Calls that enqueue GPU work are asynchronous on the bound stream unless
 *     stated otherwise.  One handle serves one stream at a time and is not
 *     thread-safe.
 *   - Streams are passed as void* holding a cudaStream_t (NULL = default
 *     stream), so that this header needs no CUDA header.
 *
 * Random draws.  The paper only asks for "random" subgroups and routes from a
 * seed.  This library defines them: element i of a draw of size N gets the
 * 64-bit key philox4x64-10(counter = (i, boundary, slot, domain),
 * key = (seed, step)) word 0 (Salmon et al., SC'11), and the permutation lists
 * the indices in ascending (key, index) order.  domain = 1 for subgroups
 * (boundary = slot = 0), domain = 2 for routing.
 */
#ifndef NOLO_H
#define NOLO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NOLO_OK        0
#define NOLO_EINVAL   (-1)  /* bad argument (range, NULL, n does not divide W, ...) */
#define NOLO_ESTATE   (-2)  /* a needed nolo_bind_* call has not been made */
#define NOLO_EALIGN   (-3)  /* pointer or stride violates the alignment rule */
#define NOLO_ECUDA    (-4)  /* a CUDA runtime call failed; see nolo_last_error() */
#define NOLO_ENOMEM   (-5)  /* allocation of the handle or its tables failed */

#define NOLO_F32   0        /* element type codes */
#define NOLO_BF16  1

#define NOLO_MAX_WORKERS 4096
#define NOLO_STATIC_MAX_WORKERS 1024   /* limit of nolo_outer_step_static */

#define NOLO_KERNEL_OUTER 0 /* kernel ids for nolo_timing_read() */
#define NOLO_KERNEL_ROUTE 1
#define NOLO_KERNEL_DIVERGENCE 2
#define NOLO_KERNEL_PREPARE 3

#define NOLO_SIM_MAX_SAMPLES (1LL << 40)  /* W*H*T*trials limit of nolo_sim_straggler */

typedef struct nolo_handle nolo_handle;

/*
 * Create a context for W workers synchronising in random subgroups of n
 * (Section 3.2: N model instances, local subgroup of n), each worker a flat
 * vector of P parameters, in a pipeline of `stages` stages (Section 3.1), with
 * momentum alpha, outer learning rate beta and local averaging weight gamma
 * (Eq. 2).
 *   W      1..NOLO_MAX_WORKERS;  n  1..W and n must divide W (subgroups are a
 *          disjoint random partition);  P >= 1;  stages >= 1;
 *   alpha, beta, gamma  finite.
 * On success *out receives a handle owned by the caller (release it with
 * nolo_destroy).  On failure *out is NULL (if out itself is non-NULL).
 * Allocates only index tables (a few KB of device memory) and CUDA events.
 * Errors: NOLO_EINVAL, NOLO_ENOMEM, NOLO_ECUDA.
 */
int nolo_create(int W, int n, int64_t P, int stages,
                float alpha, float beta, float gamma, nolo_handle** out);

/*
 * Attach the worker state (borrowed; must stay valid while bound).
 *   phi    device, float32 [W][row_stride]: slow weights phi_{t,i}
 *   theta  device, [W][row_stride] of theta_dtype (NOLO_F32 or NOLO_BF16):
 *          fast weights theta_{t+1,i} left by the inner phase
 *   delta  device, float32 [W][row_stride]: outer momentum delta_{t-1,i}
 *   row_stride  elements between consecutive workers' rows; >= P and a
 *          multiple of 8.  Columns >= P are padding: never read as parameters,
 *          never written.  (Performance only: with subgroups of hundreds of
 *          members avoid strides that are an exact multiple of 512 KiB; rows a
 *          large power of two apart share memory channels column by column,
 *          which measured 4-8 % slower.  Any extra padding removes it.)
 *   stream cudaStream_t on which all later work of this handle is enqueued.
 * All three pointers must be 16-byte aligned and the buffers must not overlap.
 * Errors: NOLO_EINVAL (NULL, bad dtype or stride), NOLO_EALIGN.
 */
int nolo_bind_state(nolo_handle* h, void* phi, void* theta, void* delta,
                    int theta_dtype, int64_t row_stride, void* stream);

/*
 * One outer step, in place, on the bound state (Section 3.2):
 *   1. draw the random partition into subgroups from (seed, step);
 *   2. Delta_j = phi_j - theta_j                        (Eq. 1; the sign that
 *      makes Eq. 2 move phi toward theta, as the convergence analysis of
 *      Appendix D and DiLoCo do);
 *   3. per subgroup G:  mean Delta and mean phi over all n members;
 *   4. delta_i <- alpha delta_i - beta mean_G(Delta) - gamma (phi_i - mean_G(phi))   (Eq. 2)
 *      phi_i   <- phi_i + delta_i                                                    (Eq. 3)
 *      theta_i <- phi_i  (rounded to nearest-even when theta is bfloat16).
 * float32 arithmetic, with the subgroup mean of phi carried to about 46 bits so
 * that gamma (phi_i - mean) is accurate for weights of any magnitude; sums in a
 * fixed order (results are reproducible bit for bit); every element of every
 * worker is fetched from device memory once and written once (subgroups of
 * more than 8 members request phi a second time, which the caches serve).
 * NaN and Inf are not special-cased: they make the same parameter of every
 * member of the subgroup non-finite and touch nothing else.
 * Asynchronous.  Errors: NOLO_EINVAL (NULL handle), NOLO_ESTATE (no state
 * bound), NOLO_ECUDA (launch failure).
 */
int nolo_outer_step(nolo_handle* h, uint64_t seed, uint64_t step);

/*
 * The outer step in two phases (Section 3.2, the remark after Eq. 3: the slow
 * weights of the partners are known once the previous outer step is done, so
 * they can be communicated then, overlapped with the inner phase; only the
 * pseudo-gradients have to be exchanged at the step itself).
 *
 * nolo_bind_prepared attaches the buffer that carries the early part:
 *   mean_phi     device, float64 [W/n][mean_stride], 16-byte aligned, borrowed,
 *                disjoint from the state; row g receives the mean of phi over
 *                subgroup g.  float64 so that gamma (phi_i - mean) loses
 *                nothing to the rounding of the mean.
 *   mean_stride  elements between rows; >= P and a multiple of 8.
 * nolo_outer_prepare(seed, next_step) draws the partition that step
 * `next_step` will use (the draw is a pure function of (seed, step), so it is
 * known in advance) and writes mean_phi[g][p] = (1/n) sum_{j in G_g} phi_j[p]
 * from the current phi.  Read-only on the state.  Call it after the last
 * change of phi, e.g. right after the previous outer step, on the same stream.
 * nolo_outer_step_prepared(seed, step) is nolo_outer_step with the mean of phi
 * in Eq. 2 taken from mean_phi instead of being reduced again; it still forms
 * Delta_j = phi_j - theta_j and its subgroup sum.  It returns NOLO_ESTATE and
 * does nothing when no means are prepared, when they were prepared for another
 * (seed, step), or when an outer step of this handle has changed phi since
 * (phi changed by the caller behind the library's back cannot be detected).
 * Results equal nolo_outer_step's to float32 rounding.  On one GPU this form
 * moves more bytes than the fused step (it reads phi once more and the means);
 * it is the building block for a worker-sharded deployment, where the early
 * exchange hides behind the inner phase.
 * Asynchronous.  Errors: NOLO_EINVAL, NOLO_EALIGN, NOLO_ESTATE, NOLO_ECUDA.
 */
int nolo_bind_prepared(nolo_handle* h, void* mean_phi, int64_t mean_stride);
int nolo_outer_prepare(nolo_handle* h, uint64_t seed, uint64_t next_step);
int nolo_outer_step_prepared(nolo_handle* h, uint64_t seed, uint64_t step);

/*
 * (No counterpart in the paper: this is a packaging variant of nolo_outer_step.)
 *
 * The same outer step for callers that must not allocate memory: a trainer whose own memory pool
 * took the whole device at start-up, a process held to a fixed device-memory budget, or a
 * latency-critical loop that cannot afford the device-wide synchronisation inside
 * cudaMalloc / cudaFree.  It needs no handle and calls no cudaMalloc, cudaFree or other
 * allocating routine, on device or host.  The subgroup table, which the handle-based path keeps
 * in memory from cudaMalloc, lives here in a fixed array inside the library's device image:
 * NOLO_STATIC_MAX_WORKERS int32 entries = 4 KiB, held by every GPU that loads the library until
 * the process exits.
 *   W, n, P, alpha, beta, gamma   as for nolo_create, but W <= NOLO_STATIC_MAX_WORKERS; a larger
 *          W is rejected with NOLO_EINVAL and a message naming the limit
 *   phi, theta, delta, theta_dtype, row_stride, stream   as for nolo_bind_state (device
 *          pointers, borrowed, updated in place)
 *   seed, step   as for nolo_outer_step; results are bit-identical to it
 *   err, err_len  optional host buffer that receives a message when the status is not NOLO_OK
 * The first call on each device looks up the array's device address (that device must be
 * current, as it must for every call); make that first call before any stream capture begins.
 * At that first call the driver may also load the library's device code, as it does at any
 * first launch, and take device memory for it once; no later call takes any.
 * All calls on a device share the one table and each call overwrites the entries it uses, so
 * nothing needs clearing between calls -- but two calls whose GPU work overlaps (different
 * streams, no ordering between them) race on the table and give undefined subgroups: order them.
 * Asynchronous.  Errors: NOLO_EINVAL, NOLO_EALIGN, NOLO_ECUDA.
 */
int nolo_outer_step_static(int W, int n, int64_t P, float alpha, float beta, float gamma,
                           void* phi, void* theta, void* delta, int theta_dtype,
                           int64_t row_stride, uint64_t seed, uint64_t step, void* stream,
                           char* err, int err_len);

/*
 * The same step for state that lives in HOST memory: columns are streamed
 * host -> bound device buffers -> host in chunks, copies overlapped with the
 * kernel, and the call returns after the last byte is back in host memory
 * (synchronous).  The device state bound with nolo_bind_state() is used as
 * the staging area and holds the new state afterwards as well.
 *   phi_host, theta_host, delta_host  host, same types and [W][host_stride]
 *          layout as the device buffers (page-locked memory is needed for the
 *          copies to overlap);  host_stride >= P, in elements.
 * Errors: as nolo_outer_step, plus NOLO_EINVAL for NULL/short strides.
 */
int nolo_outer_step_host(nolo_handle* h, uint64_t seed, uint64_t step,
                         void* phi_host, void* theta_host, void* delta_host,
                         int64_t host_stride);

/*
 * Describe the routed activations (Section 3.1; Algorithm 1).  Each of the
 * stages-1 boundaries carries M micro-batches of E elements from the W
 * replicas of one stage to the W replicas of the next; replica r holds
 * K = M / W micro-batch slots.
 *   M      number of micro-batches per boundary; a positive multiple of W
 *   E      elements per micro-batch activation (>= 1)
 *   act_dtype  NOLO_F32 or NOLO_BF16 (data are moved, never interpreted)
 *   acts_out   device, [stages-1][W][K][E]: receives the routed activations;
 *          borrowed; 16-byte aligned; must not overlap the input of nolo_route
 *   per_microbatch  0: one permutation per (step, boundary), all K slots of a
 *          replica travel together;  1: every slot k draws its own.
 * Errors: NOLO_EINVAL, NOLO_EALIGN, NOLO_ENOMEM/NOLO_ECUDA (table allocation).
 */
int nolo_bind_route(nolo_handle* h, int M, int64_t E, int act_dtype,
                    void* acts_out, int per_microbatch);

/*
 * Forward routing for all stages-1 boundaries (Section 3.1: random
 * permutations re-drawn every step; Algorithm 1, forward pass): draws
 * table[b][k][r] = sending replica of stage b whose slot k goes to replica r
 * of stage b+1 (each table[b][k][:] is a permutation of 0..W-1), then
 *   acts_out[b][r][k][:] = acts[b][table[b][k][r]][k][:]      (bit copy).
 *   acts   device, [stages-1][W][K][E], 16-byte aligned, read only.
 * stages == 1 is a valid no-op.  Uses the stream given to nolo_bind_state,
 * or the default stream if no state is bound.  Asynchronous.
 * Errors: NOLO_EINVAL, NOLO_ESTATE (nolo_bind_route not called), NOLO_EALIGN,
 * NOLO_ECUDA.
 */
int nolo_route(nolo_handle* h, uint64_t seed, uint64_t step, const void* acts);

/*
 * Forward routing of ONE stage boundary (what a single stage of Algorithm 1
 * does when it receives its inputs): draws table[boundary][:][:] for
 * (seed, step) -- the same permutation nolo_route would draw for that
 * boundary -- and gathers
 *   out_b[r][k][:] = acts_b[table[boundary][k][r]][k][:].
 *   boundary  0 .. stages-2
 *   acts_b, out_b  device, [W][K][E] of that boundary, 16-byte aligned, disjoint
 * Rows of the table that belong to other boundaries keep whatever an earlier
 * call left there.  Asynchronous.  Errors: as nolo_route.
 */
int nolo_route_boundary(nolo_handle* h, uint64_t seed, uint64_t step, int boundary,
                        const void* acts_b, void* out_b);

/*
 * Backward routing (Algorithm 1, backward pass: gradients return along the
 * path of the forward pass): with the table of (seed, step),
 *   grads_out[b][table[b][k][r]][k][:] = grads[b][r][k][:].
 *   grads, grads_out  device, [stages-1][W][K][E], 16-byte aligned, disjoint.
 * Errors: as nolo_route.
 */
int nolo_route_backward(nolo_handle* h, uint64_t seed, uint64_t step,
                        const void* grads, void* grads_out);

/*
 * Forward routing for activations in HOST memory: copies acts to a device
 * staging buffer the caller provides, routes, and copies the result back;
 * synchronous.
 *   acts_host, out_host  host, [stages-1][W][K][E]
 *   acts_dev   device scratch of the same size (input staging); the routed
 *          result is produced in the acts_out buffer of nolo_bind_route.
 */
int nolo_route_host(nolo_handle* h, uint64_t seed, uint64_t step,
                    const void* acts_host, void* out_host, void* acts_dev);

/*
 * Copy the subgroup table of the most recent outer step to the host:
 * perm[W] int32; subgroup g is perm[g*n .. g*n+n-1].  Synchronises the stream.
 * Errors: NOLO_EINVAL, NOLO_ESTATE (no outer step yet), NOLO_ECUDA.
 */
int nolo_get_groups(nolo_handle* h, int32_t* host_out);

/*
 * Copy the routing table of the most recent route call to the host:
 * int32 [stages-1][K][W].  Synchronises the stream.
 * Errors: NOLO_EINVAL, NOLO_ESTATE (no route call yet), NOLO_ECUDA.
 */
int nolo_get_route(nolo_handle* h, int32_t* host_out);

/*
 * Replica divergence of the bound slow weights phi: how far the W workers have
 * drifted apart (the quantity plotted in Fig. 3b, the standard deviation of the
 * model weights across the data-parallel replicas, before the figure's
 * normalisation by the run's maximum).  For every parameter p the population
 * variance var_p of phi[0..W-1][p] across the workers is formed; then
 *   host_out[0] = (1/P) sum_p sqrt(var_p)      mean per-parameter standard deviation
 *   host_out[1] = sqrt((1/P) sum_p var_p)      root of the mean variance
 * (the paper does not say which of the two scalars it plots).  Read-only on
 * phi; float32 per parameter, float64 sums in a fixed order (reproducible).
 * Allocates 16 bytes per 4096 parameters of device scratch on first use.
 * Synchronous: returns when the two doubles are in host memory.
 * Errors: NOLO_EINVAL, NOLO_ESTATE, NOLO_ENOMEM, NOLO_ECUDA.
 */
int nolo_divergence(nolo_handle* h, double* host_out);

/*
 * Monte-Carlo estimate of the completion time of a binary-tree all-reduce
 * over W workers when every message takes an independent LogNormal(mu,
 * sigma^2) time (Section 4.3 and the latency-analysis appendix; Fig. 5a): a
 * parent is ready when both children's messages have arrived, the result then
 * descends the same tree, and the all-reduce ends when the last leaf has it.
 * With constant message time t_c this is the paper's 2 t_c log2(W); with W = 2
 * it is the pair exchange of local averaging, max(t1,t2) + max(t3,t4).
 *   W       power of two, 2..NOLO_MAX_WORKERS;  sigma >= 0;  trials 1..2^24
 *   seed    random stream.  One philox4x64-10 block gives four times: each
 *           word x gives u = ((x >> 11) + 0.5) 2^-53; Box-Muller on the word
 *           pairs (0,1) and (2,3), r = sqrt(-2 ln u_a), gives the normals
 *           z = [r01 cos, r01 sin, r23 cos, r23 sin] of the angle 2 pi u_b;
 *           t = exp(mu + sigma z).  The message on the edge above heap node c
 *           (2..2W-1) in phase p (0 up, 1 down) of trial s is position c % 4 of
 *           the block with counter (c / 4, s, p, 3) and key (seed, 0)
 *   stream  cudaStream_t for the kernels
 *   host_stats   host, 2 doubles: mean completion time, its standard error
 *   host_trials  host, [trials] completion times, or NULL
 * float64 arithmetic.  Synchronous; allocates and frees its own scratch.
 * Errors: NOLO_EINVAL, NOLO_ENOMEM, NOLO_ECUDA.
 */
int nolo_sim_tree_allreduce(int W, double mu, double sigma, int64_t trials, uint64_t seed,
                            void* stream, double* host_stats, double* host_trials);

/*
 * Expected time of the pair exchange, E[max(t1,t2) + max(t3,t4)] =
 * 2 (1 + erf(sigma/2)) exp(mu + sigma^2/2) for i.i.d. LogNormal(mu, sigma^2)
 * message times (the appendix's closed form): the denominator of Fig. 5a's
 * ratio.  Host arithmetic only.
 */
double nolo_expected_pair_exchange(double mu, double sigma);

/*
 * Monte-Carlo simulation of the cost of the global barrier (Section 4.3,
 * Fig. 5b): every inner step of every worker takes an independent
 * LogNormal(mu, sigma^2) time (the paper: mu = 1, sigma^2 = 0.5), communication
 * is free.  Under DiLoCo all W workers meet after every H inner steps; under
 * NoLoCo a worker only waits for the n members of its random subgroup (the
 * same draw as nolo_outer_step, with step = outer iteration and boundary =
 * trial).  Reports the time for all workers to finish T outer iterations.
 *   seed    inner step k of worker w in outer iteration t of trial s is
 *           position k % 4 of the block with counter (k / 4, w, t, 4) and key
 *           (seed, s), transformed as in nolo_sim_tree_allreduce
 *   host_stats   host, 4 doubles: mean time with the global barrier, mean time
 *           with subgroup waits, then the standard errors of the two means
 *   host_trials  host, [trials][2] (barrier, subgroup) per trial, or NULL
 * Synchronous; allocates and frees its own scratch.  trials 1..2^20, and the
 * total number of samples W*H*T*trials at most NOLO_SIM_MAX_SAMPLES (2^40, about
 * 20 s of GPU time): a larger request is refused with NOLO_EINVAL rather than
 * left to occupy the device.
 * Errors: NOLO_EINVAL, NOLO_ENOMEM, NOLO_ECUDA.
 */
int nolo_sim_straggler(int W, int n, int H, int T, double mu, double sigma, int64_t trials,
                       uint64_t seed, void* stream, double* host_stats, double* host_trials);

/*
 * (Measurement aid; the paper has no counterpart.)  Times a plain
 * device-to-device copy of `bytes` bytes (a one-shot grid of 128-bit streaming
 * loads and stores, two per thread: the fastest plain copy found): 3 warm-up
 * copies, then `iters` copies between CUDA events on `stream`.  The bandwidth
 * 2 * bytes / time is the practical HBM ceiling for a half-read, half-write
 * kernel on this device, against which the other kernels can be read.
 *   src, dst  device, 16-byte aligned, disjoint;  bytes a positive multiple of 16
 *   ms_per_copy  host, receives the mean milliseconds per copy
 * Synchronous.  Errors: NOLO_EINVAL, NOLO_EALIGN, NOLO_ECUDA.
 */
int nolo_copy_probe(const void* src, void* dst, int64_t bytes, int iters, void* stream,
                    double* ms_per_copy);

/*
 * Device-time instrumentation.  With enable != 0 every later launch of the
 * fused outer-step kernel, the routing copy kernel, the divergence kernels and the
 * subgroup-mean kernel of nolo_outer_prepare is bracketed by CUDA
 * events on the bound stream (up to 4096 launches per kernel between reads).
 * nolo_timing_read synchronises the stream, returns the summed device time in
 * milliseconds and the number of bracketed launches of `kernel`
 * (NOLO_KERNEL_OUTER / _ROUTE / _DIVERGENCE / _PREPARE) since the last read, and resets them.
 */
int nolo_timing_enable(nolo_handle* h, int enable);
int nolo_timing_read(nolo_handle* h, int kernel, double* total_ms, int64_t* launches);

/*
 * Like nolo_timing_read, but returns the distribution of the bracketed
 * launches since the last read: stats[0..3] = mean, minimum, median and
 * maximum device time in milliseconds (host array of 4 doubles).  Resets the
 * record like nolo_timing_read.  Errors: NOLO_EINVAL, NOLO_ENOMEM, NOLO_ECUDA.
 */
int nolo_timing_stats(nolo_handle* h, int kernel, double* stats, int64_t* launches);

/*
 * Number of kernels this handle has launched since it was created.
 */
int nolo_launch_count(nolo_handle* h, int64_t* launches);

/*
 * Release the handle and its tables.  Bound buffers are not touched.
 * NULL is accepted.  Waits for the bound stream first.
 */
int nolo_destroy(nolo_handle* h);

/* Static text for a status code (never NULL). */
const char* nolo_strerror(int status);

/* Last detailed error message of this handle ("" if none; never NULL). */
const char* nolo_last_error(nolo_handle* h);

/* Library version, major*10000 + minor*100 + patch. */
int nolo_version(void);

#ifdef __cplusplus
}
#endif
#endif /* NOLO_H */

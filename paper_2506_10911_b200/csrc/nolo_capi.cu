// C ABI of the library (see include/nolo.h): argument validation, the handle, and the order in
// which the kernels are enqueued.  All arithmetic of the method lives in the kernels.
#include "nolo.h"
#include "nolo_internal.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

namespace {

constexpr int kMaxTimed = 4096;
constexpr int kTimedKernels = 4;

struct KernelTimer {
    cudaEvent_t* start = nullptr;
    cudaEvent_t* stop = nullptr;
    int created = 0;   // event pairs that exist
    int used = 0;      // pairs recorded since the last read
};

}  // namespace

struct nolo_handle {
    int W, n, stages;
    int64_t P;
    float alpha, beta, gamma;
    int device;

    // state (borrowed)
    float* phi = nullptr;
    void* theta = nullptr;
    float* delta = nullptr;
    int theta_dtype = NOLO_F32;
    int64_t stride = 0;
    cudaStream_t stream = nullptr;
    bool state_bound = false;

    int32_t* d_perm = nullptr;   // [2][W], owned: the table of the last outer step, then that of the last prepare
    bool groups_valid = false;

    // split-phase step: subgroup means of phi prepared ahead of the step (borrowed buffer)
    double* mean_phi = nullptr;
    int64_t mean_stride = 0;
    bool prepared_valid = false;
    uint64_t prepared_seed = 0, prepared_step = 0;

    // routing
    int M = 0, K = 0, act_dtype = NOLO_F32, per_microbatch = 0;
    int64_t E = 0;
    void* acts_out = nullptr;    // borrowed
    bool route_bound = false;
    int32_t* d_route = nullptr;  // [stages-1][K][W], owned
    bool route_valid = false;

    // divergence metric scratch (allocated on first use)
    void* d_div_partials = nullptr;
    double* d_div_out = nullptr;

    // host-streaming helpers (created on first use)
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_in = nullptr, ev_kernel = nullptr, ev_fence = nullptr;

    bool timing = false;
    KernelTimer timers[kTimedKernels];
    int64_t launches = 0;
    char err[256] = {0};
};

namespace {

int fail(nolo_handle* h, int code, const char* fmt, ...) {
    if (h) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(h->err, sizeof(h->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

int cuda_fail(nolo_handle* h, cudaError_t e, const char* what) {
    return fail(h, NOLO_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define NOLO_CUDA(h, call)                                        \
    do {                                                          \
        cudaError_t e_ = (call);                                  \
        if (e_ != cudaSuccess) return cuda_fail((h), e_, #call);  \
    } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int elem_size(int dtype) { return dtype == NOLO_BF16 ? 2 : 4; }

bool overlap(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + nb && y < x + na;
}

// Start/stop brackets around one kernel launch when timing is on.
struct Bracket {
    nolo_handle* h;
    int slot = -1;
    KernelTimer* t = nullptr;
    Bracket(nolo_handle* h_, int kernel) : h(h_) {
        if (!h->timing) return;
        t = &h->timers[kernel];
        if (t->used >= kMaxTimed) { t = nullptr; return; }
        if (t->used == t->created) {
            if (cudaEventCreate(&t->start[t->created]) != cudaSuccess) { t = nullptr; return; }
            if (cudaEventCreate(&t->stop[t->created]) != cudaSuccess) {
                cudaEventDestroy(t->start[t->created]);
                t = nullptr;
                return;
            }
            ++t->created;
        }
        slot = t->used;
        cudaEventRecord(t->start[slot], h->stream);
    }
    void done() {
        if (!t) return;
        cudaEventRecord(t->stop[slot], h->stream);
        ++t->used;
    }
};

int enqueue_outer(nolo_handle* h, int64_t col0, int64_t cols, bool prepared = false) {
    nolo::OuterArgs a;
    if (prepared) {
        a.mean_phi = h->mean_phi + col0;
        a.mean_stride = h->mean_stride;
    }
    a.phi = h->phi + col0;
    a.theta = static_cast<char*>(h->theta) + col0 * elem_size(h->theta_dtype);
    a.delta = h->delta + col0;
    a.perm = h->d_perm;
    a.stride = h->stride;
    a.P = cols;
    a.W = h->W;
    a.n = h->n;
    a.theta_bf16 = h->theta_dtype == NOLO_BF16;
    a.alpha = h->alpha; a.beta = h->beta; a.gamma = h->gamma;
    Bracket br(h, NOLO_KERNEL_OUTER);
    NOLO_CUDA(h, nolo::launch_outer(a, h->stream));
    br.done();
    ++h->launches;
    h->prepared_valid = false;   // phi has changed: means prepared from the old phi are stale
    return NOLO_OK;
}

int enqueue_group_draw(nolo_handle* h, uint64_t seed, uint64_t step) {
    NOLO_CUDA(h, nolo::launch_draw(seed, step, nolo::kDomainGroups, h->W, 1, 1, 1, h->d_perm, h->stream));
    ++h->launches;
    h->groups_valid = true;
    return NOLO_OK;
}

int enqueue_route(nolo_handle* h, uint64_t seed, uint64_t step, const void* in, void* out, int backward) {
    const int B = h->stages - 1;
    if (B == 0) return NOLO_OK;
    const int drawn = h->per_microbatch ? h->K : 1;
    NOLO_CUDA(h, nolo::launch_draw(seed, step, nolo::kDomainRoute, h->W, B, drawn, h->K, h->d_route, h->stream));
    ++h->launches;
    h->route_valid = true;
    nolo::RouteArgs a;
    a.in = in; a.out = out; a.table = h->d_route;
    a.B = B; a.R = h->W; a.K = h->K; a.E = h->E;
    a.elem_size = elem_size(h->act_dtype);
    a.backward = backward;
    Bracket br(h, NOLO_KERNEL_ROUTE);
    NOLO_CUDA(h, nolo::launch_route(a, h->stream));
    br.done();
    ++h->launches;
    return NOLO_OK;
}

size_t route_bytes(const nolo_handle* h) {
    return (size_t)(h->stages - 1) * h->W * h->K * (size_t)h->E * elem_size(h->act_dtype);
}

int ensure_host_streams(nolo_handle* h) {
    if (h->s_in) return NOLO_OK;
    NOLO_CUDA(h, cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking));
    NOLO_CUDA(h, cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking));
    NOLO_CUDA(h, cudaEventCreateWithFlags(&h->ev_in, cudaEventDisableTiming));
    NOLO_CUDA(h, cudaEventCreateWithFlags(&h->ev_kernel, cudaEventDisableTiming));
    NOLO_CUDA(h, cudaEventCreateWithFlags(&h->ev_fence, cudaEventDisableTiming));
    return NOLO_OK;
}

}  // namespace

extern "C" {

int nolo_create(int W, int n, int64_t P, int stages, float alpha, float beta, float gamma,
                nolo_handle** out) {
    if (!out) return NOLO_EINVAL;
    *out = nullptr;
    if (W < 1 || W > NOLO_MAX_WORKERS || n < 1 || n > W || W % n != 0 || P < 1 || stages < 1)
        return NOLO_EINVAL;
    if (!std::isfinite(alpha) || !std::isfinite(beta) || !std::isfinite(gamma)) return NOLO_EINVAL;
    nolo_handle* h = new (std::nothrow) nolo_handle();
    if (!h) return NOLO_ENOMEM;
    h->W = W; h->n = n; h->P = P; h->stages = stages;
    h->alpha = alpha; h->beta = beta; h->gamma = gamma;
    for (auto& t : h->timers) {
        t.start = new (std::nothrow) cudaEvent_t[kMaxTimed];
        t.stop = new (std::nothrow) cudaEvent_t[kMaxTimed];
        if (!t.start || !t.stop) { nolo_destroy(h); return NOLO_ENOMEM; }
    }
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaMalloc(&h->d_perm, sizeof(int32_t) * 2 * (size_t)W);
    if (e != cudaSuccess) {
        const int code = (e == cudaErrorMemoryAllocation) ? NOLO_ENOMEM : NOLO_ECUDA;
        nolo_destroy(h);
        return code;
    }
    *out = h;
    return NOLO_OK;
}

int nolo_bind_state(nolo_handle* h, void* phi, void* theta, void* delta, int theta_dtype,
                    int64_t row_stride, void* stream) {
    if (!h) return NOLO_EINVAL;
    if (!phi || !theta || !delta) return fail(h, NOLO_EINVAL, "state pointers must not be NULL");
    if (theta_dtype != NOLO_F32 && theta_dtype != NOLO_BF16)
        return fail(h, NOLO_EINVAL, "theta_dtype must be NOLO_F32 or NOLO_BF16");
    if (row_stride < h->P) return fail(h, NOLO_EINVAL, "row_stride %lld < P %lld", (long long)row_stride, (long long)h->P);
    if (row_stride % 8 != 0) return fail(h, NOLO_EALIGN, "row_stride must be a multiple of 8 elements");
    if (!aligned16(phi) || !aligned16(theta) || !aligned16(delta))
        return fail(h, NOLO_EALIGN, "state pointers must be 16-byte aligned");
    const size_t n4 = (size_t)h->W * row_stride * 4, nt = (size_t)h->W * row_stride * elem_size(theta_dtype);
    if (overlap(phi, n4, delta, n4) || overlap(phi, n4, theta, nt) || overlap(delta, n4, theta, nt))
        return fail(h, NOLO_EINVAL, "state buffers overlap");
    h->phi = static_cast<float*>(phi);
    h->theta = theta;
    h->delta = static_cast<float*>(delta);
    h->theta_dtype = theta_dtype;
    h->stride = row_stride;
    h->stream = static_cast<cudaStream_t>(stream);
    h->state_bound = true;
    return NOLO_OK;
}

int nolo_outer_step(nolo_handle* h, uint64_t seed, uint64_t step) {
    if (!h) return NOLO_EINVAL;
    if (!h->state_bound) return fail(h, NOLO_ESTATE, "nolo_bind_state has not been called");
    int rc = enqueue_group_draw(h, seed, step);
    if (rc != NOLO_OK) return rc;
    return enqueue_outer(h, 0, h->P);
}

int nolo_bind_prepared(nolo_handle* h, void* mean_phi, int64_t mean_stride) {
    if (!h) return NOLO_EINVAL;
    if (!h->state_bound) return fail(h, NOLO_ESTATE, "nolo_bind_state has not been called");
    if (!mean_phi) return fail(h, NOLO_EINVAL, "mean_phi must not be NULL");
    if (mean_stride < h->P) return fail(h, NOLO_EINVAL, "mean_stride %lld < P %lld", (long long)mean_stride, (long long)h->P);
    if (mean_stride % 8 != 0) return fail(h, NOLO_EALIGN, "mean_stride must be a multiple of 8 elements");
    if (!aligned16(mean_phi)) return fail(h, NOLO_EALIGN, "mean_phi must be 16-byte aligned");
    const size_t nm = (size_t)(h->W / h->n) * mean_stride * 8;
    const size_t n4 = (size_t)h->W * h->stride * 4, nt = (size_t)h->W * h->stride * elem_size(h->theta_dtype);
    if (overlap(mean_phi, nm, h->phi, n4) || overlap(mean_phi, nm, h->delta, n4) || overlap(mean_phi, nm, h->theta, nt))
        return fail(h, NOLO_EINVAL, "mean_phi overlaps the state");
    h->mean_phi = static_cast<double*>(mean_phi);
    h->mean_stride = mean_stride;
    h->prepared_valid = false;
    return NOLO_OK;
}

int nolo_outer_prepare(nolo_handle* h, uint64_t seed, uint64_t next_step) {
    if (!h) return NOLO_EINVAL;
    if (!h->state_bound) return fail(h, NOLO_ESTATE, "nolo_bind_state has not been called");
    if (!h->mean_phi) return fail(h, NOLO_ESTATE, "nolo_bind_prepared has not been called");
    int32_t* table = h->d_perm + h->W;
    NOLO_CUDA(h, nolo::launch_draw(seed, next_step, nolo::kDomainGroups, h->W, 1, 1, 1, table, h->stream));
    ++h->launches;
    Bracket br(h, NOLO_KERNEL_PREPARE);
    NOLO_CUDA(h, nolo::launch_group_mean(h->phi, table, h->W, h->n, h->stride, h->P, h->mean_phi, h->mean_stride,
                                         h->stream));
    br.done();
    ++h->launches;
    h->prepared_valid = true;
    h->prepared_seed = seed;
    h->prepared_step = next_step;
    return NOLO_OK;
}

int nolo_outer_step_prepared(nolo_handle* h, uint64_t seed, uint64_t step) {
    if (!h) return NOLO_EINVAL;
    if (!h->state_bound) return fail(h, NOLO_ESTATE, "nolo_bind_state has not been called");
    if (!h->mean_phi) return fail(h, NOLO_ESTATE, "nolo_bind_prepared has not been called");
    if (!h->prepared_valid)
        return fail(h, NOLO_ESTATE, "no prepared means: call nolo_outer_prepare after the last change of phi");
    if (h->prepared_seed != seed || h->prepared_step != step)
        return fail(h, NOLO_ESTATE, "means were prepared for (seed %llu, step %llu), not for (seed %llu, step %llu)",
                    (unsigned long long)h->prepared_seed, (unsigned long long)h->prepared_step,
                    (unsigned long long)seed, (unsigned long long)step);
    int rc = enqueue_group_draw(h, seed, step);
    if (rc != NOLO_OK) return rc;
    return enqueue_outer(h, 0, h->P, true);
}

int nolo_outer_step_host(nolo_handle* h, uint64_t seed, uint64_t step, void* phi_host,
                         void* theta_host, void* delta_host, int64_t host_stride) {
    if (!h) return NOLO_EINVAL;
    if (!h->state_bound) return fail(h, NOLO_ESTATE, "nolo_bind_state has not been called");
    if (!phi_host || !theta_host || !delta_host) return fail(h, NOLO_EINVAL, "host pointers must not be NULL");
    if (host_stride < h->P) return fail(h, NOLO_EINVAL, "host_stride < P");
    int rc = ensure_host_streams(h);
    if (rc != NOLO_OK) return rc;
    rc = enqueue_group_draw(h, seed, step);
    if (rc != NOLO_OK) return rc;

    const int ts = elem_size(h->theta_dtype);
    // Column chunks of about 128 MB per fp32 tensor, a multiple of 8 columns.
    int64_t chunk = ((int64_t(32) << 20) / h->W) & ~int64_t(7);
    if (chunk < 8) chunk = 8;
    // Earlier work on the bound stream may still use the device buffers.
    NOLO_CUDA(h, cudaEventRecord(h->ev_fence, h->stream));
    NOLO_CUDA(h, cudaStreamWaitEvent(h->s_in, h->ev_fence, 0));
    for (int64_t c0 = 0; c0 < h->P; c0 += chunk) {
        const int64_t cols = (h->P - c0 < chunk) ? h->P - c0 : chunk;
        const size_t dp4 = (size_t)h->stride * 4, hp4 = (size_t)host_stride * 4;
        const size_t dpt = (size_t)h->stride * ts, hpt = (size_t)host_stride * ts;
        char* th_d = static_cast<char*>(h->theta) + c0 * ts;
        char* th_h = static_cast<char*>(theta_host) + c0 * ts;
        float* ph_h = static_cast<float*>(phi_host) + c0;
        float* de_h = static_cast<float*>(delta_host) + c0;
        NOLO_CUDA(h, cudaMemcpy2DAsync(h->phi + c0, dp4, ph_h, hp4, (size_t)cols * 4, h->W, cudaMemcpyHostToDevice, h->s_in));
        NOLO_CUDA(h, cudaMemcpy2DAsync(th_d, dpt, th_h, hpt, (size_t)cols * ts, h->W, cudaMemcpyHostToDevice, h->s_in));
        NOLO_CUDA(h, cudaMemcpy2DAsync(h->delta + c0, dp4, de_h, hp4, (size_t)cols * 4, h->W, cudaMemcpyHostToDevice, h->s_in));
        NOLO_CUDA(h, cudaEventRecord(h->ev_in, h->s_in));
        NOLO_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_in, 0));
        rc = enqueue_outer(h, c0, cols);
        if (rc != NOLO_OK) return rc;
        NOLO_CUDA(h, cudaEventRecord(h->ev_kernel, h->stream));
        NOLO_CUDA(h, cudaStreamWaitEvent(h->s_out, h->ev_kernel, 0));
        NOLO_CUDA(h, cudaMemcpy2DAsync(ph_h, hp4, h->phi + c0, dp4, (size_t)cols * 4, h->W, cudaMemcpyDeviceToHost, h->s_out));
        NOLO_CUDA(h, cudaMemcpy2DAsync(th_h, hpt, th_d, dpt, (size_t)cols * ts, h->W, cudaMemcpyDeviceToHost, h->s_out));
        NOLO_CUDA(h, cudaMemcpy2DAsync(de_h, hp4, h->delta + c0, dp4, (size_t)cols * 4, h->W, cudaMemcpyDeviceToHost, h->s_out));
    }
    NOLO_CUDA(h, cudaStreamSynchronize(h->s_out));
    NOLO_CUDA(h, cudaStreamSynchronize(h->stream));
    return NOLO_OK;
}

int nolo_bind_route(nolo_handle* h, int M, int64_t E, int act_dtype, void* acts_out, int per_microbatch) {
    if (!h) return NOLO_EINVAL;
    if (M < 1 || M % h->W != 0) return fail(h, NOLO_EINVAL, "M must be a positive multiple of W");
    if (E < 1) return fail(h, NOLO_EINVAL, "E must be >= 1");
    if (act_dtype != NOLO_F32 && act_dtype != NOLO_BF16)
        return fail(h, NOLO_EINVAL, "act_dtype must be NOLO_F32 or NOLO_BF16");
    if (h->stages > 1 && !acts_out) return fail(h, NOLO_EINVAL, "acts_out must not be NULL");
    if (!aligned16(acts_out)) return fail(h, NOLO_EALIGN, "acts_out must be 16-byte aligned");
    const int K = M / h->W;
    if (h->stages > 1 && (K != h->K || !h->d_route)) {
        int32_t* t = nullptr;
        cudaError_t e = cudaMalloc(&t, sizeof(int32_t) * (size_t)(h->stages - 1) * K * h->W);
        if (e != cudaSuccess)
            return fail(h, e == cudaErrorMemoryAllocation ? NOLO_ENOMEM : NOLO_ECUDA,
                        "route table allocation: %s", cudaGetErrorString(e));
        if (h->d_route) cudaFree(h->d_route);
        h->d_route = t;
    }
    h->M = M; h->K = K; h->E = E; h->act_dtype = act_dtype;
    h->acts_out = acts_out;
    h->per_microbatch = per_microbatch ? 1 : 0;
    h->route_bound = true;
    h->route_valid = false;
    return NOLO_OK;
}

int nolo_route(nolo_handle* h, uint64_t seed, uint64_t step, const void* acts) {
    if (!h) return NOLO_EINVAL;
    if (!h->route_bound) return fail(h, NOLO_ESTATE, "nolo_bind_route has not been called");
    if (h->stages == 1) return NOLO_OK;
    if (!acts) return fail(h, NOLO_EINVAL, "acts must not be NULL");
    if (!aligned16(acts)) return fail(h, NOLO_EALIGN, "acts must be 16-byte aligned");
    if (overlap(acts, route_bytes(h), h->acts_out, route_bytes(h)))
        return fail(h, NOLO_EINVAL, "acts overlaps acts_out");
    return enqueue_route(h, seed, step, acts, h->acts_out, 0);
}

int nolo_route_boundary(nolo_handle* h, uint64_t seed, uint64_t step, int boundary, const void* acts_b,
                        void* out_b) {
    if (!h) return NOLO_EINVAL;
    if (!h->route_bound) return fail(h, NOLO_ESTATE, "nolo_bind_route has not been called");
    if (boundary < 0 || boundary >= h->stages - 1)
        return fail(h, NOLO_EINVAL, "boundary %d is outside 0..%d", boundary, h->stages - 2);
    if (!acts_b || !out_b) return fail(h, NOLO_EINVAL, "acts_b and out_b must not be NULL");
    if (!aligned16(acts_b) || !aligned16(out_b)) return fail(h, NOLO_EALIGN, "pointers must be 16-byte aligned");
    const size_t bytes = route_bytes(h) / (size_t)(h->stages - 1);
    if (overlap(acts_b, bytes, out_b, bytes)) return fail(h, NOLO_EINVAL, "acts_b overlaps out_b");
    const int drawn = h->per_microbatch ? h->K : 1;
    NOLO_CUDA(h, nolo::launch_draw_range(seed, step, nolo::kDomainRoute, h->W, boundary, 1, drawn, h->K,
                                         h->d_route, h->stream));
    ++h->launches;
    h->route_valid = true;
    nolo::RouteArgs a;
    a.in = acts_b; a.out = out_b;
    a.table = h->d_route + (size_t)boundary * h->K * h->W;
    a.B = 1; a.R = h->W; a.K = h->K; a.E = h->E;
    a.elem_size = elem_size(h->act_dtype);
    a.backward = 0;
    Bracket br(h, NOLO_KERNEL_ROUTE);
    NOLO_CUDA(h, nolo::launch_route(a, h->stream));
    br.done();
    ++h->launches;
    return NOLO_OK;
}

int nolo_route_backward(nolo_handle* h, uint64_t seed, uint64_t step, const void* grads, void* grads_out) {
    if (!h) return NOLO_EINVAL;
    if (!h->route_bound) return fail(h, NOLO_ESTATE, "nolo_bind_route has not been called");
    if (h->stages == 1) return NOLO_OK;
    if (!grads || !grads_out) return fail(h, NOLO_EINVAL, "grads and grads_out must not be NULL");
    if (!aligned16(grads) || !aligned16(grads_out)) return fail(h, NOLO_EALIGN, "pointers must be 16-byte aligned");
    if (overlap(grads, route_bytes(h), grads_out, route_bytes(h)))
        return fail(h, NOLO_EINVAL, "grads overlaps grads_out");
    return enqueue_route(h, seed, step, grads, grads_out, 1);
}

int nolo_route_host(nolo_handle* h, uint64_t seed, uint64_t step, const void* acts_host,
                    void* out_host, void* acts_dev) {
    if (!h) return NOLO_EINVAL;
    if (!h->route_bound) return fail(h, NOLO_ESTATE, "nolo_bind_route has not been called");
    if (h->stages == 1) return NOLO_OK;
    if (!acts_host || !out_host || !acts_dev) return fail(h, NOLO_EINVAL, "pointers must not be NULL");
    if (!aligned16(acts_dev)) return fail(h, NOLO_EALIGN, "acts_dev must be 16-byte aligned");
    const size_t bytes = route_bytes(h);
    if (overlap(acts_dev, bytes, h->acts_out, bytes)) return fail(h, NOLO_EINVAL, "acts_dev overlaps acts_out");
    NOLO_CUDA(h, cudaMemcpyAsync(acts_dev, acts_host, bytes, cudaMemcpyHostToDevice, h->stream));
    int rc = enqueue_route(h, seed, step, acts_dev, h->acts_out, 0);
    if (rc != NOLO_OK) return rc;
    NOLO_CUDA(h, cudaMemcpyAsync(out_host, h->acts_out, bytes, cudaMemcpyDeviceToHost, h->stream));
    NOLO_CUDA(h, cudaStreamSynchronize(h->stream));
    return NOLO_OK;
}

int nolo_get_groups(nolo_handle* h, int32_t* host_out) {
    if (!h) return NOLO_EINVAL;
    if (!host_out) return fail(h, NOLO_EINVAL, "host_out must not be NULL");
    if (!h->groups_valid) return fail(h, NOLO_ESTATE, "no outer step has run yet");
    NOLO_CUDA(h, cudaMemcpyAsync(host_out, h->d_perm, sizeof(int32_t) * (size_t)h->W, cudaMemcpyDeviceToHost, h->stream));
    NOLO_CUDA(h, cudaStreamSynchronize(h->stream));
    return NOLO_OK;
}

int nolo_get_route(nolo_handle* h, int32_t* host_out) {
    if (!h) return NOLO_EINVAL;
    if (!host_out) return fail(h, NOLO_EINVAL, "host_out must not be NULL");
    if (!h->route_valid) return fail(h, NOLO_ESTATE, "no route call has run yet");
    const size_t bytes = sizeof(int32_t) * (size_t)(h->stages - 1) * h->K * h->W;
    NOLO_CUDA(h, cudaMemcpyAsync(host_out, h->d_route, bytes, cudaMemcpyDeviceToHost, h->stream));
    NOLO_CUDA(h, cudaStreamSynchronize(h->stream));
    return NOLO_OK;
}

int nolo_divergence(nolo_handle* h, double* host_out) {
    if (!h) return NOLO_EINVAL;
    if (!host_out) return fail(h, NOLO_EINVAL, "host_out must not be NULL");
    if (!h->state_bound) return fail(h, NOLO_ESTATE, "nolo_bind_state has not been called");
    if (!h->d_div_partials) {
        cudaError_t e = cudaMalloc(&h->d_div_partials, (size_t)nolo::divergence_partials(h->P) * 16);
        if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&h->d_div_out), 2 * sizeof(double));
        if (e != cudaSuccess) {
            if (h->d_div_partials) { cudaFree(h->d_div_partials); h->d_div_partials = nullptr; }
            return fail(h, e == cudaErrorMemoryAllocation ? NOLO_ENOMEM : NOLO_ECUDA,
                        "divergence scratch allocation: %s", cudaGetErrorString(e));
        }
    }
    Bracket br(h, NOLO_KERNEL_DIVERGENCE);
    NOLO_CUDA(h, nolo::launch_divergence(h->phi, h->W, h->stride, h->P, h->d_div_partials, h->d_div_out, h->stream));
    br.done();
    h->launches += 2;
    NOLO_CUDA(h, cudaMemcpyAsync(host_out, h->d_div_out, 2 * sizeof(double), cudaMemcpyDeviceToHost, h->stream));
    NOLO_CUDA(h, cudaStreamSynchronize(h->stream));
    return NOLO_OK;
}

int nolo_timing_enable(nolo_handle* h, int enable) {
    if (!h) return NOLO_EINVAL;
    h->timing = enable != 0;
    return NOLO_OK;
}

int nolo_timing_read(nolo_handle* h, int kernel, double* total_ms, int64_t* launches) {
    if (!h) return NOLO_EINVAL;
    if (kernel < 0 || kernel >= kTimedKernels)
        return fail(h, NOLO_EINVAL, "unknown kernel id %d", kernel);
    if (!total_ms || !launches) return fail(h, NOLO_EINVAL, "output pointers must not be NULL");
    NOLO_CUDA(h, cudaStreamSynchronize(h->stream));
    KernelTimer& t = h->timers[kernel];
    double sum = 0.0;
    for (int i = 0; i < t.used; ++i) {
        float ms = 0.f;
        NOLO_CUDA(h, cudaEventElapsedTime(&ms, t.start[i], t.stop[i]));
        sum += ms;
    }
    *total_ms = sum;
    *launches = t.used;
    t.used = 0;
    return NOLO_OK;
}

int nolo_timing_stats(nolo_handle* h, int kernel, double* stats, int64_t* launches) {
    if (!h) return NOLO_EINVAL;
    if (kernel < 0 || kernel >= kTimedKernels) return fail(h, NOLO_EINVAL, "unknown kernel id %d", kernel);
    if (!stats || !launches) return fail(h, NOLO_EINVAL, "output pointers must not be NULL");
    NOLO_CUDA(h, cudaStreamSynchronize(h->stream));
    KernelTimer& t = h->timers[kernel];
    float* ms = new (std::nothrow) float[t.used > 0 ? t.used : 1];
    if (!ms) return fail(h, NOLO_ENOMEM, "out of host memory");
    double sum = 0.0;
    for (int i = 0; i < t.used; ++i) {
        cudaError_t e = cudaEventElapsedTime(&ms[i], t.start[i], t.stop[i]);
        if (e != cudaSuccess) { delete[] ms; return cuda_fail(h, e, "cudaEventElapsedTime"); }
        sum += ms[i];
    }
    for (int i = 1; i < t.used; ++i) {            // insertion sort: at most 4096 values
        const float v = ms[i];
        int j = i - 1;
        while (j >= 0 && ms[j] > v) { ms[j + 1] = ms[j]; --j; }
        ms[j + 1] = v;
    }
    const int n = t.used;
    stats[0] = n ? sum / n : 0.0;
    stats[1] = n ? ms[0] : 0.0;
    stats[2] = n ? (n % 2 ? ms[n / 2] : 0.5 * (ms[n / 2 - 1] + ms[n / 2])) : 0.0;
    stats[3] = n ? ms[n - 1] : 0.0;
    *launches = n;
    t.used = 0;
    delete[] ms;
    return NOLO_OK;
}

int nolo_launch_count(nolo_handle* h, int64_t* launches) {
    if (!h || !launches) return NOLO_EINVAL;
    *launches = h->launches;
    return NOLO_OK;
}

int nolo_destroy(nolo_handle* h) {
    if (!h) return NOLO_OK;
    if (h->state_bound) cudaStreamSynchronize(h->stream);
    if (h->s_in) { cudaStreamSynchronize(h->s_in); cudaStreamDestroy(h->s_in); }
    if (h->s_out) { cudaStreamSynchronize(h->s_out); cudaStreamDestroy(h->s_out); }
    if (h->ev_in) cudaEventDestroy(h->ev_in);
    if (h->ev_kernel) cudaEventDestroy(h->ev_kernel);
    if (h->ev_fence) cudaEventDestroy(h->ev_fence);
    for (auto& t : h->timers) {
        for (int i = 0; i < t.created; ++i) { cudaEventDestroy(t.start[i]); cudaEventDestroy(t.stop[i]); }
        delete[] t.start;
        delete[] t.stop;
    }
    if (h->d_perm) cudaFree(h->d_perm);
    if (h->d_route) cudaFree(h->d_route);
    if (h->d_div_partials) cudaFree(h->d_div_partials);
    if (h->d_div_out) cudaFree(h->d_div_out);
    delete h;
    return NOLO_OK;
}

int nolo_copy_probe(const void* src, void* dst, int64_t bytes, int iters, void* stream, double* ms_per_copy) {
    if (!src || !dst || bytes < 16 || bytes % 16 != 0 || iters < 1 || !ms_per_copy) return NOLO_EINVAL;
    if (!aligned16(src) || !aligned16(dst)) return NOLO_EALIGN;
    if (overlap(src, (size_t)bytes, dst, (size_t)bytes)) return NOLO_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaEvent_t a = nullptr, b = nullptr;
    cudaError_t e = cudaEventCreate(&a);
    if (e == cudaSuccess) e = cudaEventCreate(&b);
    for (int i = 0; e == cudaSuccess && i < 3; ++i) e = nolo::launch_copy_probe(src, dst, bytes, s);   // warm-up
    if (e == cudaSuccess) e = cudaEventRecord(a, s);
    for (int i = 0; e == cudaSuccess && i < iters; ++i) e = nolo::launch_copy_probe(src, dst, bytes, s);
    if (e == cudaSuccess) e = cudaEventRecord(b, s);
    if (e == cudaSuccess) e = cudaEventSynchronize(b);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (e != cudaSuccess) return NOLO_ECUDA;
    *ms_per_copy = (double)ms / iters;
    return NOLO_OK;
}

int nolo_sim_tree_allreduce(int W, double mu, double sigma, int64_t trials, uint64_t seed, void* stream,
                            double* host_stats, double* host_trials) {
    if (W < 2 || W > NOLO_MAX_WORKERS || (W & (W - 1)) || trials < 1 || trials > (int64_t(1) << 24) ||
        !std::isfinite(mu) || !std::isfinite(sigma) || sigma < 0 || !host_stats)
        return NOLO_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double* d = nullptr;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&d), sizeof(double) * ((size_t)trials + 4));
    if (e != cudaSuccess) return e == cudaErrorMemoryAllocation ? NOLO_ENOMEM : NOLO_ECUDA;
    e = nolo::launch_tree_allreduce(W, mu, sigma, trials, seed, d + 4, d, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(host_stats, d, 2 * sizeof(double), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && host_trials)
        e = cudaMemcpyAsync(host_trials, d + 4, sizeof(double) * (size_t)trials, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(d);
    return e == cudaSuccess ? NOLO_OK : NOLO_ECUDA;
}

int nolo_sim_straggler(int W, int n, int H, int T, double mu, double sigma, int64_t trials, uint64_t seed,
                       void* stream, double* host_stats, double* host_trials) {
    if (W < 1 || W > NOLO_MAX_WORKERS || n < 1 || n > W || W % n != 0 || H < 1 || T < 1 || trials < 1 ||
        trials > (int64_t(1) << 20) || !std::isfinite(mu) || !std::isfinite(sigma) || sigma < 0 || !host_stats)
        return NOLO_EINVAL;
    // One launch draws W*H*T samples per trial; a mistyped H or T must not occupy the GPU for hours.
    if ((double)W * (double)H * (double)T * (double)trials > (double)NOLO_SIM_MAX_SAMPLES) return NOLO_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double* d = nullptr;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&d), sizeof(double) * (2 * (size_t)trials + 4));
    if (e != cudaSuccess) return e == cudaErrorMemoryAllocation ? NOLO_ENOMEM : NOLO_ECUDA;
    e = nolo::launch_straggler(W, n, H, T, mu, sigma, trials, seed, d + 4, d, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(host_stats, d, 4 * sizeof(double), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && host_trials)
        e = cudaMemcpyAsync(host_trials, d + 4, sizeof(double) * 2 * (size_t)trials, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(d);
    return e == cudaSuccess ? NOLO_OK : NOLO_ECUDA;
}

double nolo_expected_pair_exchange(double mu, double sigma) {
    return 2.0 * (1.0 + std::erf(sigma / 2.0)) * std::exp(mu + sigma * sigma / 2.0);
}

const char* nolo_strerror(int status) {
    switch (status) {
        case NOLO_OK: return "ok";
        case NOLO_EINVAL: return "invalid argument";
        case NOLO_ESTATE: return "required buffers are not bound or no result exists yet";
        case NOLO_EALIGN: return "pointer or stride is not aligned as required";
        case NOLO_ECUDA: return "CUDA runtime error";
        case NOLO_ENOMEM: return "out of memory";
        default: return "unknown status";
    }
}

const char* nolo_last_error(nolo_handle* h) { return h ? h->err : ""; }

int nolo_version(void) { return 200; }

}  // extern "C"

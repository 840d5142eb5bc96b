// nolo_outer_step_static: the outer step for callers that must not allocate.
//
// The handle-based path keeps its subgroup table in memory obtained with cudaMalloc when the
// handle is created.  Some callers cannot do that: a trainer that handed the whole device to its
// own memory pool at start-up (a later cudaMalloc fails or fragments the pool), a process that runs
// under a fixed device-memory budget, or a latency-critical loop in which the device-wide
// synchronisation hidden in cudaMalloc/cudaFree is not acceptable.  For them the table lives in a
// fixed array in the library's own device image, and this entry point performs no allocation of any
// kind, on the device or on the host.
#include "nolo.h"
#include "nolo_internal.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <mutex>

namespace {

// The subgroup table of the most recent call.  Lives in every device context that loads the
// library, until the process exits: NOLO_STATIC_MAX_WORKERS * 4 bytes = 4 KiB per GPU.
static __device__ __align__(256) int32_t g_static_perm[NOLO_STATIC_MAX_WORKERS];

constexpr int kMaxDevices = 64;
int32_t* g_perm_addr[kMaxDevices];   // device address of g_static_perm on each device, once resolved
std::mutex g_setup_mutex;

int report(char* err, int err_len, int code, const char* fmt, ...) {
    if (err && err_len > 0) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(err, (size_t)err_len, fmt, ap);
        va_end(ap);
    }
    return code;
}

// In host code the name g_static_perm is only a stand-in for the symbol, not a device address, so
// it must never be handed to a kernel.  The real address on the current device comes from
// cudaGetSymbolAddress, once per device.
int resolve_scratch(int32_t** out, char* err, int err_len) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return report(err, err_len, NOLO_ECUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices)
        return report(err, err_len, NOLO_EINVAL, "device ordinal %d is outside 0..%d", dev, kMaxDevices - 1);
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_perm_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_perm);
        if (e != cudaSuccess || !p)
            return report(err, err_len, NOLO_ECUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        g_perm_addr[dev] = static_cast<int32_t*>(p);
    }
    *out = g_perm_addr[dev];
    return NOLO_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool overlap(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + nb && y < x + na;
}

}  // namespace

extern "C" int nolo_outer_step_static(int W, int n, int64_t P, float alpha, float beta, float gamma,
                                      void* phi, void* theta, void* delta, int theta_dtype,
                                      int64_t row_stride, uint64_t seed, uint64_t step, void* stream,
                                      char* err, int err_len) {
    if (err && err_len > 0) err[0] = '\0';
    if (W > NOLO_STATIC_MAX_WORKERS)
        return report(err, err_len, NOLO_EINVAL,
                      "W = %d exceeds the %d workers the built-in subgroup table holds; use nolo_create / "
                      "nolo_outer_step for larger W", W, NOLO_STATIC_MAX_WORKERS);
    if (W < 1 || n < 1 || n > W || W % n != 0 || P < 1)
        return report(err, err_len, NOLO_EINVAL, "need W >= 1, 1 <= n <= W, n dividing W, P >= 1");
    if (!std::isfinite(alpha) || !std::isfinite(beta) || !std::isfinite(gamma))
        return report(err, err_len, NOLO_EINVAL, "alpha, beta and gamma must be finite");
    if (!phi || !theta || !delta) return report(err, err_len, NOLO_EINVAL, "state pointers must not be NULL");
    if (theta_dtype != NOLO_F32 && theta_dtype != NOLO_BF16)
        return report(err, err_len, NOLO_EINVAL, "theta_dtype must be NOLO_F32 or NOLO_BF16");
    if (row_stride < P) return report(err, err_len, NOLO_EINVAL, "row_stride < P");
    if (row_stride % 8 != 0) return report(err, err_len, NOLO_EALIGN, "row_stride must be a multiple of 8 elements");
    if (!aligned16(phi) || !aligned16(theta) || !aligned16(delta))
        return report(err, err_len, NOLO_EALIGN, "state pointers must be 16-byte aligned");
    const size_t n4 = (size_t)W * row_stride * 4;
    const size_t nt = (size_t)W * row_stride * (theta_dtype == NOLO_BF16 ? 2 : 4);
    if (overlap(phi, n4, delta, n4) || overlap(phi, n4, theta, nt) || overlap(delta, n4, theta, nt))
        return report(err, err_len, NOLO_EINVAL, "state buffers overlap");

    int32_t* perm = nullptr;
    const int rc = resolve_scratch(&perm, err, err_len);
    if (rc != NOLO_OK) return rc;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The draw overwrites entries 0..W-1, all that the step reads: nothing has to start at zero.
    cudaError_t e = nolo::launch_draw(seed, step, nolo::kDomainGroups, W, 1, 1, 1, perm, s);
    if (e != cudaSuccess) return report(err, err_len, NOLO_ECUDA, "subgroup draw launch: %s", cudaGetErrorString(e));
    nolo::OuterArgs a;
    a.phi = static_cast<float*>(phi);
    a.theta = theta;
    a.delta = static_cast<float*>(delta);
    a.perm = perm;
    a.stride = row_stride;
    a.P = P;
    a.W = W;
    a.n = n;
    a.theta_bf16 = theta_dtype == NOLO_BF16;
    a.alpha = alpha; a.beta = beta; a.gamma = gamma;
    e = nolo::launch_outer(a, s);
    if (e != cudaSuccess) return report(err, err_len, NOLO_ECUDA, "outer step launch: %s", cudaGetErrorString(e));
    return NOLO_OK;
}

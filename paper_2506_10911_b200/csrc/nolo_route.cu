// Random pipeline routing (Section 3.1, Algorithm 1) as a permutation gather of micro-batch
// activations between the replicas of consecutive stages.  A pure copy: every byte is read once
// and written once, 128 bits per access, streaming cache policy.
//
//   forward :  out[b][r][k][:] = in[b][table[b][k][r]][k][:]
//   backward:  out[b][table[b][k][r]][k][:] = in[b][r][k][:]     (same path, reversed)
#include "nolo_internal.h"

namespace nolo {

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;                      // 128-bit loads in flight per thread (routing: 4 measured 15 % above 2)
constexpr int kTileVecs = kThreads * kVecPerThread;   // vectors per tile

struct Blocks {
    int64_t src, dst;   // block indices into [B][R][K]
};

__device__ __forceinline__ Blocks resolve(int64_t blk, const int32_t* __restrict__ table, int R, int K,
                                          int backward) {
    const int k = (int)(blk % K);
    const int r = (int)((blk / K) % R);
    const int64_t b = blk / ((int64_t)K * R);
    const int peer = __ldg(table + (b * K + k) * R + r);
    const int64_t other = (b * R + peer) * K + k;
    Blocks o;
    o.src = backward ? blk : other;
    o.dst = backward ? other : blk;
    return o;
}

// Blocks of `vecs` 16-byte vectors each; tiles of kTileVecs vectors; one tile per CTA.
__global__ void __launch_bounds__(kThreads)
route_copy16_kernel(const uint4* __restrict__ in, uint4* __restrict__ out,
                    const int32_t* __restrict__ table, int R, int K, int64_t vecs,
                    int64_t tiles_per_block, int64_t total_tiles, int backward) {
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int64_t blk = tile / tiles_per_block;
        const int64_t v0 = (tile - blk * tiles_per_block) * kTileVecs + threadIdx.x;
        const Blocks w = resolve(blk, table, R, K, backward);
        const uint4* s = in + w.src * vecs;
        uint4* d = out + w.dst * vecs;
        uint4 v[kVecPerThread];
#pragma unroll
        for (int i = 0; i < kVecPerThread; ++i) {
            const int64_t x = v0 + (int64_t)i * kThreads;
            if (x < vecs) v[i] = __ldcs(s + x);
        }
#pragma unroll
        for (int i = 0; i < kVecPerThread; ++i) {
            const int64_t x = v0 + (int64_t)i * kThreads;
            if (x < vecs) __stcs(d + x, v[i]);
        }
    }
}

// Fallback for blocks whose byte size is not a multiple of 16: element-wise copy.
template <typename T>
__global__ void __launch_bounds__(kThreads)
route_copy_elem_kernel(const T* __restrict__ in, T* __restrict__ out, const int32_t* __restrict__ table,
                       int R, int K, int64_t E, int64_t tiles_per_block, int64_t total_tiles,
                       int backward) {
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int64_t blk = tile / tiles_per_block;
        const int64_t e0 = (tile - blk * tiles_per_block) * kTileVecs + threadIdx.x;
        const Blocks w = resolve(blk, table, R, K, backward);
        const T* s = in + w.src * E;
        T* d = out + w.dst * E;
#pragma unroll
        for (int i = 0; i < kVecPerThread; ++i) {
            const int64_t x = e0 + (int64_t)i * kThreads;
            if (x < E) d[x] = s[x];
        }
    }
}

// Plain device-to-device copy, a one-shot grid of 128-bit streaming loads and stores like the
// routing copy: the yardstick the other kernels are compared with.  Two vectors per thread is the
// fastest plain copy found on B200 (6.97 TB/s against 6.90 with four and 6.87 with eight; 256-bit
// loads and stores gave the same 6.9-7.0).
constexpr int kProbeVecPerThread = 2;
constexpr int kProbeTileVecs = kThreads * kProbeVecPerThread;

__global__ void __launch_bounds__(kThreads)
copy_probe_kernel(const uint4* __restrict__ in, uint4* __restrict__ out, int64_t vecs) {
    const int64_t v0 = (int64_t)blockIdx.x * kProbeTileVecs + threadIdx.x;
    uint4 v[kProbeVecPerThread];
#pragma unroll
    for (int i = 0; i < kProbeVecPerThread; ++i) {
        const int64_t x = v0 + (int64_t)i * kThreads;
        if (x < vecs) v[i] = __ldcs(in + x);
    }
#pragma unroll
    for (int i = 0; i < kProbeVecPerThread; ++i) {
        const int64_t x = v0 + (int64_t)i * kThreads;
        if (x < vecs) __stcs(out + x, v[i]);
    }
}

// One CTA per tile (a one-shot grid streams through memory in address order, which measured
// about 10 % faster on B200 than a resident grid striding over the tiles); the kernels still loop
// so that a tile count beyond the grid limit stays correct.
int tile_grid(int64_t total_tiles) {
    return (int)(total_tiles < 0x7fffffffll ? total_tiles : 0x7fffffffll);
}

}  // namespace

cudaError_t launch_copy_probe(const void* in, void* out, int64_t bytes, cudaStream_t stream) {
    const int64_t vecs = bytes / 16;
    const int64_t tiles = (vecs + kProbeTileVecs - 1) / kProbeTileVecs;
    if (tiles <= 0) return cudaSuccess;
    if (tiles > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    copy_probe_kernel<<<(unsigned)tiles, kThreads, 0, stream>>>(static_cast<const uint4*>(in),
                                                                static_cast<uint4*>(out), vecs);
    return cudaGetLastError();
}

cudaError_t launch_route(const RouteArgs& a, cudaStream_t stream) {
    const int64_t blocks = (int64_t)a.B * a.R * a.K;
    if (blocks <= 0 || a.E <= 0) return cudaSuccess;
    const int64_t bytes = a.E * a.elem_size;
    if (bytes % 16 == 0) {
        const int64_t vecs = bytes / 16;
        const int64_t tpb = (vecs + kTileVecs - 1) / kTileVecs;
        const int64_t total = tpb * blocks;
        route_copy16_kernel<<<tile_grid(total), kThreads, 0, stream>>>(
            static_cast<const uint4*>(a.in), static_cast<uint4*>(a.out), a.table, a.R, a.K, vecs, tpb,
            total, a.backward);
    } else {
        const int64_t tpb = (a.E + kTileVecs - 1) / kTileVecs;
        const int64_t total = tpb * blocks;
        const int grid = tile_grid(total);
        if (a.elem_size == 4)
            route_copy_elem_kernel<uint32_t><<<grid, kThreads, 0, stream>>>(
                static_cast<const uint32_t*>(a.in), static_cast<uint32_t*>(a.out), a.table, a.R, a.K,
                a.E, tpb, total, a.backward);
        else
            route_copy_elem_kernel<uint16_t><<<grid, kThreads, 0, stream>>>(
                static_cast<const uint16_t*>(a.in), static_cast<uint16_t*>(a.out), a.table, a.R, a.K,
                a.E, tpb, total, a.backward);
    }
    return cudaGetLastError();
}

}  // namespace nolo

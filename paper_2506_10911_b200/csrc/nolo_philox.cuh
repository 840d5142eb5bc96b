// Philox-4x64-10 counter-based generator (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
// easy as 1, 2, 3", SC'11) for device code.  Integer arithmetic only.
#pragma once

#include <stdint.h>

namespace nolo {

struct Philox4 {
    uint64_t w0, w1, w2, w3;
};

// Published Philox4x64 multipliers and Weyl key increments.
constexpr uint64_t kPhiloxM0 = 0xD2E7470EE14C6C93ull;
constexpr uint64_t kPhiloxM1 = 0xCA5A826395121157ull;
constexpr uint64_t kPhiloxW0 = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kPhiloxW1 = 0xBB67AE8584CAA73Bull;

__device__ __forceinline__ Philox4 philox4x64_10(uint64_t c0, uint64_t c1, uint64_t c2, uint64_t c3,
                                                 uint64_t k0, uint64_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t hi0 = __umul64hi(kPhiloxM0, c0), lo0 = kPhiloxM0 * c0;
        const uint64_t hi1 = __umul64hi(kPhiloxM1, c2), lo1 = kPhiloxM1 * c2;
        const uint64_t n0 = hi1 ^ c1 ^ k0;
        const uint64_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += kPhiloxW0; k1 += kPhiloxW1;
    }
    Philox4 o;
    o.w0 = c0; o.w1 = c1; o.w2 = c2; o.w3 = c3;
    return o;
}

// Sort key of element i of a permutation draw: counter (i, boundary, slot, domain), key (seed, step).
__device__ __forceinline__ uint64_t draw_key(uint64_t i, uint64_t boundary, uint64_t slot, uint64_t domain,
                                             uint64_t seed, uint64_t step) {
    return philox4x64_10(i, boundary, slot, domain, seed, step).w0;
}

}  // namespace nolo

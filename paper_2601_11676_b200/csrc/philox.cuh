// Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11), device side.
#pragma once
#include <stdint.h>

namespace halo {

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t (&out)[4]) {
    constexpr uint32_t kMul0 = 0xD2511F53u, kMul1 = 0xCD9E8D57u;
    constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(kMul0, c0), lo0 = kMul0 * c0;
        const uint32_t hi1 = __umulhi(kMul1, c2), lo1 = kMul1 * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += kWeyl0; k1 += kWeyl1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Arrival of virtual device `dev` at (step, layer): word 0 against the 33-bit loss threshold.
__device__ __forceinline__ bool device_arrives(uint32_t seed_lo, uint32_t seed_hi, uint32_t step, uint32_t layer,
                                               uint32_t dev, unsigned long long loss_thresh) {
    uint32_t r[4];
    philox4x32_10(step, layer, dev, 0u, seed_lo, seed_hi, r);
    return static_cast<unsigned long long>(r[0]) >= loss_thresh;
}

}  // namespace halo

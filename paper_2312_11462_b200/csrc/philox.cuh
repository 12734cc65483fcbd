// Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11), device side.
#pragma once
#include <stdint.h>

namespace csd {

struct Philox4 { uint32_t w[4]; };

__host__ __device__ inline Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                  uint32_t k0, uint32_t k1) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        uint64_t a = (uint64_t)M0 * c0;
        uint64_t b = (uint64_t)M1 * c2;
        uint32_t hi_a = (uint32_t)(a >> 32), lo_a = (uint32_t)a;
        uint32_t hi_b = (uint32_t)(b >> 32), lo_b = (uint32_t)b;
        uint32_t t0 = hi_b ^ c1 ^ k0;
        uint32_t t2 = hi_a ^ c3 ^ k1;
        c0 = t0; c1 = lo_b; c2 = t2; c3 = lo_a;
        k0 += W0; k1 += W1;
    }
    Philox4 r;
    r.w[0] = c0; r.w[1] = c1; r.w[2] = c2; r.w[3] = c3;
    return r;
}

// uniform in [0,1) from the top 24 bits of a word
__host__ __device__ inline double word_uniform(uint32_t w) { return (double)(w >> 8) * (1.0 / 16777216.0); }

}  // namespace csd

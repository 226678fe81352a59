// Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11) and the
// minibatch index draw of Algorithm 1 step 2.  Integer arithmetic only.
#pragma once
#include <stdint.h>

namespace dpsgd {

struct Philox4 { uint32_t v[4]; };

__host__ __device__ __forceinline__ void philox_mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
    const uint64_t p = (uint64_t)a * (uint64_t)b;
    hi = (uint32_t)(p >> 32);
    lo = (uint32_t)p;
}

__host__ __device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                          uint32_t k0, uint32_t k1) {
    constexpr uint32_t kMul0 = 0xD2511F53u, kMul1 = 0xCD9E8D57u;
    constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0, lo0, hi1, lo1;
        philox_mulhilo(kMul0, c0, hi0, lo0);
        philox_mulhilo(kMul1, c2, hi1, lo1);
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += kWeyl0; k1 += kWeyl1;
    }
    Philox4 out;
    out.v[0] = c0; out.v[1] = c1; out.v[2] = c2; out.v[3] = c3;
    return out;
}

// Draw b of node i at iteration k: word (b mod 4) of the block with counter
// (b div 4, i, k_lo, k_hi), key = seed; index = floor(u * m / 2^32), uniform on [0, m).
__host__ __device__ __forceinline__ int32_t sample_index(uint64_t seed, uint64_t k, uint32_t node, uint32_t b,
                                                         uint32_t m) {
    const Philox4 r = philox4x32_10(b >> 2, node, (uint32_t)k, (uint32_t)(k >> 32), (uint32_t)seed,
                                    (uint32_t)(seed >> 32));
    const uint32_t u = r.v[b & 3];
    return (int32_t)(((uint64_t)u * (uint64_t)m) >> 32);
}

}  // namespace dpsgd

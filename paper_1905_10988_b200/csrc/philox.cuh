// Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11), device side.
// Counter layout used by this library: (low32(q), high32(q), worker, domain) where q is the
// index of a group of four consecutive elements; word w of the output belongs to element 4q+w.
#pragma once

#include "common.cuh"

namespace natcomp {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;

enum : uint32_t { kDomainCnat = 0u, kDomainDnat = 1u, kDomainSelect = 2u };

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxKeys& keys, uint32_t (&out)[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * c0;   // one 32x32->64 multiply each
        const uint64_t p1 = (uint64_t)kPhiloxM1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ keys.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ keys.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The four stream words of the element group q.
__device__ __forceinline__ void stream_words4(uint64_t q, uint32_t worker, uint32_t domain,
                                              const PhiloxKeys& keys, uint32_t (&out)[4]) {
    philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), worker, domain, keys, out);
}

// Within one tile only the low counter word changes: (high32(q), worker, domain) are fixed.
// Round 0 multiplies the fixed word c2 = worker, so after round 0 the words c0 and c1 are the
// same for every group of the tile, and so is the product of round 1 that consumes c0.  These
// are computed once per tile; a block then costs 18 wide multiplies instead of 20.
struct PhiloxTile {
    uint32_t r0_c0, r0_c1;     // c0, c1 after round 0
    uint32_t r1_hi0, r1_lo0;   // M0 * r0_c0
    uint32_t dom_k;            // domain ^ k1[0]
};

__device__ __forceinline__ PhiloxTile philox_tile(uint32_t q_hi, uint32_t worker, uint32_t domain,
                                                  const PhiloxKeys& keys) {
    PhiloxTile t;
    const uint64_t p1 = (uint64_t)kPhiloxM1 * worker;
    t.r0_c0 = (uint32_t)(p1 >> 32) ^ q_hi ^ keys.k0[0];
    t.r0_c1 = (uint32_t)p1;
    const uint64_t p0 = (uint64_t)kPhiloxM0 * t.r0_c0;
    t.r1_hi0 = (uint32_t)(p0 >> 32);
    t.r1_lo0 = (uint32_t)p0;
    t.dom_k = domain ^ keys.k1[0];
    return t;
}

// Same output as stream_words4(q, ...) for q = (q_hi << 32) | q_lo of the tile `t` was made for.
__device__ __forceinline__ void stream_words4_tile(uint32_t q_lo, const PhiloxTile& t,
                                                   const PhiloxKeys& keys, uint32_t (&out)[4]) {
    // round 0, varying half: c0 = q_lo, c3 = domain
    const uint64_t a0 = (uint64_t)kPhiloxM0 * q_lo;
    uint32_t c2 = (uint32_t)(a0 >> 32) ^ t.dom_k;
    uint32_t c3 = (uint32_t)a0;
    // round 1: c0 = t.r0_c0 (fixed), c1 = t.r0_c1 (fixed)
    const uint64_t b1 = (uint64_t)kPhiloxM1 * c2;
    uint32_t c0 = (uint32_t)(b1 >> 32) ^ t.r0_c1 ^ keys.k0[1];
    uint32_t c1 = (uint32_t)b1;
    c2 = t.r1_hi0 ^ c3 ^ keys.k1[1];
    c3 = t.r1_lo0;
#pragma unroll
    for (int r = 2; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * c0;
        const uint64_t p1 = (uint64_t)kPhiloxM1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ keys.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ keys.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

}  // namespace natcomp

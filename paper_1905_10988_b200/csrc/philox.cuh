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

}  // namespace natcomp

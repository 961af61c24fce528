// Natural compression of binary64 vectors (Sec. 2 of arXiv 1905.10988: "11 bits for the exponent
// and 1 for the sign"), for sm_100a.
//
// Code planes: exp_lo[j] = low 8 bits of the rounded 11-bit exponent field; a nibble plane with
// (sign << 3) | (exponent field >> 8), element j in nibble j mod 2 of byte j / 2: 12 bits per entry.
// The integer rule of the binary32 kernel carries over: with v = bits & 0x7FF..F and r52 a 52-bit
// random threshold, v + (~r52 & (2^52 - 1)) carries into the exponent field iff r52 < mantissa,
// i.e. with probability m; the add is suppressed for exponent fields 2046 and 2047.
// r52 = (low 23 bits of the element's domain-0 stream word) << 29 | (its domain-3 word >> 3).
//
// One warp owns a tile of 1024 entries; per step a lane takes 4 consecutive entries (one 256-bit
// load, one block of each of the two Philox streams, one 32-bit word of exponent bytes, one
// 16-bit word of nibbles).
#include "common.cuh"
#include "philox.cuh"

namespace natcomp {

constexpr uint32_t kDomainLow64 = 3u;

struct Compress64Batch {
    const double* x[NC_MAX_WORKERS];
    uint8_t* exp_lo[NC_MAX_WORKERS];
    uint8_t* hi[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

struct Planes64 {
    const uint8_t* exp_lo[NC_MAX_WORKERS];
    const uint8_t* hi[NC_MAX_WORKERS];
};

struct W8 {
    uint32_t v[8];
};

__device__ __forceinline__ W8 ld_stream_w8(const void* p) {
    W8 r;
    asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]),
                   "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}

__device__ __forceinline__ void st_stream_w8(void* p, const W8& r) {
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(r.v[0]),
                 "r"(r.v[1]), "r"(r.v[2]), "r"(r.v[3]), "r"(r.v[4]), "r"(r.v[5]), "r"(r.v[6]),
                 "r"(r.v[7])
                 : "memory");
}

__device__ __forceinline__ uint32_t stream_word_of(uint64_t j, uint32_t worker, uint32_t domain,
                                                   const PhiloxKeys& keys) {
    uint32_t r4[4];
    stream_words4(j >> 2, worker, domain, keys, r4);
    return (j & 3) == 0 ? r4[0] : (j & 3) == 1 ? r4[1] : (j & 3) == 2 ? r4[2] : r4[3];
}

// 12-bit code (sign << 11 | exponent field) of C_nat(x) for x = (hi : lo) and the two stream words
__device__ __forceinline__ uint32_t cnat64_code(uint32_t lo, uint32_t hi, uint32_t w0, uint32_t w3) {
    unsigned long long v = ((unsigned long long)(hi & 0x7FFFFFFFu) << 32) | lo;
    const unsigned long long r52 = ((unsigned long long)(w0 & 0x7FFFFFu) << 29) | (w3 >> 3);
    if ((hi & 0x7FFFFFFFu) < 0x7FE00000u) v += ~r52 & 0xFFFFFFFFFFFFFull;
    return (uint32_t)(v >> 52) | ((hi >> 31) << 11);
}

// grid: (ceil(tiles / warps per block), n workers)
__global__ void __launch_bounds__(kBlockThreads)
nc64_compress_kernel(const __grid_constant__ Compress64Batch batch, const uint64_t d,
                     const __grid_constant__ PhiloxKeys keys) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    const int w = blockIdx.y;
    const double* __restrict__ x = batch.x[w];
    uint8_t* __restrict__ exp_lo = batch.exp_lo[w];
    uint8_t* __restrict__ hi = batch.hi[w];
    const uint32_t worker = batch.worker[w];
    if (base + kTile <= d) {
        const PhiloxTile pt0 = philox_tile((uint32_t)(base >> 34), worker, kDomainCnat, keys);
        const PhiloxTile pt3 = philox_tile((uint32_t)(base >> 34), worker, kDomainLow64, keys);
        const uint32_t q_lo = (uint32_t)(base >> 2) + lane;
#pragma unroll 2
        for (int k = 0; k < 8; ++k) {
            const W8 u = ld_stream_w8(x + base + k * 128 + lane * 4);
            uint32_t r0[4], r3[4];
            stream_words4_tile(q_lo + k * 32, pt0, keys, r0);
            stream_words4_tile(q_lo + k * 32, pt3, keys, r3);
            uint32_t e = 0, nib = 0;
#pragma unroll
            for (int c = 3; c >= 0; --c) {
                const uint32_t code = cnat64_code(u.v[2 * c], u.v[2 * c + 1], r0[c], r3[c]);
                e = (e << 8) | (code & 0xFFu);
                nib = (nib << 4) | (code >> 8);
            }
            st_stream_u32(exp_lo + base + k * 128 + lane * 4, e);
            *reinterpret_cast<uint16_t*>(hi + ((base + k * 128 + lane * 4) >> 1)) = (uint16_t)nib;
        }
        return;
    }
    // ragged last tile: two entries per lane per step (one nibble byte), zero padding of both
    // planes up to a multiple of 16 bytes
    const uint64_t exp_end = round_up16(d);
    const uint64_t hi_bytes = (d + 1) / 2;
    const uint64_t hi_end = round_up16(hi_bytes);
    for (uint64_t j0 = base; j0 < exp_end || (j0 >> 1) < hi_end; j0 += 64) {
        const uint64_t j = j0 + 2 * lane;
        uint32_t nib = 0;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t code = 0;
            if (j + c < d) {
                const unsigned long long bits = (unsigned long long)__double_as_longlong(x[j + c]);
                code = cnat64_code((uint32_t)bits, (uint32_t)(bits >> 32),
                                   stream_word_of(j + c, worker, kDomainCnat, keys),
                                   stream_word_of(j + c, worker, kDomainLow64, keys));
            }
            if (j + c < exp_end) exp_lo[j + c] = (uint8_t)(code & 0xFFu);
            nib |= (code >> 8) << (4 * c);
        }
        if ((j >> 1) < hi_end) hi[j >> 1] = (uint8_t)nib;
    }
}

__device__ __forceinline__ double decode12(uint32_t e_lo, uint32_t nib) {
    const unsigned long long bits =
        ((unsigned long long)((nib << 8) | e_lo)) << 52;     // sign lands in bit 63
    return __longlong_as_double((long long)bits);
}

// grid: ceil(tiles / warps per block).  out = sum of the decoded values in worker order (from +0)
__global__ void __launch_bounds__(kBlockThreads)
nc64_aggregate_kernel(const __grid_constant__ Planes64 planes, const int n, const uint64_t d,
                      double* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    if (base + kTile <= d) {
#pragma unroll 2
        for (int k = 0; k < 8; ++k) {
            const uint64_t j = base + k * 128 + lane * 4;
            double acc[4] = {0.0, 0.0, 0.0, 0.0};
            for (int i = 0; i < n; ++i) {
                const uint32_t e = ld_stream_u32(planes.exp_lo[i] + j);
                const uint32_t nb = __ldcs(reinterpret_cast<const unsigned short*>(planes.hi[i] + (j >> 1)));
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    acc[c] = __dadd_rn(acc[c], decode12((e >> (8 * c)) & 0xFFu, (nb >> (4 * c)) & 0xFu));
            }
            W8 o;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const unsigned long long b = (unsigned long long)__double_as_longlong(acc[c]);
                o.v[2 * c] = (uint32_t)b;
                o.v[2 * c + 1] = (uint32_t)(b >> 32);
            }
            st_stream_w8(out + j, o);
        }
        return;
    }
    for (uint64_t j = base + lane; j < d; j += 32) {
        double acc = 0.0;
        for (int i = 0; i < n; ++i) {
            const uint32_t nb = (planes.hi[i][j >> 1] >> (4 * (j & 1))) & 0xFu;
            acc = __dadd_rn(acc, decode12(planes.exp_lo[i][j], nb));
        }
        out[j] = acc;
    }
}

}  // namespace natcomp

using namespace natcomp;

extern "C" {

nc_status nc64_compress_batch(const double* const* xs, size_t d, uint64_t seed,
                              const uint32_t* workers, uint8_t* const* exp_los,
                              uint8_t* const* his, int n, cudaStream_t stream) {
    if (!xs || !workers || !exp_los || !his || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    Compress64Batch batch;
    for (int i = 0; i < n; ++i) {
        if (!xs[i] || !exp_los[i] || !his[i]) return NC_ERR_INVALID;
        if (!aligned32(xs[i]) || !aligned16(exp_los[i]) || !aligned16(his[i])) return NC_ERR_ALIGN;
        batch.x[i] = xs[i];
        batch.exp_lo[i] = exp_los[i];
        batch.hi[i] = his[i];
        batch.worker[i] = workers[i];
    }
    const uint64_t tiles = (d + kTile - 1) / kTile;
    const dim3 grid((unsigned)((tiles + kWarpsPerBlock - 1) / kWarpsPerBlock), (unsigned)n);
    nc64_compress_kernel<<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d,
                                                             make_philox_keys(seed));
    return launch_status();
}

nc_status nc64_compress(const double* x, size_t d, uint64_t seed, uint32_t worker, uint8_t* exp_lo,
                        uint8_t* hi, cudaStream_t stream) {
    return nc64_compress_batch(&x, d, seed, &worker, &exp_lo, &hi, 1, stream);
}

nc_status nc64_aggregate(const uint8_t* const* exp_los, const uint8_t* const* his, int n, size_t d,
                         double* out, cudaStream_t stream) {
    if (!exp_los || !his || !out || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned32(out)) return NC_ERR_ALIGN;
    Planes64 planes;
    for (int i = 0; i < n; ++i) {
        if (!exp_los[i] || !his[i]) return NC_ERR_INVALID;
        if (!aligned16(exp_los[i]) || !aligned16(his[i])) return NC_ERR_ALIGN;
        planes.exp_lo[i] = exp_los[i];
        planes.hi[i] = his[i];
    }
    const uint64_t tiles = (d + kTile - 1) / kTile;
    nc64_aggregate_kernel<<<(unsigned)((tiles + kWarpsPerBlock - 1) / kWarpsPerBlock),
                            kBlockThreads, 0, stream>>>(planes, n, (uint64_t)d, out);
    return launch_status();
}

}  // extern "C"

// C_nat (Def. 1 of arXiv 1905.10988) of binary16 vectors with 10-bit thresholds, for sm_100a.
//
// A binary16 value has at most 10 mantissa bits, so its up-probability m is a multiple of 1/1024
// and 10 random bits decide the rounding exactly.  Entry j draws the low 10 bits of half-word
// (j mod 2) of stream word j / 2 of domain 5, so one generator block serves 8 entries.  The value
// is converted exactly to binary32 (a binary16 subnormal becomes a normal number); its threshold
// m * 2^23 is a multiple of 2^13, so "up" iff r10 * 2^13 < mantissa field, which is the carry of
// bits + ((~r10 & 1023) << 13) into the exponent.  Output: the binary32 exponent-byte and sign-bit
// planes.
//
// A warp owns a tile of 1024 entries: 4 steps of 256; per step a lane takes 8 consecutive entries
// (one 128-bit load, one generator block, 8 exponent bytes, 8 sign bits).
#include <cuda_fp16.h>

#include "common.cuh"
#include "philox.cuh"

namespace natcomp {

constexpr uint32_t kDomainF16Halves = 5u;

struct CompressF16Batch {
    const uint16_t* x[NC_MAX_WORKERS];
    uint8_t* exp[NC_MAX_WORKERS];
    uint32_t* sign[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

// exponent byte of C_nat(value of the binary16 pattern whose exact binary32 magnitude bits are
// `mag`) for the 10-bit draw in bits 13..22 of `inv` (already complemented)
__device__ __forceinline__ uint32_t cnat_f16_exp(uint32_t mag, uint32_t inv) {
    // inf and NaN (mag >= 0x7F800000) may carry past the exponent field: clamp to 255
    return min((mag + inv) >> 23, 255u);
}

// two entries (one 32-bit word of two binary16 values) and their stream word: two exponent bytes
// in bits 0..7 and 8..15
__device__ __forceinline__ uint32_t cnat_f16_x2(uint32_t w, uint32_t rnd) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
    const uint32_t inv_lo = (~rnd << 13) & 0x7FE000u;
    const uint32_t inv_hi = (~rnd >> 3) & 0x7FE000u;
    const uint32_t e0 = cnat_f16_exp(__float_as_uint(f.x) & 0x7FFFFFFFu, inv_lo);
    const uint32_t e1 = cnat_f16_exp(__float_as_uint(f.y) & 0x7FFFFFFFu, inv_hi);
    return e0 | (e1 << 8);
}

// grid: (ceil(tiles / warps per block), n workers)
__global__ void __launch_bounds__(kBlockThreads)
nc_compress_f16_r16_kernel(const __grid_constant__ CompressF16Batch batch, const uint64_t d,
                           const __grid_constant__ PhiloxKeys keys) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    const int w = blockIdx.y;
    const uint16_t* __restrict__ x = batch.x[w];
    uint8_t* __restrict__ exp = batch.exp[w];
    uint32_t* __restrict__ sign = batch.sign[w];
    const uint32_t worker = batch.worker[w];

    if (base + kTile <= d) {
        uint4 u[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) u[k] = ld_stream_u4(x + base + k * 256 + lane * 8);
        // generator block q = j / 8; within a tile only the low counter word changes
        const PhiloxTile pt = philox_tile((uint32_t)(base >> 35), worker, kDomainF16Halves, keys);
        const uint32_t q_lo = (uint32_t)(base >> 3) + lane;
        uint32_t sbytes = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t rnd[4];
            stream_words4_tile(q_lo + k * 32, pt, keys, rnd);
            uint2 e;
            e.x = cnat_f16_x2(u[k].x, rnd[0]) | (cnat_f16_x2(u[k].y, rnd[1]) << 16);
            e.y = cnat_f16_x2(u[k].z, rnd[2]) | (cnat_f16_x2(u[k].w, rnd[3]) << 16);
            __stcs(reinterpret_cast<uint2*>(exp + base + k * 256 + lane * 8), e);
            // sign bits of the 8 entries: the high bytes of the 8 half-words, bit 7 of each
            const uint32_t s_lo = __byte_perm(u[k].x, u[k].y, 0x7531) & 0x80808080u;
            const uint32_t s_hi = __byte_perm(u[k].z, u[k].w, 0x7531) & 0x80808080u;
            const uint32_t s8 = ((s_lo * 0x00204081u) >> 28) | (((s_hi * 0x00204081u) >> 28) << 4);
            sbytes |= s8 << (8 * k);
        }
        // lane 4g+i holds byte i of sign word (k, g) = word k*8 + g of the tile
        const uint32_t word = transpose_bytes_4x4(sbytes, lane);
        st_stream_u32(sign + (base >> 5) + (lane & 3) * 8 + (lane >> 2), word);
        return;
    }

    // ragged last tile, one entry per lane per step (a ballot gives the sign word); also writes
    // the zero padding of both planes
    const uint64_t exp_end = round_up16(d);
    const uint64_t sign_words = (d + 31) / 32;
    const uint64_t sign_words_padded = (sign_words + 3) & ~(uint64_t)3;
    for (uint64_t j0 = base; j0 < exp_end; j0 += 32) {
        const uint64_t j = j0 + lane;
        uint32_t e = 0, sgn = 0;
        if (j < d) {
            uint32_t rnd[4];
            stream_words4(j >> 3, worker, kDomainF16Halves, keys, rnd);
            const int c = (int)((j >> 1) & 3);
            const uint32_t word = c == 0 ? rnd[0] : c == 1 ? rnd[1] : c == 2 ? rnd[2] : rnd[3];
            const uint32_t r10 = (word >> (16 * (j & 1))) & 0x3FFu;
            const uint32_t h = x[j];
            const uint32_t mag =
                __float_as_uint(__half2float(__ushort_as_half((unsigned short)h))) & 0x7FFFFFFFu;
            e = cnat_f16_exp(mag, (~r10 & 0x3FFu) << 13);
            sgn = h >> 15;
        }
        if (j < exp_end) exp[j] = (uint8_t)e;
        const uint32_t ballot = __ballot_sync(0xFFFFFFFFu, sgn != 0);
        if (lane == 0 && (j0 >> 5) < sign_words) sign[j0 >> 5] = ballot;
    }
    if (lane < (int)(sign_words_padded - sign_words)) sign[sign_words + lane] = 0;
}

}  // namespace natcomp

using namespace natcomp;

extern "C" {

nc_status nc_compress_f16_r16_batch(const void* const* xs, size_t d, uint64_t seed,
                                    const uint32_t* workers, uint8_t* const* exps,
                                    uint32_t* const* signs, int n, cudaStream_t stream) {
    if (!xs || !workers || !exps || !signs || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    CompressF16Batch batch;
    for (int i = 0; i < n; ++i) {
        if (!xs[i] || !exps[i] || !signs[i]) return NC_ERR_INVALID;
        if (!aligned32(xs[i]) || !aligned16(exps[i]) || !aligned16(signs[i])) return NC_ERR_ALIGN;
        batch.x[i] = static_cast<const uint16_t*>(xs[i]);
        batch.exp[i] = exps[i];
        batch.sign[i] = signs[i];
        batch.worker[i] = workers[i];
    }
    const uint64_t tiles = (d + kTile - 1) / kTile;
    const dim3 grid((unsigned)((tiles + kWarpsPerBlock - 1) / kWarpsPerBlock), (unsigned)n);
    nc_compress_f16_r16_kernel<<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d,
                                                                   make_philox_keys(seed));
    return launch_status();
}

nc_status nc_compress_f16_r16(const void* x, size_t d, uint64_t seed, uint32_t worker,
                              uint8_t* exp, uint32_t* sign, cudaStream_t stream) {
    return nc_compress_f16_r16_batch(&x, d, seed, &worker, &exp, &sign, 1, stream);
}

}  // extern "C"

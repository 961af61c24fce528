// C_nat (Def. 1 of arXiv 1905.10988) of bfloat16 vectors with 7-bit thresholds, for sm_100a.
//
// A bfloat16 value has 7 mantissa bits, so its up-probability m is a multiple of 1/128 and 7
// random bits decide the rounding exactly: "up" iff r7 < (mantissa field).  Entry j draws the low
// 7 bits of byte (j mod 4) of stream word j / 4 of domain 4, so one generator block serves 16
// entries instead of 4 and the kernel is bound by memory traffic (2 bytes read, 9 bits written per
// entry), not by the generator.  Output: the same exponent-byte and sign-bit planes as for
// binary32 (the exponent ranges coincide).
//
// A warp owns a tile of 2048 entries: 4 steps of 512; per step a lane takes 16 consecutive entries
// (one 32-byte load, one generator block, one 16-byte store of exponent bytes, 16 sign bits).  The
// rounding works on four entries at a time, one per byte of a 32-bit word:
//   E = exponent fields, M = mantissa fields (7 bits), R = draws (7 bits);
//   M + (127 - R) has bit 7 set iff R < M, no carry leaves a byte; the bit is dropped where
//   E >= 254 (2^127 and above, inf, NaN are never rounded up) and added to E.
#include "common.cuh"
#include "philox.cuh"

namespace natcomp {

constexpr uint32_t kDomainBf16Bytes = 4u;
constexpr int kBf16Tile = 2048;

struct CompressBf16Batch {
    const uint16_t* x[NC_MAX_WORKERS];
    uint8_t* exp[NC_MAX_WORKERS];
    uint32_t* sign[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

struct H16 {            // 16 bfloat16 values: word i = entries 2i (low half) and 2i + 1
    uint32_t v[8];
};

__device__ __forceinline__ H16 ld_stream_h16(const void* p) {
    H16 r;
    asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]),
                   "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}

// four entries (wa = entries 0, 1; wb = entries 2, 3) and their four draw bytes `rnd`:
// returns the four rounded exponent bytes, adds the four sign bits to `signs` at bit `pos`
__device__ __forceinline__ uint32_t cnat_bf16_x4(uint32_t wa, uint32_t wb, uint32_t rnd,
                                                 uint32_t& signs, int pos) {
    const uint32_t hi = __byte_perm(wa, wb, 0x7531);       // sign + exponent bits 7..1
    const uint32_t lo = __byte_perm(wa, wb, 0x6420);       // exponent bit 0 + mantissa
    const uint32_t e = ((hi << 1) & 0xFEFEFEFEu) | ((lo >> 7) & 0x01010101u);
    const uint32_t sum = (lo & 0x7F7F7F7Fu) + (~rnd & 0x7F7F7F7Fu);
    const uint32_t top = ((e & 0x7F7F7F7Fu) + 0x02020202u) & e;      // bit 7: field >= 254
    const uint32_t up = ((sum & ~top) & 0x80808080u) >> 7;
    signs |= (((hi & 0x80808080u) * 0x00204081u) >> 28) << pos;      // bits 7,15,23,31 -> 0..3
    return e + up;
}

// code of one entry (ragged tail): exponent byte, sign bit
__device__ __forceinline__ void cnat_bf16_one(uint32_t h, uint32_t byte, uint32_t& e,
                                              uint32_t& sgn) {
    const uint32_t field = (h >> 7) & 0xFFu;
    const uint32_t up = ((byte & 0x7Fu) < (h & 0x7Fu)) && field < 254u;
    e = field + up;
    sgn = h >> 15;
}

// grid: (ceil(tiles / warps per block), n workers)
__global__ void __launch_bounds__(kBlockThreads)
nc_compress_bf16_r8_kernel(const __grid_constant__ CompressBf16Batch batch, const uint64_t d,
                           const __grid_constant__ PhiloxKeys keys) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kBf16Tile;
    if (base >= d) return;
    const int w = blockIdx.y;
    const uint16_t* __restrict__ x = batch.x[w];
    uint8_t* __restrict__ exp = batch.exp[w];
    uint32_t* __restrict__ sign = batch.sign[w];
    const uint32_t worker = batch.worker[w];

    if (base + kBf16Tile <= d) {
        H16 u[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) u[k] = ld_stream_h16(x + base + k * 512 + lane * 16);
        // generator block q = j / 16; within a tile only the low counter word changes
        const PhiloxTile pt = philox_tile((uint32_t)(base >> 36), worker, kDomainBf16Bytes, keys);
        const uint32_t q_lo = (uint32_t)(base >> 4) + lane;
        uint32_t s16[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t rnd[4];
            stream_words4_tile(q_lo + k * 32, pt, keys, rnd);
            uint32_t signs = 0;
            uint4 e;
            e.x = cnat_bf16_x4(u[k].v[0], u[k].v[1], rnd[0], signs, 0);
            e.y = cnat_bf16_x4(u[k].v[2], u[k].v[3], rnd[1], signs, 4);
            e.z = cnat_bf16_x4(u[k].v[4], u[k].v[5], rnd[2], signs, 8);
            e.w = cnat_bf16_x4(u[k].v[6], u[k].v[7], rnd[3], signs, 12);
            st_stream_u4(exp + base + k * 512 + lane * 16, e);
            s16[k] = signs;
        }
        // a sign word covers two neighbouring lanes of one step: the even lane assembles the
        // word of the even step, the odd lane that of the odd step
        const bool odd = lane & 1;
#pragma unroll
        for (int k = 0; k < 4; k += 2) {
            const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, odd ? s16[k] : s16[k + 1], 1);
            const uint32_t word = odd ? (got | (s16[k + 1] << 16)) : (s16[k] | (got << 16));
            st_stream_u32(sign + (base >> 5) + (k + (odd ? 1 : 0)) * 16 + (lane >> 1), word);
        }
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
            stream_words4(j >> 4, worker, kDomainBf16Bytes, keys, rnd);
            const int c = (int)((j >> 2) & 3);
            const uint32_t word = c == 0 ? rnd[0] : c == 1 ? rnd[1] : c == 2 ? rnd[2] : rnd[3];
            cnat_bf16_one(x[j], word >> (8 * (j & 3)), e, sgn);
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

nc_status nc_compress_bf16_r8_batch(const void* const* xs, size_t d, uint64_t seed,
                                    const uint32_t* workers, uint8_t* const* exps,
                                    uint32_t* const* signs, int n, cudaStream_t stream) {
    if (!xs || !workers || !exps || !signs || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    CompressBf16Batch batch;
    for (int i = 0; i < n; ++i) {
        if (!xs[i] || !exps[i] || !signs[i]) return NC_ERR_INVALID;
        if (!aligned32(xs[i]) || !aligned16(exps[i]) || !aligned16(signs[i])) return NC_ERR_ALIGN;
        batch.x[i] = static_cast<const uint16_t*>(xs[i]);
        batch.exp[i] = exps[i];
        batch.sign[i] = signs[i];
        batch.worker[i] = workers[i];
    }
    const uint64_t tiles = (d + kBf16Tile - 1) / kBf16Tile;
    const dim3 grid((unsigned)((tiles + kWarpsPerBlock - 1) / kWarpsPerBlock), (unsigned)n);
    nc_compress_bf16_r8_kernel<<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d,
                                                                   make_philox_keys(seed));
    return launch_status();
}

nc_status nc_compress_bf16_r8(const void* x, size_t d, uint64_t seed, uint32_t worker,
                              uint8_t* exp, uint32_t* sign, cudaStream_t stream) {
    return nc_compress_bf16_r8_batch(&x, d, seed, &worker, &exp, &sign, 1, stream);
}

}  // extern "C"

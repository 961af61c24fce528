// Natural compression C_nat (Def. 1 / Sec. 2 of arXiv 1905.10988) and the master-side
// aggregation of Algorithm 1, hand-written for sm_100a.
//
// Work decomposition: one warp owns a tile of 1024 consecutive elements.  Lane l loads the
// float4 groups k*32 + l (k = 0..7) of the tile, so every warp-wide access is one contiguous
// 512-byte (loads, fp32 stores) or 128-byte (exponent bytes, sign words) segment.  A float4
// group is exactly one Philox4x32-10 block, so no random word is computed twice.
//
// C_nat on the binary32 fields is integer-only: with v = bits & 0x7FFFFFFF and r23 the low 23
// random bits, v + (~r23 & 0x7FFFFF) carries into the exponent field iff r23 < mantissa, i.e.
// with probability m (Sec. 2: round up with probability m).  The add is suppressed for biased
// exponents 254 and 255 (saturation / inf / NaN policy).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "philox.cuh"

namespace natcomp {

struct CompressBatch {
    const float* x[NC_MAX_WORKERS];
    uint8_t* exp[NC_MAX_WORKERS];
    uint32_t* sign[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

struct PackedPlanes {
    const uint8_t* exp[NC_MAX_WORKERS];
    const uint32_t* sign[NC_MAX_WORKERS];
};

struct DensePlanes {
    const float* x[NC_MAX_WORKERS];
};

// With this value in place of the random word, "up iff r23 < mantissa" becomes "up iff the
// mantissa field is at least 2^22", i.e. rounding to the nearest power of two, ties upward.
constexpr uint32_t kNearestThreshold = 0x3FFFFFu;

// exponent byte of C_nat(bits) given the element's random word
__device__ __forceinline__ uint32_t cnat_exp_byte(uint32_t bits, uint32_t rnd) {
    uint32_t v = bits & 0x7FFFFFFFu;
    const uint32_t rr = ~rnd & 0x7FFFFFu;
    if (v < 0x7F000000u) v += rr;
    return v >> 23;
}

// C_nat of one full tile held in registers (lane l: float4 groups k*32 + l, k = 0..7):
// writes the tile's 1024 exponent bytes and 32 sign words.
template <bool kDet>
__device__ __forceinline__ void cnat_full_tile(const uint4 (&u)[8], const uint64_t base,
                                               const uint32_t worker, const PhiloxKeys& keys,
                                               uint8_t* __restrict__ exp,
                                               uint32_t* __restrict__ sign, const int lane) {
    uint32_t* ev = reinterpret_cast<uint32_t*>(exp + base);
    const PhiloxTile pt = philox_tile((uint32_t)(base >> 34), worker, kDomainCnat, keys);
    const uint32_t q_lo = (uint32_t)(base >> 2) + lane;   // + k*32 stays below 2^32: no carry

    // Biased exponents 254 / 255 must not be rounded up.  If every element of the tile has
    // (bits & 0x7F000000) != 0x7F000000 the guard can be dropped; the OR over the lane's
    // elements is a cheap conservative test (false positives only cost the guarded path).
    uint32_t any = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) any |= u[k].x | u[k].y | u[k].z | u[k].w;
    const bool guarded = __any_sync(0xFFFFFFFFu, (any & 0x7F000000u) == 0x7F000000u);

    uint32_t nib = 0;   // sign bits of this lane's 32 elements: bit 4k+c <-> group k, element c
    if (!guarded) {
#pragma unroll
        for (int k = 7; k >= 0; --k) {
            uint32_t rnd[4];
            if (kDet) rnd[0] = rnd[1] = rnd[2] = rnd[3] = kNearestThreshold;
            else stream_words4_tile(q_lo + k * 32, pt, keys, rnd);
            const uint32_t b0 = u[k].x, b1 = u[k].y, b2 = u[k].z, b3 = u[k].w;
            // (bits + (~r23 & 0x7FFFFF)) << 1: sign shifted out, rounded exponent in byte 3
            const uint32_t t0 = (b0 + (~rnd[0] & 0x7FFFFFu)) << 1;
            const uint32_t t1 = (b1 + (~rnd[1] & 0x7FFFFFu)) << 1;
            const uint32_t t2 = (b2 + (~rnd[2] & 0x7FFFFFu)) << 1;
            const uint32_t t3 = (b3 + (~rnd[3] & 0x7FFFFFu)) << 1;
            const uint32_t e = __byte_perm(__byte_perm(t0, t1, 0x0073),
                                           __byte_perm(t2, t3, 0x0073), 0x5410);
            st_stream_u32(ev + k * 32 + lane, e);
            nib = __funnelshift_l(b3, nib, 1);
            nib = __funnelshift_l(b2, nib, 1);
            nib = __funnelshift_l(b1, nib, 1);
            nib = __funnelshift_l(b0, nib, 1);
        }
    } else {
#pragma unroll
        for (int k = 7; k >= 0; --k) {
            uint32_t rnd[4];
            if (kDet) rnd[0] = rnd[1] = rnd[2] = rnd[3] = kNearestThreshold;
            else stream_words4_tile(q_lo + k * 32, pt, keys, rnd);
            const uint32_t b0 = u[k].x, b1 = u[k].y, b2 = u[k].z, b3 = u[k].w;
            uint32_t e = cnat_exp_byte(b3, rnd[3]);
            e = (e << 8) | cnat_exp_byte(b2, rnd[2]);
            e = (e << 8) | cnat_exp_byte(b1, rnd[1]);
            e = (e << 8) | cnat_exp_byte(b0, rnd[0]);
            st_stream_u32(ev + k * 32 + lane, e);
            nib = __funnelshift_l(b3, nib, 1);
            nib = __funnelshift_l(b2, nib, 1);
            nib = __funnelshift_l(b1, nib, 1);
            nib = __funnelshift_l(b0, nib, 1);
        }
    }
    // lane 8g+i holds nibble k of sign word (k, g); after the transpose lane 8g+k holds the
    // whole word covering elements k*128 + g*32 .. +31 of the tile.
    const uint32_t word = transpose_nibbles_8x8(nib, lane);
    st_stream_u32(sign + (base >> 5) + (lane & 7) * 4 + (lane >> 3), word);
}

// C_nat of the ragged last tile, one element per lane per step (a ballot gives the sign word);
// also writes the zero padding of both planes.  load_bits(j) returns the binary32 pattern of
// element j.
template <bool kDet, typename LoadBits>
__device__ __forceinline__ void cnat_ragged_tile(LoadBits load_bits, const uint64_t base,
                                                 const uint64_t d, const uint32_t worker,
                                                 const PhiloxKeys& keys, uint8_t* __restrict__ exp,
                                                 uint32_t* __restrict__ sign, const int lane) {
    const uint64_t exp_end = round_up16(d);                 // bytes incl. zero padding
    const uint64_t sign_words = (d + 31) / 32;
    const uint64_t sign_words_padded = (sign_words + 3) & ~(uint64_t)3;
    for (uint64_t j0 = base; j0 < exp_end; j0 += 32) {
        const uint64_t j = j0 + lane;
        uint32_t bits = 0, e = 0;
        if (j < d) {
            bits = load_bits(j);
            uint32_t r = kNearestThreshold;
            if (!kDet) {
                uint32_t rnd[4];
                stream_words4(j >> 2, worker, kDomainCnat, keys, rnd);
                r = (j & 3) == 0 ? rnd[0] : (j & 3) == 1 ? rnd[1] : (j & 3) == 2 ? rnd[2] : rnd[3];
            }
            e = cnat_exp_byte(bits, r);
        }
        if (j < exp_end) NC_STORE(exp + j, (uint8_t)e);
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, (bits >> 31) != 0);
        if (lane == 0 && (j0 >> 5) < sign_words) NC_STORE(sign + (j0 >> 5), word);
    }
    if (lane < (int)(sign_words_padded - sign_words)) NC_STORE(sign + sign_words + lane, 0u);
}

// grid: (ceil(tiles / warps per block), n workers).  kDet: round to the nearest power of two
// instead of drawing (the paper's "deterministic" control variant, no generator).
template <bool kDet>
__global__ void __launch_bounds__(kBlockThreads)
nc_compress_kernel(const __grid_constant__ CompressBatch batch, const uint64_t d,
                   const __grid_constant__ PhiloxKeys keys) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    const int w = blockIdx.y;
    const float* __restrict__ x = batch.x[w];
    if (base + kTile <= d) {
        const uint4* xv = reinterpret_cast<const uint4*>(x + base);
        uint4 u[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) u[k] = ld_stream_u4(xv + k * 32 + lane);
        cnat_full_tile<kDet>(u, base, batch.worker[w], keys, batch.exp[w], batch.sign[w], lane);
        return;
    }
    cnat_ragged_tile<kDet>([&](uint64_t j) { return __float_as_uint(x[j]); }, base, d,
                           batch.worker[w], keys, batch.exp[w], batch.sign[w], lane);
}

// ---- 16-bit inputs --------------------------------------------------------------------
// bfloat16 and binary16 values are binary32 values, so C_nat of such an input is the binary32
// rule applied to the exactly converted value: the up-probability m (7 or 10 mantissa bits, or a
// binary16 subnormal's fraction) is compared with r23 at full width.  Same tile layout; a lane
// loads 4 consecutive 16-bit elements (8 bytes) per step and widens them.
struct Compress16Batch {
    const uint16_t* x[NC_MAX_WORKERS];
    uint8_t* exp[NC_MAX_WORKERS];
    uint32_t* sign[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

template <int DT>
__device__ __forceinline__ uint32_t widen16(uint32_t h) {          // one element, low 16 bits
    if (DT == NC_DTYPE_BF16) return h << 16;
    // the conversion may return a canonical NaN: the sign bit is taken from the input
    const uint32_t f = __float_as_uint(__half2float(__ushort_as_half((unsigned short)h)));
    return (f & 0x7FFFFFFFu) | ((h & 0x8000u) << 16);
}

template <int DT>
__device__ __forceinline__ void widen16x2(uint32_t w, uint32_t& lo, uint32_t& hi) {
    if (DT == NC_DTYPE_BF16) {
        lo = w << 16;
        hi = w & 0xFFFF0000u;
    } else {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
        lo = (__float_as_uint(f.x) & 0x7FFFFFFFu) | ((w << 16) & 0x80000000u);   // sign of a NaN
        hi = (__float_as_uint(f.y) & 0x7FFFFFFFu) | (w & 0x80000000u);
    }
}

// grid: (ceil(tiles / warps per block), n workers)
template <int DT>
__global__ void __launch_bounds__(kBlockThreads)
nc_compress16_kernel(const __grid_constant__ Compress16Batch batch, const uint64_t d,
                     const __grid_constant__ PhiloxKeys keys) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    const int w = blockIdx.y;
    const uint16_t* __restrict__ x = batch.x[w];
    if (base + kTile <= d) {
        const uint2* xv = reinterpret_cast<const uint2*>(x + base);
        uint2 h[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) h[k] = __ldcs(xv + k * 32 + lane);
        uint4 u[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            widen16x2<DT>(h[k].x, u[k].x, u[k].y);
            widen16x2<DT>(h[k].y, u[k].z, u[k].w);
        }
        cnat_full_tile<false>(u, base, batch.worker[w], keys, batch.exp[w], batch.sign[w], lane);
        return;
    }
    cnat_ragged_tile<false>([&](uint64_t j) { return widen16<DT>(x[j]); }, base, d,
                            batch.worker[w], keys, batch.exp[w], batch.sign[w], lane);
}

// value of a 9-bit code: exponent byte in byte `BYTE` of `e4`, sign in bit `BYTE` of `s4` (4 valid
// bits, the rest zero).  The exponent byte is shifted to bits 30..23 and the sign bit to bit 31;
// one three-input logic operation takes bits 30..23 from the first and everything else from the
// second, so what the shifts drag along is dropped.
template <int BYTE>
__device__ __forceinline__ float decode9(uint32_t e4, uint32_t s4) {
    const uint32_t a = BYTE == 3 ? (e4 >> 1) : (e4 << (23 - 8 * BYTE));
    const uint32_t b = s4 << (31 - BYTE);
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(r) : "r"(0x7F800000u), "r"(a), "r"(b));
    return __uint_as_float(r);
}

// Staging of the workers' planes for the aggregation sweep: the 1024 exponent bytes and 32 sign
// words of a tile are copied global -> shared with cp.async (16 bytes per lane and copy), three
// workers ahead of the one being decoded, in a ring that is private to the warp.  The loads of
// several workers are in flight without holding registers, so the sweep is not bound by the
// latency of one worker's loads.
constexpr int kAggStages = 4;

struct AggStage {
    uint32_t e[256];     // exponent bytes of the tile, word k*32 + l = lane l's group k
    uint32_t s[32];      // sign words of the tile
};

__device__ __forceinline__ void agg_stage_issue(AggStage* st, const uint8_t* __restrict__ exp_tile,
                                                const uint32_t* __restrict__ sign_tile,
                                                const int lane) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&st->e[lane * 4]);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(exp_tile + lane * 16)
                 : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 512u),
                 "l"(exp_tile + 512 + lane * 16)
                 : "memory");
    if (lane < 8) {
        const uint32_t dsts = (uint32_t)__cvta_generic_to_shared(&st->s[lane * 4]);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dsts),
                     "l"(sign_tile + lane * 4)
                     : "memory");
    }
}

// acc[k] += decoded values of workers 0..n-1, in that order, for one full tile
__device__ __forceinline__ void aggregate_full_tile(const PackedPlanes& planes, const int n,
                                                    const uint64_t base, float4 (&acc)[8],
                                                    const int lane) {
    __shared__ __align__(16) AggStage s_ring[kWarpsPerBlock][kAggStages];
    AggStage* ring = s_ring[threadIdx.x >> 5];
    const int sh = 4 * (lane & 7);
#pragma unroll
    for (int j = 0; j < kAggStages - 1; ++j) {
        if (j < n) agg_stage_issue(&ring[j], planes.exp[j] + base, planes.sign[j] + (base >> 5), lane);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int i = 0; i < n; ++i) {
        const int ahead = i + kAggStages - 1;
        if (ahead < n)
            agg_stage_issue(&ring[ahead % kAggStages], planes.exp[ahead] + base,
                            planes.sign[ahead] + (base >> 5), lane);
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group %0;" ::"n"(kAggStages - 1) : "memory");
        __syncwarp();                                   // worker i's planes are in the ring
        const AggStage* st = &ring[i % kAggStages];
        const uint32_t sw = st->s[lane];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t e = st->e[k * 32 + lane];
            // sign word (k, g) lives in lane 4k+g; this lane needs group g = lane / 8
            const uint32_t s = (__shfl_sync(0xFFFFFFFFu, sw, k * 4 + (lane >> 3)) >> sh) & 0xFu;
            acc[k].x += decode9<0>(e, s);
            acc[k].y += decode9<1>(e, s);
            acc[k].z += decode9<2>(e, s);
            acc[k].w += decode9<3>(e, s);
        }
        __syncwarp();                                   // the stage may be overwritten now
    }
}

// The same sweep with plain loads, for the kernel that compresses the sum again: that one is
// bound by its own generator and packing work, and the shared-memory ring only costs it residency.
__device__ __forceinline__ void aggregate_full_tile_direct(const PackedPlanes& planes, const int n,
                                                           const uint64_t base, float4 (&acc)[8],
                                                           const int lane) {
    const int sh = 4 * (lane & 7);
    for (int i = 0; i < n; ++i) {
        const uint32_t* ev = reinterpret_cast<const uint32_t*>(planes.exp[i] + base);
        const uint32_t sw = ld_stream_u32(planes.sign[i] + (base >> 5) + lane);
        uint32_t e[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) e[k] = ld_stream_u32(ev + k * 32 + lane);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t s = (__shfl_sync(0xFFFFFFFFu, sw, k * 4 + (lane >> 3)) >> sh) & 0xFu;
            acc[k].x += decode9<0>(e[k], s);
            acc[k].y += decode9<1>(e[k], s);
            acc[k].z += decode9<2>(e[k], s);
            acc[k].w += decode9<3>(e[k], s);
        }
    }
}

// the same sum for one element (ragged tile)
__device__ __forceinline__ float aggregate_element(const PackedPlanes& planes, const int n,
                                                   const uint64_t j, float a) {
    for (int i = 0; i < n; ++i) {
        const uint32_t e = planes.exp[i][j];
        const uint32_t s = (planes.sign[i][j >> 5] >> (j & 31)) & 1u;
        a += __uint_as_float((e << 23) | (s << 31));
    }
    return a;
}

// out[j] = (init + v_0j) + v_1j + ... ; init = +0 (aggregate) or acc[j] (decode-accumulate).
// grid: ceil(tiles / warps per block)
template <bool kFromAcc>
__global__ void __launch_bounds__(kBlockThreads, 4)
nc_aggregate_kernel(const __grid_constant__ PackedPlanes planes, const int n, const uint64_t d,
                    float* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;

    if (base + kTile <= d) {
        float4 acc[8];
        float4* ov = reinterpret_cast<float4*>(out + base);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (kFromAcc) acc[k] = __ldcs(ov + k * 32 + lane);
            else acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        aggregate_full_tile(planes, n, base, acc, lane);
#pragma unroll
        for (int k = 0; k < 8; ++k) st_stream_f4(ov + k * 32 + lane, acc[k]);
        return;
    }
    for (uint64_t j = base + lane; j < d; j += 32)      // ragged last tile: scalar
        NC_STORE(out + j, aggregate_element(planes, n, j, kFromAcc ? out[j] : 0.f));
}

// Master side with compression of the aggregate (Algorithm 1: g = C_M(sum_i Delta_i) with
// C_M = C_nat): the fp32 sum never leaves the registers, only its 9-bit code is written.
// The call covers the elements [first, d) of a longer vector (first a multiple of the tile size):
// every pointer is the address element 0 of that vector would have, so that the stream index and
// the memory index of an element are the same number.
// grid: ceil(tiles in [first, d) / warps per block)
__global__ void __launch_bounds__(kBlockThreads, 4)
nc_aggregate_compress_kernel(const __grid_constant__ PackedPlanes planes, const int n,
                             const uint64_t first, const uint64_t d, const uint32_t master,
                             const __grid_constant__ PhiloxKeys keys, uint8_t* __restrict__ exp,
                             uint32_t* __restrict__ sign) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = first + tile * kTile;
    if (base >= d) return;
    if (base + kTile <= d) {
        float4 acc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        aggregate_full_tile_direct(planes, n, base, acc, lane);
        uint4 u[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
            u[k] = make_uint4(__float_as_uint(acc[k].x), __float_as_uint(acc[k].y),
                              __float_as_uint(acc[k].z), __float_as_uint(acc[k].w));
        cnat_full_tile<false>(u, base, master, keys, exp, sign, lane);
        return;
    }
    cnat_ragged_tile<false>(
        [&](uint64_t j) { return __float_as_uint(aggregate_element(planes, n, j, 0.f)); }, base,
        d, master, keys, exp, sign, lane);
}

// uncompressed reference point: n-way fp32 sum in worker order
__global__ void __launch_bounds__(kBlockThreads)
nc_sum_fp32_kernel(const __grid_constant__ DensePlanes planes, const int n, const uint64_t d,
                   float* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    if (base + kTile <= d) {
        float4 acc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int i = 0; i < n; ++i) {
            const float4* xv = reinterpret_cast<const float4*>(planes.x[i] + base);
            float4 v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = __ldcs(xv + k * 32 + lane);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                acc[k].x += v[k].x; acc[k].y += v[k].y; acc[k].z += v[k].z; acc[k].w += v[k].w;
            }
        }
        float4* ov = reinterpret_cast<float4*>(out + base);
#pragma unroll
        for (int k = 0; k < 8; ++k) st_stream_f4(ov + k * 32 + lane, acc[k]);
        return;
    }
    for (uint64_t j = base + lane; j < d; j += 32) {
        float a = 0.f;
        for (int i = 0; i < n; ++i) a += planes.x[i][j];
        NC_STORE(out + j, a);
    }
}

inline unsigned tile_blocks(uint64_t d) {
    const uint64_t tiles = (d + kTile - 1) / kTile;
    return (unsigned)((tiles + kWarpsPerBlock - 1) / kWarpsPerBlock);
}

}  // namespace natcomp

using namespace natcomp;

extern "C" {

static nc_status compress_batch_impl(const float* const* xs, size_t d, uint64_t seed,
                                     const uint32_t* workers, uint8_t* const* exps,
                                     uint32_t* const* signs, int n, bool deterministic,
                                     cudaStream_t stream) {
    if (!xs || !exps || !signs || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (!workers && !deterministic) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    CompressBatch batch;
    BoundsScope scope;
    for (int i = 0; i < n; ++i) {
        if (!xs[i] || !exps[i] || !signs[i]) return NC_ERR_INVALID;
        if (!aligned32(xs[i]) || !aligned16(exps[i]) || !aligned16(signs[i])) return NC_ERR_ALIGN;
        batch.x[i] = xs[i];
        batch.exp[i] = exps[i];
        batch.sign[i] = signs[i];
        batch.worker[i] = workers ? workers[i] : 0u;
        scope.add(exps[i], nc_exp_bytes(d));
        scope.add(signs[i], nc_sign_bytes(d));
    }
    scope.commit(stream);
    const PhiloxKeys keys = make_philox_keys(seed);
    dim3 grid(tile_blocks(d), (unsigned)n);
    if (deterministic)
        nc_compress_kernel<true><<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d, keys);
    else
        nc_compress_kernel<false><<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d, keys);
    return launch_status();
}

nc_status nc_compress_batch(const float* const* xs, size_t d, uint64_t seed,
                            const uint32_t* workers, uint8_t* const* exps,
                            uint32_t* const* signs, int n, cudaStream_t stream) {
    return compress_batch_impl(xs, d, seed, workers, exps, signs, n, false, stream);
}

nc_status nc_compress_nearest_batch(const float* const* xs, size_t d, uint8_t* const* exps,
                                    uint32_t* const* signs, int n, cudaStream_t stream) {
    return compress_batch_impl(xs, d, 0, nullptr, exps, signs, n, true, stream);
}

nc_status nc_compress_nearest(const float* x, size_t d, uint8_t* exp, uint32_t* sign,
                              cudaStream_t stream) {
    return compress_batch_impl(&x, d, 0, nullptr, &exp, &sign, 1, true, stream);
}

nc_status nc_compress(const float* x, size_t d, uint64_t seed, uint32_t worker, uint8_t* exp,
                      uint32_t* sign, cudaStream_t stream) {
    return nc_compress_batch(&x, d, seed, &worker, &exp, &sign, 1, stream);
}

nc_status nc_compress_typed_batch(const void* const* xs, int dtype, size_t d, uint64_t seed,
                                  const uint32_t* workers, uint8_t* const* exps,
                                  uint32_t* const* signs, int n, cudaStream_t stream) {
    if (dtype == NC_DTYPE_F32)
        return nc_compress_batch(reinterpret_cast<const float* const*>(xs), d, seed, workers, exps,
                                 signs, n, stream);
    if (dtype != NC_DTYPE_BF16 && dtype != NC_DTYPE_F16) return NC_ERR_UNSUPPORTED;
    if (!xs || !workers || !exps || !signs || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    Compress16Batch batch;
    BoundsScope scope;
    for (int i = 0; i < n; ++i) {
        if (!xs[i] || !exps[i] || !signs[i]) return NC_ERR_INVALID;
        if (!aligned16(xs[i]) || !aligned16(exps[i]) || !aligned16(signs[i])) return NC_ERR_ALIGN;
        batch.x[i] = reinterpret_cast<const uint16_t*>(xs[i]);
        batch.exp[i] = exps[i];
        batch.sign[i] = signs[i];
        batch.worker[i] = workers[i];
        scope.add(exps[i], nc_exp_bytes(d));
        scope.add(signs[i], nc_sign_bytes(d));
    }
    scope.commit(stream);
    const PhiloxKeys keys = make_philox_keys(seed);
    dim3 grid(tile_blocks(d), (unsigned)n);
    if (dtype == NC_DTYPE_BF16)
        nc_compress16_kernel<NC_DTYPE_BF16><<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d,
                                                                               keys);
    else
        nc_compress16_kernel<NC_DTYPE_F16><<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d,
                                                                              keys);
    return launch_status();
}

nc_status nc_compress_typed(const void* x, int dtype, size_t d, uint64_t seed, uint32_t worker,
                            uint8_t* exp, uint32_t* sign, cudaStream_t stream) {
    return nc_compress_typed_batch(&x, dtype, d, seed, &worker, &exp, &sign, 1, stream);
}

nc_status nc_aggregate(const uint8_t* const* exps, const uint32_t* const* signs, int n, size_t d,
                       float* out, cudaStream_t stream) {
    if (!exps || !signs || !out || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned32(out)) return NC_ERR_ALIGN;
    PackedPlanes planes;
    for (int i = 0; i < n; ++i) {
        if (!exps[i] || !signs[i]) return NC_ERR_INVALID;
        if (!aligned16(exps[i]) || !aligned16(signs[i])) return NC_ERR_ALIGN;
        planes.exp[i] = exps[i];
        planes.sign[i] = signs[i];
    }
    BoundsScope scope;
    scope.add(out, 4 * (size_t)d);
    scope.commit(stream);
    nc_aggregate_kernel<false><<<tile_blocks(d), kBlockThreads, 0, stream>>>(planes, n,
                                                                             (uint64_t)d, out);
    return launch_status();
}

nc_status nc_aggregate_compress_shard(const uint8_t* const* exps, const uint32_t* const* signs,
                                      int n, size_t d, uint64_t first_index, uint64_t seed,
                                      uint32_t master, uint8_t* out_exp, uint32_t* out_sign,
                                      cudaStream_t stream) {
    if (!exps || !signs || !out_exp || !out_sign || n < 1 || n > NC_MAX_WORKERS)
        return NC_ERR_INVALID;
    if (first_index % kTile != 0) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40) || first_index > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned16(out_exp) || !aligned16(out_sign)) return NC_ERR_ALIGN;
    // the kernel indexes by position in the whole vector: move every pointer back by the shard's
    // offset (first_index bytes of exponents, first_index / 8 bytes of sign words)
    const uintptr_t exp_back = (uintptr_t)first_index, sign_back = (uintptr_t)(first_index / 8);
    PackedPlanes planes;
    for (int i = 0; i < n; ++i) {
        if (!exps[i] || !signs[i]) return NC_ERR_INVALID;
        if (!aligned16(exps[i]) || !aligned16(signs[i])) return NC_ERR_ALIGN;
        planes.exp[i] = reinterpret_cast<const uint8_t*>((uintptr_t)exps[i] - exp_back);
        planes.sign[i] = reinterpret_cast<const uint32_t*>((uintptr_t)signs[i] - sign_back);
    }
    const PhiloxKeys keys = make_philox_keys(seed);
    BoundsScope scope;
    scope.add(out_exp, nc_exp_bytes(d));
    scope.add(out_sign, nc_sign_bytes(d));
    scope.commit(stream);
    nc_aggregate_compress_kernel<<<tile_blocks(d), kBlockThreads, 0, stream>>>(
        planes, n, first_index, first_index + (uint64_t)d, master, keys,
        reinterpret_cast<uint8_t*>((uintptr_t)out_exp - exp_back),
        reinterpret_cast<uint32_t*>((uintptr_t)out_sign - sign_back));
    return launch_status();
}

nc_status nc_aggregate_compress(const uint8_t* const* exps, const uint32_t* const* signs, int n,
                                size_t d, uint64_t seed, uint32_t master, uint8_t* out_exp,
                                uint32_t* out_sign, cudaStream_t stream) {
    return nc_aggregate_compress_shard(exps, signs, n, d, 0, seed, master, out_exp, out_sign,
                                       stream);
}

nc_status nc_decode_accumulate(const uint8_t* exp, const uint32_t* sign, size_t d, float* acc,
                               cudaStream_t stream) {
    if (!exp || !sign || !acc) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned16(exp) || !aligned16(sign) || !aligned32(acc)) return NC_ERR_ALIGN;
    PackedPlanes planes;
    planes.exp[0] = exp;
    planes.sign[0] = sign;
    BoundsScope scope;
    scope.add(acc, 4 * (size_t)d);
    scope.commit(stream);
    nc_aggregate_kernel<true><<<tile_blocks(d), kBlockThreads, 0, stream>>>(planes, 1,
                                                                            (uint64_t)d, acc);
    return launch_status();
}

nc_status nc_sum_fp32(const float* const* xs, int n, size_t d, float* out, cudaStream_t stream) {
    if (!xs || !out || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned32(out)) return NC_ERR_ALIGN;
    DensePlanes planes;
    for (int i = 0; i < n; ++i) {
        if (!xs[i]) return NC_ERR_INVALID;
        if (!aligned32(xs[i])) return NC_ERR_ALIGN;
        planes.x[i] = xs[i];
    }
    BoundsScope scope;
    scope.add(out, 4 * (size_t)d);
    scope.commit(stream);
    nc_sum_fp32_kernel<<<tile_blocks(d), kBlockThreads, 0, stream>>>(planes, n, (uint64_t)d, out);
    return launch_status();
}

}  // extern "C"

// The 8-bit wire format and the integer aggregation of the paper's own implementation
// (experimental set-up appendix and "fast aggregation" appendix of arXiv 1905.10988), for sm_100a.
//
// Worker: C_nat as in nc_compress, then one byte per entry:
//     bit 7 = sign, bit 6 = "is zero", bits 0..5 = exponent + 50 with the exponent clipped to
//     [-50, 10] (so +-inf and anything above 2^10 become +-2^10, anything below 2^-50 that is not
//     zero becomes +-2^-50).
// Master: every code is restored as a 64-bit integer with one non-zero bit, +-2^(exponent + 50),
// and the workers' integers are added.  Integer addition is associative, so the result does not
// depend on the order of the workers; it is exact as long as |sum| < 2^63 (always for n <= 7, and
// for any n when no entry sits at the clip ceiling).  The sum is returned as fp32
// (fl32(sum) * 2^-50) or compressed again with C_nat into the same 8-bit format.
//
// A code byte c restores with a single shift: (c & 0x7F) is the shift amount, and the zero flag
// (bit 6) makes it >= 64, which the 64-bit shift instruction turns into 0.
#include "common.cuh"
#include "philox.cuh"

namespace natcomp {

struct Compress8Batch {
    const float* x[NC_MAX_WORKERS];
    uint8_t* code[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

struct Code8Planes {
    const uint8_t* code[NC_MAX_WORKERS];
};

constexpr uint32_t kExpLo = 127 - 50;   // biased exponent of 2^-50
constexpr uint32_t kExpHi = 127 + 10;   // biased exponent of 2^10

// 8-bit code from the biased exponent byte of C_nat(x) and the sign bit
__device__ __forceinline__ uint32_t code8_from_exp(uint32_t e, uint32_t sign_bit) {
    const uint32_t c = (e == 0u) ? 0x40u : (min(max(e, kExpLo), kExpHi) - kExpLo);
    return c | (sign_bit << 7);
}

__device__ __forceinline__ uint32_t cnat_code8(uint32_t bits, uint32_t rnd) {
    uint32_t v = bits & 0x7FFFFFFFu;
    if (v < 0x7F000000u) v += ~rnd & 0x7FFFFFu;   // no rounding up at the top exponents
    return code8_from_exp(v >> 23, bits >> 31);
}

// Restores byte K of a word of four codes: +1 or -1 as a 64-bit integer (high word = the sign
// bit spread by an arithmetic shift, low word = that | 1), shifted left by the 7-bit field (the
// zero flag makes the shift >= 64, which gives 0).
template <int K>
__device__ __forceinline__ long long restore8_of(uint32_t c4) {
    const int hi = (int)(c4 << (24 - 8 * K)) >> 31;                      // 0 or -1
    const unsigned long long one =
        ((unsigned long long)(uint32_t)hi << 32) | (uint32_t)(hi | 1);   // +1 or -1
    unsigned long long v;
    asm("shl.b64 %0, %1, %2;" : "=l"(v) : "l"(one), "r"((c4 >> (8 * K)) & 0x7Fu));
    return (long long)v;
}

// grid: (ceil(tiles / warps per block), n workers)
__global__ void __launch_bounds__(kBlockThreads)
nc8_compress_kernel(const __grid_constant__ Compress8Batch batch, const uint64_t d,
                    const __grid_constant__ PhiloxKeys keys) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    const int w = blockIdx.y;
    const float* __restrict__ x = batch.x[w];
    uint8_t* __restrict__ code = batch.code[w];
    const uint32_t worker = batch.worker[w];
    if (base + kTile <= d) {
        const uint4* xv = reinterpret_cast<const uint4*>(x + base);
        uint4 u[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) u[k] = ld_stream_u4(xv + k * 32 + lane);
        uint32_t* cv = reinterpret_cast<uint32_t*>(code + base);
        const PhiloxTile pt = philox_tile((uint32_t)(base >> 34), worker, kDomainCnat, keys);
        const uint32_t q_lo = (uint32_t)(base >> 2) + lane;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t rnd[4];
            stream_words4_tile(q_lo + k * 32, pt, keys, rnd);
            const uint32_t c = cnat_code8(u[k].x, rnd[0]) | (cnat_code8(u[k].y, rnd[1]) << 8) |
                               (cnat_code8(u[k].z, rnd[2]) << 16) |
                               (cnat_code8(u[k].w, rnd[3]) << 24);
            st_stream_u32(cv + k * 32 + lane, c);
        }
        return;
    }
    const uint64_t end = round_up16(d);          // zero padding up to the plane size
    for (uint64_t j = base + lane; j < end; j += 32) {
        uint32_t c = 0;
        if (j < d) {
            uint32_t rnd[4];
            stream_words4(j >> 2, worker, kDomainCnat, keys, rnd);
            const uint32_t r = (j & 3) == 0 ? rnd[0] : (j & 3) == 1 ? rnd[1]
                             : (j & 3) == 2 ? rnd[2] : rnd[3];
            c = cnat_code8(__float_as_uint(x[j]), r);
        }
        code[j] = (uint8_t)c;
    }
}

// C_nat of the integer s (value s * 2^-50), as an 8-bit code.  The up-probability is the
// fraction of |s| above its leading one, truncated to 23 bits.
__device__ __forceinline__ uint32_t cnat_code8_of_int(long long s, uint32_t rnd) {
    if (s == 0) return 0x40u;
    const uint32_t sign_bit = s < 0 ? 1u : 0u;
    const unsigned long long a = s < 0 ? 0ull - (unsigned long long)s : (unsigned long long)s;
    const int e = 63 - __clzll((long long)a);                  // leading one: 2^e <= a < 2^(e+1)
    const unsigned long long frac = a - (1ull << e);
    const uint32_t thr = e >= 23 ? (uint32_t)(frac >> (e - 23)) : (uint32_t)(frac << (23 - e));
    const uint32_t up = (rnd & 0x7FFFFFu) < thr ? 1u : 0u;
    const uint32_t biased = (uint32_t)(e - 50 + 127) + up;     // exponent of the rounded value
    return code8_from_exp(biased, sign_bit);
}

__device__ __forceinline__ void add_codes4(long long* acc, uint32_t c4) {
    acc[0] += restore8_of<0>(c4);
    acc[1] += restore8_of<1>(c4);
    acc[2] += restore8_of<2>(c4);
    acc[3] += restore8_of<3>(c4);
}

// kCompress = false: out32[j] = fl32(sum) * 2^-50;  true: out8[j] = code of C_nat(sum)
// A thread owns 16 consecutive entries (one 128-bit load per worker, the next worker's load in
// flight while this one's codes are added).
// grid: ceil(d / (threads * 16))
template <bool kCompress>
__global__ void __launch_bounds__(kBlockThreads)
nc8_aggregate_kernel(const __grid_constant__ Code8Planes planes, const int n, const uint64_t d,
                     float* __restrict__ out32, uint8_t* __restrict__ out8, const uint32_t master,
                     const __grid_constant__ PhiloxKeys keys) {
    const uint64_t j0 = ((uint64_t)blockIdx.x * kBlockThreads + threadIdx.x) * 16;
    if (j0 >= d) return;          // the plane's padding up to 16 bytes lies in the last group
    long long acc[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) acc[c] = 0;
    // planes are padded to 16 bytes, so the 16-byte load stays inside the plane
    uint4 cur = ld_stream_u4(planes.code[0] + j0);
    for (int i = 0; i < n; ++i) {
        uint4 nxt = make_uint4(0u, 0u, 0u, 0u);
        if (i + 1 < n) nxt = ld_stream_u4(planes.code[i + 1] + j0);
        add_codes4(acc + 0, cur.x);
        add_codes4(acc + 4, cur.y);
        add_codes4(acc + 8, cur.z);
        add_codes4(acc + 12, cur.w);
        cur = nxt;
    }
    if (!kCompress) {
        if (j0 + 16 <= d) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                float4 o;
                o.x = __fmul_rn(__ll2float_rn(acc[4 * g + 0]), 8.8817841970012523e-16f);
                o.y = __fmul_rn(__ll2float_rn(acc[4 * g + 1]), 8.8817841970012523e-16f);
                o.z = __fmul_rn(__ll2float_rn(acc[4 * g + 2]), 8.8817841970012523e-16f);
                o.w = __fmul_rn(__ll2float_rn(acc[4 * g + 3]), 8.8817841970012523e-16f);
                __stcs(reinterpret_cast<float4*>(out32 + j0) + g, o);
            }
        } else {
#pragma unroll
            for (int c = 0; c < 16; ++c)
                if (j0 + c < d)
                    out32[j0 + c] = __fmul_rn(__ll2float_rn(acc[c]), 8.8817841970012523e-16f);
        }
    } else {
        uint32_t c4[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            uint32_t rnd[4];
            stream_words4((j0 >> 2) + g, master, kDomainCnat, keys, rnd);
            c4[g] = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (j0 + 4 * g + c < d) c4[g] |= cnat_code8_of_int(acc[4 * g + c], rnd[c]) << (8 * c);
        }
        st_stream_u4(out8 + j0, make_uint4(c4[0], c4[1], c4[2], c4[3]));   // zero padding past d
    }
}

}  // namespace natcomp

using namespace natcomp;

extern "C" {

nc_status nc8_compress_batch(const float* const* xs, size_t d, uint64_t seed,
                             const uint32_t* workers, uint8_t* const* codes, int n,
                             cudaStream_t stream) {
    if (!xs || !workers || !codes || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    Compress8Batch batch;
    for (int i = 0; i < n; ++i) {
        if (!xs[i] || !codes[i]) return NC_ERR_INVALID;
        if (!aligned32(xs[i]) || !aligned16(codes[i])) return NC_ERR_ALIGN;
        batch.x[i] = xs[i];
        batch.code[i] = codes[i];
        batch.worker[i] = workers[i];
    }
    const PhiloxKeys keys = make_philox_keys(seed);
    const uint64_t tiles = (d + kTile - 1) / kTile;
    const dim3 grid((unsigned)((tiles + kWarpsPerBlock - 1) / kWarpsPerBlock), (unsigned)n);
    nc8_compress_kernel<<<grid, kBlockThreads, 0, stream>>>(batch, (uint64_t)d, keys);
    return launch_status();
}

nc_status nc8_compress(const float* x, size_t d, uint64_t seed, uint32_t worker, uint8_t* code,
                       cudaStream_t stream) {
    return nc8_compress_batch(&x, d, seed, &worker, &code, 1, stream);
}

static nc_status nc8_planes(const uint8_t* const* codes, int n, Code8Planes* planes) {
    for (int i = 0; i < n; ++i) {
        if (!codes[i]) return NC_ERR_INVALID;
        if (!aligned16(codes[i])) return NC_ERR_ALIGN;
        planes->code[i] = codes[i];
    }
    return NC_OK;
}

nc_status nc8_aggregate(const uint8_t* const* codes, int n, size_t d, float* out,
                        cudaStream_t stream) {
    if (!codes || !out || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned32(out)) return NC_ERR_ALIGN;
    Code8Planes planes;
    const nc_status st = nc8_planes(codes, n, &planes);
    if (st != NC_OK) return st;
    const uint64_t groups = round_up16(d) / 16;
    const unsigned grid = (unsigned)((groups + kBlockThreads - 1) / kBlockThreads);
    const PhiloxKeys keys = make_philox_keys(0);
    nc8_aggregate_kernel<false><<<grid, kBlockThreads, 0, stream>>>(planes, n, (uint64_t)d, out,
                                                                    nullptr, 0u, keys);
    return launch_status();
}

nc_status nc8_aggregate_compress(const uint8_t* const* codes, int n, size_t d, uint64_t seed,
                                 uint32_t master, uint8_t* out_code, cudaStream_t stream) {
    if (!codes || !out_code || n < 1 || n > NC_MAX_WORKERS) return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned16(out_code)) return NC_ERR_ALIGN;
    Code8Planes planes;
    const nc_status st = nc8_planes(codes, n, &planes);
    if (st != NC_OK) return st;
    const uint64_t groups = round_up16(d) / 16;
    const unsigned grid = (unsigned)((groups + kBlockThreads - 1) / kBlockThreads);
    const PhiloxKeys keys = make_philox_keys(seed);
    nc8_aggregate_kernel<true><<<grid, kBlockThreads, 0, stream>>>(planes, n, (uint64_t)d, nullptr,
                                                                   out_code, master, keys);
    return launch_status();
}

}  // extern "C"

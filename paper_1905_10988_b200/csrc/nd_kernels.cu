// Natural dithering D_nat^{p,s} (Def. 3 of arXiv 1905.10988 with the levels 2^-u) for
// sm_100a: per-bucket p-norm, level rounding + packing, and the master-side decode / n-way sum.
//
// Work decomposition: one warp owns a tile of 1024 consecutive elements in four steps of 256;
// in a step lane l owns the 8 consecutive elements 8l..8l+7 (one 256-bit load, two Philox
// blocks, one 32-bit word of level nibbles, one byte of sign bits).
//
// Norms are deterministic: every (tile, bucket) overlap writes one partial into its own slot
// (slot = tile index + bucket index, strictly increasing along the vector), and one block per
// bucket adds the bucket's slots in a fixed order.  No atomics, no zero-filling.
//
// Level rounding (given the bucket norm): y = fl32(|x| * fl32(1/norm)), z = y * 2^s (exact).
// For z >= 2 the level below is 2^(E_z - 127 - s) and the up-probability is the mantissa
// fraction of z, exactly as in C_nat; for z < 2 (y below the smallest level 2^(1-s)) the
// up-probability is y * 2^(s-1), obtained as the mantissa of 1 + z/2 rounded toward zero.
// In both cases  code = min(((bits(w) + (~r23 & 0x7FFFFF)) >> 23) - 127, s).
#include "common.cuh"
#include "philox.cuh"

namespace natcomp {

struct DitherPlanes {
    const float* norms[NC_MAX_WORKERS];
    const uint8_t* level[NC_MAX_WORKERS];
    const uint32_t* sign[NC_MAX_WORKERS];
};

struct DitherBatch {
    const float* x[NC_MAX_WORKERS];
    float* norms[NC_MAX_WORKERS];
    uint8_t* level[NC_MAX_WORKERS];
    uint32_t* sign[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

struct V8 {
    uint32_t v[8];
};

__device__ __forceinline__ V8 ld_stream_v8(const void* p) {
    V8 r;
    asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]),
                   "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}

__device__ __forceinline__ void st_stream_v8(void* p, const V8& r) {
    if (!NC_STORE_OK(p, 32u)) return;
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(r.v[0]),
                 "r"(r.v[1]), "r"(r.v[2]), "r"(r.v[3]), "r"(r.v[4]), "r"(r.v[5]), "r"(r.v[6]),
                 "r"(r.v[7])
                 : "memory");
}

// largest b in [0, B-1] with off[b] <= pos (pos < off[B]); skips empty buckets by construction
__device__ __forceinline__ int find_bucket(const uint64_t* __restrict__ off, int B, uint64_t pos) {
    int lo = 0, hi = B;   // invariant: off[lo] <= pos < off[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(off + mid) <= pos) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ uint32_t warp_max(uint32_t v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// One partial per (tile, bucket) overlap.  p = 1: sum |x| (chains of at most 8 terms in
// binary32, everything above that in binary64), p = 2: sum x^2 with squares and sums in
// binary64, p = inf: the largest |x| as a bit pattern (NaN patterns compare above inf, so a
// NaN survives).
template <int P>
struct NormAcc {
    float f[4];
    double q[4];
    double dsum;
    uint32_t m;
    __device__ __forceinline__ void init() {
        f[0] = f[1] = f[2] = f[3] = 0.f;
        q[0] = q[1] = q[2] = q[3] = 0.0;
        dsum = 0.0;
        m = 0;
    }
    __device__ __forceinline__ void add(uint32_t bits, int chain) {
        const uint32_t a = bits & 0x7FFFFFFFu;
        if (P == NC_P_INF) m = max(m, a);
        else if (P == 1) f[chain] += __uint_as_float(a);
        else {
            // squares in binary64: a binary32 square underflows for |x| < 2^-63
            const double v = (double)__uint_as_float(a);
            q[chain] = fma(v, v, q[chain]);
        }
    }
    __device__ __forceinline__ void flush() {
        if (P == 1) {
            dsum += ((double)f[0] + (double)f[1]) + ((double)f[2] + (double)f[3]);
            f[0] = f[1] = f[2] = f[3] = 0.f;
        } else if (P == 2) {
            dsum += (q[0] + q[1]) + (q[2] + q[3]);
            q[0] = q[1] = q[2] = q[3] = 0.0;
        }
    }
    // warp-wide result as 64 bits for the slot
    __device__ __forceinline__ uint64_t reduce() {
        if (P == NC_P_INF) return (uint64_t)warp_max(m);
        flush();
        return (uint64_t)__double_as_longlong(warp_sum(dsum));
    }
};

// norm partial(s) of one tile; `u` holds the tile's entries if it is full
template <int P>
__device__ __forceinline__ void norm_tile(const float* __restrict__ x, uint64_t* __restrict__ slots,
                                          const uint64_t tile, const uint64_t d,
                                          const uint64_t* __restrict__ off, const int B,
                                          uint32_t* __restrict__ tile_bucket, const V8 (&u)[4],
                                          const bool full, const int lane) {
    const uint64_t base = tile * kTile;
    const uint64_t end = full ? base + kTile : d;
    int b = find_bucket(off, B, base);
    if (lane == 0) NC_STORE(tile_bucket + tile, (uint32_t)b);

    NormAcc<P> acc;
    if (full && __ldg(off + b + 1) >= end) {
        acc.init();
#pragma unroll
        for (int it = 0; it < 4; ++it) {
#pragma unroll
            for (int c = 0; c < 8; ++c) acc.add(u[it].v[c], c & 3);
        }
        const uint64_t r = acc.reduce();
        if (lane == 0) NC_STORE(slots + tile + (uint64_t)b, r);
        return;
    }
    // the tile spans several buckets or is ragged: one segment at a time, lane-strided
    uint64_t pos = base;
    while (pos < end) {
        uint64_t seg_end = __ldg(off + b + 1);
        if (seg_end > end) seg_end = end;
        acc.init();
        int cnt = 0;
        for (uint64_t j = pos + lane; j < seg_end; j += 32) {
            acc.add(__float_as_uint(x[j]), 0);
            if (++cnt == 8) { acc.flush(); cnt = 0; }
        }
        const uint64_t r = acc.reduce();
        if (lane == 0) NC_STORE(slots + tile + (uint64_t)b, r);
        pos = seg_end;
        if (pos < end) {
            ++b;
            while (__ldg(off + b + 1) <= pos) ++b;   // skip empty buckets
        }
    }
}

// Persistent warps: a warp takes the tiles w, w + W, w + 2W, ... (W = warps in the grid row) and
// loads the next tile before it reduces the current one, so every warp always has 4 KB in flight.
// grid: (blocks resident on the device, n workers); worker w uses slots + w * slot_stride
template <int P>
__global__ void __launch_bounds__(kBlockThreads, 2)
nd_norm_partials_kernel(const __grid_constant__ DitherBatch batch, const uint64_t d,
                        const uint64_t* __restrict__ off, const int B,
                        uint64_t* __restrict__ slots_all, const uint64_t slot_stride,
                        uint32_t* __restrict__ tile_bucket) {
    const int lane = threadIdx.x & 31;
    const uint64_t tiles = (d + kTile - 1) / kTile;
    const uint64_t stride = (uint64_t)gridDim.x * kWarpsPerBlock;
    uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (tile >= tiles) return;
    const float* __restrict__ x = batch.x[blockIdx.y];
    uint64_t* __restrict__ slots = slots_all + (uint64_t)blockIdx.y * slot_stride;
    V8 u[4], nx[4];
    bool full = (tile + 1) * kTile <= d;
    if (full) {
#pragma unroll
        for (int it = 0; it < 4; ++it) u[it] = ld_stream_v8(x + tile * kTile + it * 256 + lane * 8);
    }
    for (;;) {
        const uint64_t next = tile + stride;
        const bool next_full = next < tiles && (next + 1) * kTile <= d;
        if (next_full) {
#pragma unroll
            for (int it = 0; it < 4; ++it)
                nx[it] = ld_stream_v8(x + next * kTile + it * 256 + lane * 8);
        }
        norm_tile<P>(x, slots, tile, d, off, B, tile_bucket, u, full, lane);
        if (next >= tiles) break;
        tile = next;
        full = next_full;
#pragma unroll
        for (int it = 0; it < 4; ++it) u[it] = nx[it];
    }
}

// one block per (bucket, worker): fixed-order sum (or max) of the bucket's slots -> norms[b]
template <int P>
__global__ void __launch_bounds__(kBlockThreads)
nd_norm_finalize_kernel(const __grid_constant__ DitherBatch batch,
                        const uint64_t* __restrict__ off, const int B,
                        const uint64_t* __restrict__ slots_all, const uint64_t slot_stride,
                        uint32_t* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x;
    const uint64_t* __restrict__ slots = slots_all + (uint64_t)blockIdx.y * slot_stride;
    float* __restrict__ norms = batch.norms[blockIdx.y];
    __shared__ double s_sum[kWarpsPerBlock];
    __shared__ uint32_t s_max[kWarpsPerBlock];
    const uint64_t lo = off[b], hi = off[b + 1];
    if (hi <= lo) {                      // empty bucket (uniform over the block)
        if (threadIdx.x == 0) NC_STORE(norms + b, 0.f);
        return;
    }
    const uint64_t t_first = lo / kTile, t_last = (hi - 1) / kTile;
    uint32_t m = 0;
    double s = 0.0;
    for (uint64_t t = t_first + threadIdx.x; t <= t_last; t += kBlockThreads) {
        const uint64_t v = slots[t + (uint64_t)b];
        if (P == NC_P_INF) m = max(m, (uint32_t)v);
        else s += __longlong_as_double((long long)v);
    }
    if (P == NC_P_INF) m = warp_max(m);
    else s = warp_sum(s);
    if (lane == 0) {
        s_sum[threadIdx.x >> 5] = s;
        s_max[threadIdx.x >> 5] = m;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float result;
        if (P == NC_P_INF) {
            for (int w = 1; w < kWarpsPerBlock; ++w) m = max(m, s_max[w]);
            result = __uint_as_float(m);
        } else {
            double tot = 0.0;
            for (int w = 0; w < kWarpsPerBlock; ++w) tot += s_sum[w];     // fixed order
            if (P == 2) tot = sqrt(tot);
            result = (float)tot;
        }
        NC_STORE(norms + b, result);
        // a bucket that holds an inf or a NaN: its codes will all be 0, the caller is told here
        if (status && !(result <= 3.40282347e38f)) atomicAdd(status, 1u);
    }
}

struct BucketScale {
    float pre;       // 1, or 2^24 when the norm is subnormal (its reciprocal would overflow)
    float rinv;      // fl32(1 / (norm * pre)), or 0 for a degenerate bucket
    uint32_t smax;   // s, or 0 for a degenerate bucket (forces every code to 0)
};

// Degenerate: norm 0 (x = 0 gives D(x) = 0, Def. 3) or not finite.  A subnormal norm is an
// ordinary one: entries and norm are scaled by 2^24 first, which is exact and leaves y unchanged.
__device__ __forceinline__ BucketScale bucket_scale(float norm, int s) {
    BucketScale r;
    const bool ok = (norm > 0.f) && (norm <= 3.40282347e38f);
    r.pre = norm < 1.17549435e-38f ? 16777216.f : 1.f;
    r.rinv = ok ? __fdiv_rn(1.0f, __fmul_rn(norm, r.pre)) : 0.f;
    r.smax = ok ? (uint32_t)s : 0u;
    return r;
}

// level code of one entry; pow2s = 2^s as a float
__device__ __forceinline__ uint32_t level_code(uint32_t bits, uint32_t rnd, const BucketScale sc,
                                               float pow2s) {
    const float y = __fmul_rn(__fmul_rn(fabsf(__uint_as_float(bits)), sc.pre), sc.rinv);
    const float z = __fmul_rn(y, pow2s);
    // below 2 the bottom interval [0, 2^(1-s)] is mapped onto [1, 2): w = 1 + z/2 (> z there);
    // from 2 on 1 + z/2 <= z, so one max selects the right branch
    const float w = fmaxf(z, __fmaf_rz(z, 0.5f, 1.0f));
    const uint32_t t = __float_as_uint(w) + (~rnd & 0x7FFFFFu) - 0x3F800000u;
    return min(t >> 23, sc.smax);
}

// level code from z = |x| * (rinv * 2^s) directly (see the fast path of the rounding kernel)
__device__ __forceinline__ uint32_t level_code_scaled(uint32_t bits, uint32_t rnd, float rinv_s,
                                                      uint32_t smax) {
    const float z = __fmul_rn(fabsf(__uint_as_float(bits)), rinv_s);
    // below 2 the bottom interval [0, 2^(1-s)] is mapped onto [1, 2): w = 1 + z/2 (> z there);
    // from 2 on 1 + z/2 <= z, so one max selects the right branch
    const float w = fmaxf(z, __fmaf_rz(z, 0.5f, 1.0f));
    const uint32_t t = __float_as_uint(w) + (~rnd & 0x7FFFFFu) - 0x3F800000u;
    return min(t >> 23, smax);
}

// grid: ceil(tiles / warps per block).  kClamp: the norms are the caller's, not necessarily those
// of the entries, so |x| / norm may exceed 1 (or be NaN) and the level code is clamped to s.
template <bool kClamp>
__global__ void __launch_bounds__(kBlockThreads, 4)
nd_round_pack_kernel(const __grid_constant__ DitherBatch batch, const uint64_t d,
                     const uint64_t* __restrict__ off, const int B, const int s,
                     const __grid_constant__ PhiloxKeys keys,
                     const uint32_t* __restrict__ tile_bucket) {
    const int lane = threadIdx.x & 31;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint64_t base = tile * kTile;
    if (base >= d) return;
    const float* __restrict__ x = batch.x[blockIdx.y];
    const float* __restrict__ norms = batch.norms[blockIdx.y];
    uint8_t* __restrict__ level = batch.level[blockIdx.y];
    uint32_t* __restrict__ sign = batch.sign[blockIdx.y];
    const uint32_t worker = batch.worker[blockIdx.y];
    const bool full = (base + kTile <= d);
    const float pow2s = __uint_as_float((uint32_t)(127 + s) << 23);

    V8 u[4];
    if (full) {
#pragma unroll
        for (int it = 0; it < 4; ++it) u[it] = ld_stream_v8(x + base + it * 256 + lane * 8);
    }
    // the norm pass leaves the bucket of every tile's first entry in the workspace; the rounding
    // pass on its own looks it up (the loads above are in flight meanwhile)
    int b = tile_bucket ? (int)tile_bucket[tile] : find_bucket(off, B, base);

    // Fast path: the tile lies in one bucket.  z = fl32(fl32(|x| * rinv) * 2^s) is computed as
    // fl32(|x| * (rinv * 2^s)): scaling by 2^s is exact, so the two agree whenever the inner
    // product is a normal number, and when it is subnormal both give z < 2^-100, threshold 0 and
    // level code 0.  If rinv * 2^s overflows (norm below 2^(s-126)) the general path is used.
    const BucketScale sc0 = bucket_scale(norms[b], s);
    const float rinv_s = __fmul_rn(sc0.rinv, pow2s);
    // No clamp of the code in this path unless kClamp: the norm was computed from the same entries, so
    // |x| <= norm, |x| * rinv <= 1 + 2^-24 rounds to at most 1 (a tie goes to the even mantissa 0)
    // and z <= 2^s has a zero mantissa at the top exponent, which the random increment cannot carry
    // out of.  A degenerate bucket (norm 0 or not finite; all codes 0) and one with a subnormal
    // norm take the general path, which clamps.
    if (full && __ldg(off + b + 1) >= base + kTile && rinv_s <= 3.40282347e38f && sc0.smax != 0u &&
        sc0.pre == 1.0f) {
        uint32_t* lv = reinterpret_cast<uint32_t*>(level + (base >> 1));
        const PhiloxTile pt = philox_tile((uint32_t)(base >> 34), worker, kDomainDnat, keys);
        const uint32_t q_lo = (uint32_t)(base >> 2) + (uint32_t)(lane * 2);
        uint32_t sbytes = 0;     // byte `it` = sign bits of this lane's 8 elements in step it
#pragma unroll
        for (int it = 3; it >= 0; --it) {
            uint32_t rnd[8];
            const uint32_t q = q_lo + (uint32_t)(it * 64);   // stays below 2^32: no carry
            {
                uint32_t r4[4];
                stream_words4_tile(q, pt, keys, r4);
                rnd[0] = r4[0]; rnd[1] = r4[1]; rnd[2] = r4[2]; rnd[3] = r4[3];
                stream_words4_tile(q + 1, pt, keys, r4);
                rnd[4] = r4[0]; rnd[5] = r4[1]; rnd[6] = r4[2]; rnd[7] = r4[3];
            }
            // The codes are packed as nib = nib * 16 + e with e = code + 127 (the biased exponent
            // after the carry), and 127 * 0x11111111 is taken off the word at the end:
            // the arithmetic is linear mod 2^32, so the result is the packed codes exactly, the
            // per-entry subtraction is gone and the packing is multiply-add work, which runs
            // beside the integer pipe that bounds this kernel.
            uint32_t nib = 0;
#pragma unroll
            for (int c = 7; c >= 0; --c) {
                float z = __fmul_rn(fabsf(__uint_as_float(u[it].v[c])), rinv_s);
                if (kClamp) z = fminf(z, pow2s);      // y >= 1 (and a NaN ratio): the top level
                const float w = fmaxf(z, __fmaf_rz(z, 0.5f, 1.0f));       // see level_code_scaled
                const uint32_t e = (__float_as_uint(w) + (~rnd[c] & 0x7FFFFFu)) >> 23;
                nib = nib * 16u + e;
                sbytes = __funnelshift_l(u[it].v[c], sbytes, 1);
            }
            st_stream_u32(lv + it * 32 + lane, nib - 127u * 0x11111111u);
        }
        // lane 4g+i holds byte i of sign word (it, g) = word it*8 + g of the tile
        const uint32_t word = transpose_bytes_4x4(sbytes, lane);
        st_stream_u32(sign + (base >> 5) + (lane & 3) * 8 + (lane >> 2), word);
        return;
    }

    // tile spans several buckets or is the ragged end: one element per lane per step
    const uint64_t lvl_end = round_up16((d + 1) / 2) * 2;   // elements covered by level bytes
    const uint64_t sign_words = (d + 31) / 32;
    const uint64_t sign_words_padded = (sign_words + 3) & ~(uint64_t)3;
    uint64_t tile_end = base + kTile;
    if (!full) tile_end = lvl_end > base ? lvl_end : base;
    if (tile_end > base + kTile) tile_end = base + kTile;
    int bl = b;                    // per-lane bucket cursor
    uint64_t bend = __ldg(off + bl + 1);
    BucketScale sc = bucket_scale(norms[bl], s);
    for (uint64_t j0 = base; j0 < tile_end; j0 += 32) {
        const uint64_t j = j0 + lane;
        uint32_t bits = 0, code = 0;
        if (j < d) {
            if (j >= bend) {
                do { ++bl; bend = __ldg(off + bl + 1); } while (j >= bend);
                sc = bucket_scale(norms[bl], s);
            }
            bits = __float_as_uint(x[j]);
            uint32_t r4[4];
            stream_words4(j >> 2, worker, kDomainDnat, keys, r4);
            const uint32_t r = (j & 3) == 0 ? r4[0] : (j & 3) == 1 ? r4[1]
                             : (j & 3) == 2 ? r4[2] : r4[3];
            code = level_code(bits, r, sc, pow2s);
        }
        const uint32_t next = __shfl_down_sync(0xFFFFFFFFu, code, 1);
        if ((lane & 1) == 0 && j < lvl_end) NC_STORE(level + (j >> 1), (uint8_t)(code | (next << 4)));
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, (bits >> 31) != 0);
        if (lane == 0 && (j0 >> 5) < sign_words) NC_STORE(sign + (j0 >> 5), word);
    }
    if (!full && lane < (int)(sign_words_padded - sign_words)) NC_STORE(sign + sign_words + lane, 0u);
}

// ---- master side ------------------------------------------------------------------------

// 8 level nibbles -> exponent bytes of 2^(c-s) (0 for c = 0), four per register
__device__ __forceinline__ void level_exp_bytes(uint32_t nib8, uint32_t kexp, uint32_t& lo4,
                                                uint32_t& hi4) {
    // spread nibbles to bytes: lo4 = nibbles 0..3, hi4 = nibbles 4..7
    uint32_t a = nib8 & 0xFFFFu, b = nib8 >> 16;
    a = (a | (a << 8)) & 0x00FF00FFu;
    a = (a | (a << 4)) & 0x0F0F0F0Fu;
    b = (b | (b << 8)) & 0x00FF00FFu;
    b = (b | (b << 4)) & 0x0F0F0F0Fu;
    // add (127 - s) to every non-zero byte: (x + 0x7F) has bit 7 set iff x >= 1
    const uint32_t ma = ((a + 0x7F7F7F7Fu) & 0x80808080u) >> 7;
    const uint32_t mb = ((b + 0x7F7F7F7Fu) & 0x80808080u) >> 7;
    lo4 = a + ma * kexp;
    hi4 = b + mb * kexp;
}

// +-2^(c-s) (or +-0) of entry K of a group of eight: the exponent byte BYTE of e4 moved to bits
// 30..23, the sign bit K of sg8 (8 valid bits, the rest zero) moved to bit 31, merged by one
// three-input logic operation that takes bits 30..23 from the first and the rest from the second
// operand.  Whatever else the shifts drag along lands in bits that the merge does not take.
template <int BYTE, int K>
__device__ __forceinline__ float pow2_signed(uint32_t e4, uint32_t sg8) {
    const uint32_t a = BYTE == 3 ? (e4 >> 1) : (e4 << (23 - 8 * BYTE));
    const uint32_t b = sg8 << (31 - K);
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(r) : "r"(0x7F800000u), "r"(a), "r"(b));
    return __uint_as_float(r);
}

// fl32(norm * p) followed by a separate binary32 add (p = +-2^(c-s) or +-0)
__device__ __forceinline__ float add_scaled(float acc, float norm, float p) {
    return __fadd_rn(acc, __fmul_rn(norm, p));
}

// One worker's contribution to the 1024 entries of a tile.  The caller guarantees
// |norm| >= 2^(s-126): every product norm * 2^(c-s), c >= 1, is then a normal number, hence exact,
// and one fused multiply-add gives the bits of the multiplication followed by the addition.
// kWide: some code of the tile is above 7, the exponent bytes come from arithmetic instead of the
// byte-permute table.
template <bool kWide>
__device__ __forceinline__ void add_worker_tile(V8 (&acc)[4], const uint32_t (&nb)[4],
                                                const uint32_t (&sg)[4], const float norm,
                                                const uint32_t tbl_lo, const uint32_t tbl_hi,
                                                const uint32_t kexp) {
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        uint32_t lo4, hi4;
        if (kWide) {
            level_exp_bytes(nb[it], kexp, lo4, hi4);
        } else {
            lo4 = __byte_perm(tbl_lo, tbl_hi, nb[it]);
            hi4 = __byte_perm(tbl_lo, tbl_hi, nb[it] >> 16);
        }
        float* a = reinterpret_cast<float*>(acc[it].v);
        a[0] = __fmaf_rn(norm, pow2_signed<0, 0>(lo4, sg[it]), a[0]);
        a[1] = __fmaf_rn(norm, pow2_signed<1, 1>(lo4, sg[it]), a[1]);
        a[2] = __fmaf_rn(norm, pow2_signed<2, 2>(lo4, sg[it]), a[2]);
        a[3] = __fmaf_rn(norm, pow2_signed<3, 3>(lo4, sg[it]), a[3]);
        a[4] = __fmaf_rn(norm, pow2_signed<0, 4>(hi4, sg[it]), a[4]);
        a[5] = __fmaf_rn(norm, pow2_signed<1, 5>(hi4, sg[it]), a[5]);
        a[6] = __fmaf_rn(norm, pow2_signed<2, 6>(hi4, sg[it]), a[6]);
        a[7] = __fmaf_rn(norm, pow2_signed<3, 7>(hi4, sg[it]), a[7]);
    }
}

// a worker's planes of one tile as a lane holds them: the nibble words of its 4 x 8 entries and,
// per group of 8, the byte of the sign plane with their sign bits
struct WorkerTile {
    uint32_t nb[4];
    uint32_t sg[4];
    float norm;
};

__device__ __forceinline__ void load_worker_tile(WorkerTile& t, const DitherPlanes& planes,
                                                 const int i, const uint64_t base, const int b,
                                                 const int lane) {
    const uint32_t* lv = reinterpret_cast<const uint32_t*>(planes.level[i] + (base >> 1));
    const uint8_t* sb = reinterpret_cast<const uint8_t*>(planes.sign[i]) + (base >> 3);
    t.norm = __ldg(planes.norms[i] + b);
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        t.nb[it] = ld_stream_u32(lv + it * 32 + lane);
        t.sg[it] = sb[it * 32 + lane];
    }
}

__device__ __forceinline__ void add_worker(V8 (&acc)[4], const WorkerTile& t,
                                           const uint32_t tbl_lo, const uint32_t tbl_hi,
                                           const uint32_t kexp) {
    const uint32_t high = (t.nb[0] | t.nb[1] | t.nb[2] | t.nb[3]) & 0x88888888u;
    if (__any_sync(0xFFFFFFFFu, high != 0u))
        add_worker_tile<true>(acc, t.nb, t.sg, t.norm, tbl_lo, tbl_hi, kexp);
    else
        add_worker_tile<false>(acc, t.nb, t.sg, t.norm, tbl_lo, tbl_hi, kexp);
}

// The same for a piece of 256 entries (8 per lane; base a multiple of 256): one nibble word and one
// byte of the sign plane per lane and worker.  Used at the end of the vector, see the kernel.
template <bool kFromAcc>
__device__ __forceinline__ void aggregate_small_piece(const DitherPlanes& planes, const int n,
                                                      const uint64_t base, const int b,
                                                      const uint32_t tbl_lo, const uint32_t tbl_hi,
                                                      const uint32_t kexp,
                                                      float* __restrict__ out, const int lane) {
    V8 acc;
    if (kFromAcc) acc = ld_stream_v8(out + base + lane * 8);
    else {
#pragma unroll
        for (int c = 0; c < 8; ++c) acc.v[c] = 0u;
    }
    float* a = reinterpret_cast<float*>(acc.v);
    uint32_t nb = ld_stream_u32(planes.level[0] + (base >> 1) + lane * 4);
    uint32_t sg = reinterpret_cast<const uint8_t*>(planes.sign[0])[(base >> 3) + lane];
    float norm = __ldg(planes.norms[0] + b);
    for (int i = 0; i < n; ++i) {
        uint32_t nb_n = 0u, sg_n = 0u;
        float norm_n = 0.f;
        if (i + 1 < n) {
            nb_n = ld_stream_u32(planes.level[i + 1] + (base >> 1) + lane * 4);
            sg_n = reinterpret_cast<const uint8_t*>(planes.sign[i + 1])[(base >> 3) + lane];
            norm_n = __ldg(planes.norms[i + 1] + b);
        }
        uint32_t lo4, hi4;
        if (__any_sync(0xFFFFFFFFu, (nb & 0x88888888u) != 0u)) {
            level_exp_bytes(nb, kexp, lo4, hi4);
        } else {
            lo4 = __byte_perm(tbl_lo, tbl_hi, nb);
            hi4 = __byte_perm(tbl_lo, tbl_hi, nb >> 16);
        }
        a[0] = __fmaf_rn(norm, pow2_signed<0, 0>(lo4, sg), a[0]);
        a[1] = __fmaf_rn(norm, pow2_signed<1, 1>(lo4, sg), a[1]);
        a[2] = __fmaf_rn(norm, pow2_signed<2, 2>(lo4, sg), a[2]);
        a[3] = __fmaf_rn(norm, pow2_signed<3, 3>(lo4, sg), a[3]);
        a[4] = __fmaf_rn(norm, pow2_signed<0, 4>(hi4, sg), a[4]);
        a[5] = __fmaf_rn(norm, pow2_signed<1, 5>(hi4, sg), a[5]);
        a[6] = __fmaf_rn(norm, pow2_signed<2, 6>(hi4, sg), a[6]);
        a[7] = __fmaf_rn(norm, pow2_signed<3, 7>(hi4, sg), a[7]);
        nb = nb_n;
        sg = sg_n;
        norm = norm_n;
    }
    st_stream_v8(out + base + lane * 8, acc);
}

// Warps 0 .. big_tiles-1 take one tile of 1024 entries each; the entries after those tiles are cut
// into pieces of 256, one per warp.  Blocks start in index order, so the small pieces run last
// and fill the SMs evenly while the grid drains: a warp's life is long here (n workers per tile),
// and with whole tiles to the end the SMs were busy only three quarters of the kernel's duration.
// grid: ceil((big_tiles + small pieces) / warps per block)
template <bool kFromAcc>
__global__ void __launch_bounds__(kBlockThreads)
nd_aggregate_kernel(const __grid_constant__ DitherPlanes planes, const int n, const uint64_t d,
                    const uint64_t* __restrict__ off, const int B, const int s,
                    const uint64_t big_tiles, float* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = (uint64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const bool big = warp < big_tiles;
    const uint64_t len = big ? kTile : kTile / 4;
    const uint64_t base = big ? warp * kTile : big_tiles * kTile + (warp - big_tiles) * (kTile / 4);
    if (base >= d) return;
    const bool full = (base + len <= d);
    int b = find_bucket(off, B, base);

    // The vector path needs a whole piece inside one bucket whose norms are all finite and either
    // zero or at least 2^(s-126) (see add_worker_tile); anything else takes the scalar path.
    bool vector = full && __ldg(off + b + 1) >= base + len;
    if (vector) {
        const float fused_min = __uint_as_float((uint32_t)(s + 1) << 23);   // 2^(s-126)
        bool ok = true;
        for (int i = lane; i < n; i += 32) {
            const float a = fabsf(__ldg(planes.norms[i] + b));
            ok = ok && (a == 0.f || (a >= fused_min && a <= 3.40282347e38f));
        }
        vector = __all_sync(0xFFFFFFFFu, ok);
    }

    if (vector) {
        const uint32_t kexp = (uint32_t)(127 - s);
        // exponent bytes of 2^(c-s) for c = 0..7 (0 for c = 0): a byte-permute with the four level
        // nibbles as selector looks four of them up at once; codes 8..15 take the arithmetic path
        uint32_t tbl_lo = 0, tbl_hi = 0;
#pragma unroll
        for (int c = 1; c < 8; ++c) {
            const uint32_t e = (uint32_t)c + kexp;
            if (c < 4) tbl_lo |= e << (8 * c); else tbl_hi |= e << (8 * (c - 4));
        }
        if (!big) {
            aggregate_small_piece<kFromAcc>(planes, n, base, b, tbl_lo, tbl_hi, kexp, out, lane);
            return;
        }
        V8 acc[4];
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            if (kFromAcc) acc[it] = ld_stream_v8(out + base + it * 256 + lane * 8);
            else {
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[it].v[c] = 0u;
            }
        }
        // software pipeline over the workers, two register sets in turn: the planes of worker
        // i+1 are in flight while worker i is decoded
        WorkerTile ta, tb;
        load_worker_tile(ta, planes, 0, base, b, lane);
        for (int i = 0; i < n; i += 2) {
            const bool second = i + 1 < n;
            if (second) load_worker_tile(tb, planes, i + 1, base, b, lane);
            add_worker(acc, ta, tbl_lo, tbl_hi, kexp);
            if (second) {
                if (i + 2 < n) load_worker_tile(ta, planes, i + 2, base, b, lane);
                add_worker(acc, tb, tbl_lo, tbl_hi, kexp);
            }
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) st_stream_v8(out + base + it * 256 + lane * 8, acc[it]);
        return;
    }

    // the piece spans several buckets or is ragged: scalar, per-lane bucket cursor
    const uint64_t end = full ? base + len : d;
    uint64_t bend = __ldg(off + b + 1);
    for (uint64_t j = base + lane; j < end; j += 32) {
        while (j >= bend) { ++b; bend = __ldg(off + b + 1); }
        float a = kFromAcc ? out[j] : 0.f;
        for (int i = 0; i < n; ++i) {
            const float norm = __ldg(planes.norms[i] + b);
            const uint32_t c = (planes.level[i][j >> 1] >> (4 * (j & 1))) & 0xFu;
            const uint32_t sg = (planes.sign[i][j >> 5] >> (j & 31)) & 1u;
            const uint32_t pb = (c ? ((c + 127u - (uint32_t)s) << 23) : 0u) | (sg << 31);
            // level 0 is the value 0 whatever the norm; any other level is norm * 2^(c-s) as it
            // comes, so a norm that is not finite shows in the sum
            a = c ? add_scaled(a, norm, __uint_as_float(pb)) : __fadd_rn(a, __uint_as_float(pb));
        }
        NC_STORE(out + j, a);
    }
}

struct NormLists {
    const float* norms[NC_MAX_WORKERS];
};

// status += number of the n * B norms that are inf or NaN; grid: (ceil(B / threads), n)
__global__ void __launch_bounds__(kBlockThreads)
nd_norm_status_kernel(const __grid_constant__ NormLists lists, const int B,
                      uint32_t* __restrict__ status) {
    const int b = blockIdx.x * kBlockThreads + threadIdx.x;
    const bool bad = b < B && !(fabsf(lists.norms[blockIdx.y][b]) <= 3.40282347e38f);
    const uint32_t votes = __ballot_sync(0xFFFFFFFFu, bad);
    if ((threadIdx.x & 31) == 0 && votes) atomicAdd(status, (uint32_t)__popc(votes));
}

inline unsigned nd_tile_blocks(uint64_t d) {
    const uint64_t tiles = (d + kTile - 1) / kTile;
    return (unsigned)((tiles + kWarpsPerBlock - 1) / kWarpsPerBlock);
}

inline uint64_t nd_tiles(uint64_t d) { return (d + kTile - 1) / kTile; }

// The aggregate kernel runs in small blocks (2 warps).  Tiles of 1024 entries except for the last
// `nd_small_region_tiles` tiles' worth of entries, which are cut into pieces of 256: half a wave
// of resident warps (4 blocks of 8 warps' worth per SM), and nothing when all tiles are resident
// at once anyway.
constexpr int kAggregateThreads = 64;

inline uint64_t nd_aggregate_big_tiles(uint64_t d) {
    const uint64_t tiles = nd_tiles(d);
    const uint64_t resident = (uint64_t)device_sm_count() * 32u;
    if (tiles <= resident) return tiles;
    return tiles - resident / 2;
}

inline unsigned nd_aggregate_blocks(uint64_t d, uint64_t big_tiles) {
    const uint64_t rest = d > big_tiles * kTile ? d - big_tiles * kTile : 0;
    const uint64_t warps = big_tiles + (rest + kTile / 4 - 1) / (kTile / 4);
    const uint64_t per = kAggregateThreads / 32;
    return (unsigned)((warps + per - 1) / per);
}

}  // namespace natcomp

using namespace natcomp;

extern "C" {

size_t nd_batch_workspace_bytes(size_t d, int num_buckets, int n) {
    if (num_buckets < 0) num_buckets = 0;
    if (n < 1) n = 1;
    const uint64_t tiles = nd_tiles(d);
    // per worker: one 64-bit partial per (tile, bucket) overlap; shared: the tile -> bucket map
    return (size_t)n * round_up16((tiles + (uint64_t)num_buckets + 1) * 8) + round_up16(tiles * 4);
}

size_t nd_workspace_bytes(size_t d, int num_buckets) {
    return nd_batch_workspace_bytes(d, num_buckets, 1);
}

// shared argument checks of the dithering compress calls; fills `batch`
static nc_status nd_check_batch(const float* const* xs, size_t d, const uint64_t* bucket_off, int B,
                                const uint32_t* workers, float* const* norms,
                                uint8_t* const* levels, uint32_t* const* signs, int n,
                                bool need_planes, DitherBatch* batch) {
    if (!xs || !bucket_off || !norms || n < 1 || n > NC_MAX_WORKERS || B < 1) return NC_ERR_INVALID;
    if (need_planes && (!workers || !levels || !signs)) return NC_ERR_INVALID;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if ((uintptr_t)bucket_off & 7u) return NC_ERR_ALIGN;
    for (int i = 0; i < n; ++i) {
        if (!xs[i] || !norms[i]) return NC_ERR_INVALID;
        if (!aligned32(xs[i]) || !aligned4(norms[i])) return NC_ERR_ALIGN;
        batch->x[i] = xs[i];
        batch->norms[i] = norms[i];
        batch->level[i] = nullptr;
        batch->sign[i] = nullptr;
        batch->worker[i] = 0;
        if (need_planes) {
            if (!levels[i] || !signs[i]) return NC_ERR_INVALID;
            if (!aligned16(levels[i]) || !aligned16(signs[i])) return NC_ERR_ALIGN;
            batch->level[i] = levels[i];
            batch->sign[i] = signs[i];
            batch->worker[i] = workers[i];
        }
    }
    return NC_OK;
}

// debug build: what a dithering compress call may write
static void nd_scope_batch(BoundsScope& scope, const DitherBatch& batch, uint64_t d, int B, int n,
                           bool norms, bool planes, void* workspace) {
    for (int i = 0; i < n; ++i) {
        if (norms) scope.add(batch.norms[i], 4 * (size_t)B);
        if (planes) {
            scope.add(batch.level[i], nd_level_bytes(d));
            scope.add(batch.sign[i], nc_sign_bytes(d));
        }
    }
    if (workspace) scope.add(workspace, nd_batch_workspace_bytes(d, B, n));
}

// the two norm launches; returns the tile -> bucket map they leave in the workspace
static uint32_t* nd_launch_norms(const DitherBatch& batch, uint64_t d, const uint64_t* bucket_off,
                                 int B, int p, int n, void* workspace, uint32_t* status,
                                 cudaStream_t stream) {
    const uint64_t tiles = nd_tiles(d);
    const uint64_t slot_stride = round_up16((tiles + (uint64_t)B + 1) * 8) / 8;
    uint64_t* slots = reinterpret_cast<uint64_t*>(workspace);
    uint32_t* tile_bucket = reinterpret_cast<uint32_t*>(slots + (uint64_t)n * slot_stride);
    const unsigned resident = 2u * (unsigned)device_sm_count();
    const dim3 ngrid(nd_tile_blocks(d) < resident ? nd_tile_blocks(d) : resident, (unsigned)n);
    const dim3 fgrid((unsigned)B, (unsigned)n);
    if (p == 1) {
        nd_norm_partials_kernel<1><<<ngrid, kBlockThreads, 0, stream>>>(
            batch, d, bucket_off, B, slots, slot_stride, tile_bucket);
        nd_norm_finalize_kernel<1><<<fgrid, kBlockThreads, 0, stream>>>(batch, bucket_off, B,
                                                                        slots, slot_stride, status);
    } else if (p == 2) {
        nd_norm_partials_kernel<2><<<ngrid, kBlockThreads, 0, stream>>>(
            batch, d, bucket_off, B, slots, slot_stride, tile_bucket);
        nd_norm_finalize_kernel<2><<<fgrid, kBlockThreads, 0, stream>>>(batch, bucket_off, B,
                                                                        slots, slot_stride, status);
    } else {
        nd_norm_partials_kernel<NC_P_INF><<<ngrid, kBlockThreads, 0, stream>>>(
            batch, d, bucket_off, B, slots, slot_stride, tile_bucket);
        nd_norm_finalize_kernel<NC_P_INF><<<fgrid, kBlockThreads, 0, stream>>>(
            batch, bucket_off, B, slots, slot_stride, status);
    }
    return tile_bucket;
}

nc_status nd_norms_batch(const float* const* xs, size_t d, const uint64_t* bucket_off, int B, int p,
                         float* const* norms, int n, void* workspace, size_t workspace_bytes,
                         uint32_t* status, cudaStream_t stream) {
    if (p != 1 && p != 2 && p != NC_P_INF) return NC_ERR_UNSUPPORTED;
    DitherBatch batch;
    const nc_status st = nd_check_batch(xs, d, bucket_off, B, nullptr, norms, nullptr, nullptr, n,
                                        false, &batch);
    if (st != NC_OK) return st;
    if (d == 0) return NC_OK;
    if (!workspace) return NC_ERR_INVALID;
    if (!aligned16(workspace) || !aligned4(status)) return NC_ERR_ALIGN;
    if (workspace_bytes < nd_batch_workspace_bytes(d, B, n)) return NC_ERR_WORKSPACE;
    BoundsScope scope;
    nd_scope_batch(scope, batch, d, B, n, true, false, workspace);
    scope.commit(stream);
    nd_launch_norms(batch, d, bucket_off, B, p, n, workspace, status, stream);
    return launch_status();
}

nc_status nd_round_batch(const float* const* xs, size_t d, const uint64_t* bucket_off, int B, int s,
                         uint64_t seed, const uint32_t* workers, const float* const* norms,
                         uint8_t* const* levels, uint32_t* const* signs, int n,
                         cudaStream_t stream) {
    if (s < 1 || s > 15) return NC_ERR_INVALID;
    DitherBatch batch;
    const nc_status st = nd_check_batch(xs, d, bucket_off, B, workers,
                                        const_cast<float* const*>(norms), levels, signs, n, true,
                                        &batch);
    if (st != NC_OK) return st;
    if (d == 0) return NC_OK;
    const PhiloxKeys keys = make_philox_keys(seed);
    const dim3 grid(nd_tile_blocks(d), (unsigned)n);
    BoundsScope scope;
    nd_scope_batch(scope, batch, d, B, n, false, true, nullptr);
    scope.commit(stream);
    nd_round_pack_kernel<true><<<grid, kBlockThreads, 0, stream>>>(batch, d, bucket_off, B, s, keys,
                                                                   nullptr);
    return launch_status();
}

nc_status nd_compress_batch(const float* const* xs, size_t d, const uint64_t* bucket_off, int B,
                            int p, int s, uint64_t seed, const uint32_t* workers,
                            float* const* norms, uint8_t* const* levels, uint32_t* const* signs,
                            int n, void* workspace, size_t workspace_bytes, uint32_t* status,
                            cudaStream_t stream) {
    if (s < 1 || s > 15) return NC_ERR_INVALID;
    if (p != 1 && p != 2 && p != NC_P_INF) return NC_ERR_UNSUPPORTED;
    DitherBatch batch;
    const nc_status st = nd_check_batch(xs, d, bucket_off, B, workers, norms, levels, signs, n,
                                        true, &batch);
    if (st != NC_OK) return st;
    if (d == 0) return NC_OK;
    if (!workspace) return NC_ERR_INVALID;
    if (!aligned16(workspace) || !aligned4(status)) return NC_ERR_ALIGN;
    if (workspace_bytes < nd_batch_workspace_bytes(d, B, n)) return NC_ERR_WORKSPACE;
    BoundsScope scope;
    nd_scope_batch(scope, batch, d, B, n, true, true, workspace);
    scope.commit(stream);
    const uint32_t* tile_bucket =
        nd_launch_norms(batch, d, bucket_off, B, p, n, workspace, status, stream);
    const PhiloxKeys keys = make_philox_keys(seed);
    const dim3 grid(nd_tile_blocks(d), (unsigned)n);
    nd_round_pack_kernel<false><<<grid, kBlockThreads, 0, stream>>>(batch, d, bucket_off, B, s,
                                                                    keys, tile_bucket);
    return launch_status();
}

nc_status nd_compress(const float* x, size_t d, const uint64_t* bucket_off, int B, int p, int s,
                      uint64_t seed, uint32_t worker, float* norms, uint8_t* level,
                      uint32_t* sign, void* workspace, size_t workspace_bytes, uint32_t* status,
                      cudaStream_t stream) {
    if (!x || !norms || !level || !sign) return NC_ERR_INVALID;
    return nd_compress_batch(&x, d, bucket_off, B, p, s, seed, &worker, &norms, &level, &sign, 1,
                             workspace, workspace_bytes, status, stream);
}

static nc_status nd_check_planes(const float* const* norms, const uint8_t* const* levels,
                                 const uint32_t* const* signs, int n, DitherPlanes* planes) {
    for (int i = 0; i < n; ++i) {
        if (!norms[i] || !levels[i] || !signs[i]) return NC_ERR_INVALID;
        if (!aligned4(norms[i]) || !aligned16(levels[i]) || !aligned16(signs[i]))
            return NC_ERR_ALIGN;
        planes->norms[i] = norms[i];
        planes->level[i] = levels[i];
        planes->sign[i] = signs[i];
    }
    return NC_OK;
}

nc_status nd_aggregate(const float* const* norms, const uint8_t* const* levels,
                       const uint32_t* const* signs, int n, size_t d, const uint64_t* bucket_off,
                       int B, int s, float* out, cudaStream_t stream) {
    if (!norms || !levels || !signs || !bucket_off || !out || n < 1 || n > NC_MAX_WORKERS ||
        B < 1 || s < 1 || s > 15)
        return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned32(out) || ((uintptr_t)bucket_off & 7u)) return NC_ERR_ALIGN;
    DitherPlanes planes;
    const nc_status st = nd_check_planes(norms, levels, signs, n, &planes);
    if (st != NC_OK) return st;
    const uint64_t big_tiles = nd_aggregate_big_tiles(d);
    BoundsScope scope;
    scope.add(out, 4 * (size_t)d);
    scope.commit(stream);
    nd_aggregate_kernel<false><<<nd_aggregate_blocks(d, big_tiles), kAggregateThreads, 0, stream>>>(
        planes, n, (uint64_t)d, bucket_off, B, s, big_tiles, out);
    return launch_status();
}

nc_status nd_norm_status(const float* const* norms, int n, int B, uint32_t* status,
                         cudaStream_t stream) {
    if (!norms || !status || n < 1 || n > NC_MAX_WORKERS || B < 0) return NC_ERR_INVALID;
    if (!aligned4(status)) return NC_ERR_ALIGN;
    if (B == 0) return NC_OK;
    NormLists lists;
    for (int i = 0; i < n; ++i) {
        if (!norms[i]) return NC_ERR_INVALID;
        if (!aligned4(norms[i])) return NC_ERR_ALIGN;
        lists.norms[i] = norms[i];
    }
    const dim3 grid((unsigned)((B + kBlockThreads - 1) / kBlockThreads), (unsigned)n);
    nd_norm_status_kernel<<<grid, kBlockThreads, 0, stream>>>(lists, B, status);
    return launch_status();
}

nc_status nd_decode_accumulate(const float* norms, const uint8_t* level, const uint32_t* sign,
                               size_t d, const uint64_t* bucket_off, int B, int s, float* acc,
                               cudaStream_t stream) {
    if (!norms || !level || !sign || !bucket_off || !acc || B < 1 || s < 1 || s > 15)
        return NC_ERR_INVALID;
    if (d == 0) return NC_OK;
    if (d > ((uint64_t)1 << 40)) return NC_ERR_INVALID;
    if (!aligned32(acc) || ((uintptr_t)bucket_off & 7u)) return NC_ERR_ALIGN;
    DitherPlanes planes;
    const nc_status st = nd_check_planes(&norms, &level, &sign, 1, &planes);
    if (st != NC_OK) return st;
    const uint64_t big_tiles = nd_aggregate_big_tiles(d);
    BoundsScope scope;
    scope.add(acc, 4 * (size_t)d);
    scope.commit(stream);
    nd_aggregate_kernel<true><<<nd_aggregate_blocks(d, big_tiles), kAggregateThreads, 0, stream>>>(
        planes, 1, (uint64_t)d, bucket_off, B, s, big_tiles, acc);
    return launch_status();
}

}  // extern "C"

// ---- nd_compress without a caller-provided workspace ------------------------------------
//
// Scratch for callers that cannot allocate device memory: a fixed array that lives in the
// library image on every GPU that loads it.  In host code `g_nd_static_scratch` is only a
// handle for the runtime; its device address is looked up once per device with
// cudaGetSymbolAddress and passed to the kernels like any other workspace pointer.
namespace natcomp {

constexpr size_t kStaticScratchBytes = (size_t)1 << 20;   // 1 MiB

static __device__ __align__(256) unsigned char g_nd_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_static_scratch_addr[kMaxDevices];   // per device ordinal; 0 = not looked up yet

// Device address of the scratch array on the current device (nullptr on failure).
static void* static_scratch_address() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    void* p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (p) return p;
    if (cudaGetSymbolAddress(&p, g_nd_static_scratch) != cudaSuccess || !p) return nullptr;
    __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);
    return p;
}

}  // namespace natcomp

extern "C" {

size_t nd_static_scratch_bytes(void) { return kStaticScratchBytes; }

nc_status nd_compress_static(const float* x, size_t d, const uint64_t* bucket_off, int B, int p,
                             int s, uint64_t seed, uint32_t worker, float* norms, uint8_t* level,
                             uint32_t* sign, uint32_t* status, cudaStream_t stream) {
    if (!x || !bucket_off || !norms || !level || !sign || B < 1) return NC_ERR_INVALID;
    if (nd_workspace_bytes(d, B) > kStaticScratchBytes) return NC_ERR_TOO_LARGE;
    void* scratch = static_scratch_address();
    if (!scratch) return NC_ERR_CUDA;
    return nd_compress(x, d, bucket_off, B, p, s, seed, worker, norms, level, sign, scratch,
                       kStaticScratchBytes, status, stream);
}

}  // extern "C"

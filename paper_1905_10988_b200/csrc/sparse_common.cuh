// Pieces shared by the sparsifier kernels (independent per-coordinate selection) and the
// exact-count selection kernels (radix select): argument blocks, workspace layout, warp helpers,
// the level rounding of Def. 3 for a single gathered entry, and the host routine that turns a
// selection bitmask into the compact list.
#pragma once
#include "common.cuh"
#include "philox.cuh"

namespace natcomp {

constexpr int kScanThreads = 1024;

struct SparseBatch {
    const float* x[NC_MAX_WORKERS];
    uint32_t* idx[NC_MAX_WORKERS];
    uint8_t* codes[NC_MAX_WORKERS];
    uint32_t* count[NC_MAX_WORKERS];
    float* norm[NC_MAX_WORKERS];
    uint32_t worker[NC_MAX_WORKERS];
};

struct SparseWorkspace {
    uint32_t* bitmask;      // tiles * 32 words
    uint32_t* block_count;   // one per block of 8 tiles (the exclusive offset after the scan)
    uint64_t* block_partial; // one per block of 8 tiles
    uint8_t* stage;          // 64 bytes per group of 8 tiles: see kStageEntries
    uint8_t* tmp_codes;     // cap bytes
};

__host__ __device__ inline uint64_t sparse_tiles(uint64_t d) { return (d + kTile - 1) / kTile; }

inline size_t sparse_ws_bytes(uint64_t d, uint64_t cap) {
    const uint64_t t = sparse_tiles(d);
    return round_up16(t * 128) + round_up16(t * 4) + round_up16(t * 8) +
           round_up16(((t + 7) / 8) * 64) + round_up16(cap);
}

__host__ __device__ inline SparseWorkspace sparse_ws_carve(void* ws, uint64_t d) {
    const uint64_t t = sparse_tiles(d);
    char* p = reinterpret_cast<char*>(ws);
    SparseWorkspace w;
    w.bitmask = reinterpret_cast<uint32_t*>(p);      p += round_up16(t * 128);
    w.block_count = reinterpret_cast<uint32_t*>(p);   p += round_up16(t * 4);
    w.block_partial = reinterpret_cast<uint64_t*>(p); p += round_up16(t * 8);
    w.stage = reinterpret_cast<uint8_t*>(p);          p += round_up16(((t + 7) / 8) * 64);
    w.tmp_codes = reinterpret_cast<uint8_t*>(p);
    return w;
}

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
// warp-wide integer reductions: one redux instruction each
__device__ __forceinline__ uint32_t warp_max_u(uint32_t v) {
    return __reduce_max_sync(0xFFFFFFFFu, v);
}
__device__ __forceinline__ uint32_t warp_sum_u(uint32_t v) {
    return __reduce_add_sync(0xFFFFFFFFu, v);
}

// Lists the set bits of a 1024-bit tile mask (lane l holds word l) in ascending order into the
// warp's shared-memory list as in-tile positions; returns how many there are.  After this the
// t-th kept entry can be handled by lane t mod 32, so the gathers from x run in parallel
// instead of one dependent load per set bit of a lane's own word.
__device__ __forceinline__ uint32_t warp_list_positions(uint32_t word, int lane,
                                                        uint16_t* __restrict__ list) {
    const uint32_t cnt = __popc(word);
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    uint32_t at = incl - cnt;
    while (word) {
        const int bit = __ffs(word) - 1;
        word &= word - 1;
        list[at++] = (uint16_t)(lane * 32 + bit);
    }
    __syncwarp();
    return __shfl_sync(0xFFFFFFFFu, incl, 31);
}

// Lists of kept positions for a group of 8 tiles (8192 coordinates, the unit of the per-block
// counts): at 1 % density a single tile has about ten kept entries, so the sparse passes give a
// warp a whole group and work on the listed entries with all lanes busy.
// >= kTile: one tile always fits into an empty list.  Not larger either: the level filter is bound
// by its gathers and its shared-memory traffic and is sensitive to how the driver splits L1 and
// shared memory (with 4 KB lists and one more kilobyte per block it got five resident blocks, a
// 228 KB carve-out and 24 KB of L1, and took 640 instead of 430 us on 8 x 2^28 coordinates).
constexpr uint32_t kGroupListCap = 1024;

// The level filter of the compact form leaves the codes of a group's surviving entries in the
// workspace, so that the emit pass needs neither the gather from x nor the generator again:
// 64 bytes per group = up to 126 four-bit codes in ascending position order (code r in bits
// 4 (r mod 2).. of byte r / 2) and, in byte 63, 1 if the codes are there.  A group with more
// surviving entries, or more than 128 kept ones, is not staged and is emitted the long way.
constexpr uint32_t kStageEntries = 126;
constexpr uint32_t kStageBytes = 64;

// appends the positions (inside the group, tile w) of the set bits of `word` (lane l = word l of
// the tile) to list[at ..]; returns how many
__device__ __forceinline__ uint32_t group_list_append(uint32_t word, int lane, int w,
                                                      uint16_t* __restrict__ list, uint32_t at) {
    const uint32_t cnt = __popc(word);
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    uint32_t pos = at + incl - cnt;
    while (word) {
        const int bit = __ffs(word) - 1;
        word &= word - 1;
        list[pos++] = (uint16_t)(w * kTile + lane * 32 + bit);
    }
    return __shfl_sync(0xFFFFFFFFu, incl, 31);
}

// The same for all 8 tiles of a group at once (lane l holds word l of every tile): the per-tile
// prefix sums over the lanes run as ONE scan over two 64-bit values that carry the eight counts
// in 16-bit fields (a tile has at most 1024 set bits, so no field overflows), 24 shuffles instead
// of the 80 that eight separate scans and eight warp sums take; shuffles share the queue of the
// shared-memory instructions, which is what these kernels wait for.  tile_cnt[w] = kept entries of
// tile w; returns their sum.  The list is written only if it fits (sum <= kGroupListCap).
__device__ __forceinline__ uint32_t group_list_build(const uint32_t (&word)[8], const int lane,
                                                     uint16_t* __restrict__ list,
                                                     uint32_t (&tile_cnt)[8]) {
    unsigned long long ia = 0, ib = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        ia |= (unsigned long long)__popc(word[w]) << (16 * w);
        ib |= (unsigned long long)__popc(word[w + 4]) << (16 * w);
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long va = __shfl_up_sync(0xFFFFFFFFu, ia, o);
        const unsigned long long vb = __shfl_up_sync(0xFFFFFFFFu, ib, o);
        if (lane >= o) {
            ia += va;
            ib += vb;
        }
    }
    const unsigned long long ta = __shfl_sync(0xFFFFFFFFu, ia, 31);
    const unsigned long long tb = __shfl_sync(0xFFFFFFFFu, ib, 31);
    uint32_t start[8], total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        tile_cnt[w] = (uint32_t)(((w < 4 ? ta : tb) >> (16 * (w & 3))) & 0xFFFFu);
        start[w] = total;
        total += tile_cnt[w];
    }
    if (total > kGroupListCap) return total;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        uint32_t wd = word[w];
        const uint32_t incl = (uint32_t)(((w < 4 ? ia : ib) >> (16 * (w & 3))) & 0xFFFFu);
        uint32_t pos = start[w] + incl - (uint32_t)__popc(wd);
        while (wd) {
            const int bit = __ffs(wd) - 1;
            wd &= wd - 1;
            list[pos++] = (uint16_t)(w * kTile + lane * 32 + bit);
        }
    }
    return total;
}

// A lane's 32 per-element bits in the load layout (bit 4k+c <-> element k*128 + 4*lane + c of
// the tile) -> canonical order: lane l returns the word of elements 32l .. 32l+31.
__device__ __forceinline__ uint32_t canonical_mask_word(uint32_t nib, int lane) {
    const uint32_t word = transpose_nibbles_8x8(nib, lane);   // lane 8g+k holds word 4k+g
    return __shfl_sync(0xFFFFFFFFu, word, 8 * (lane & 3) + (lane >> 2));
}

// For one tile per warp (all warps of the block must call): gathers the kept entries of the
// tile (mask word of lane l = elements 32l..32l+31), accumulates the norm partial of the scaled
// kept entries, and thread 0 writes the block's kept count and partial.  P = 1, 2 or NC_P_INF.
template <int P>
__device__ __forceinline__ void kept_count_and_partial(const uint32_t word, const int lane,
                                                       const float* __restrict__ x,
                                                       const uint64_t base, const float scale,
                                                       uint32_t* __restrict__ block_count,
                                                       uint64_t* __restrict__ block_partial) {
    __shared__ uint32_t s_cnt[kWarpsPerBlock];
    __shared__ uint64_t s_part[kWarpsPerBlock];
    __shared__ uint16_t s_list[kWarpsPerBlock][kTile];
    uint16_t* list = s_list[threadIdx.x >> 5];
    const uint32_t cnt = warp_sum_u(__popc(word));
    double dsum = 0.0;
    uint32_t vmax = 0;
    if (cnt <= 96u) {
        // few kept entries (the 1 % workloads): every lane walks the bits of its own word
        uint32_t w = word;
        while (w) {
            const int bit = __ffs(w) - 1;
            w &= w - 1;
            const float xs = __fmul_rn(scale, x[base + (uint64_t)(lane * 32 + bit)]);
            const uint32_t a = __float_as_uint(xs) & 0x7FFFFFFFu;
            if (P == NC_P_INF) vmax = max(vmax, a);
            else if (P == 1) dsum += (double)__uint_as_float(a);
            else dsum = fma((double)xs, (double)xs, dsum);
        }
    } else {
        // many: list the positions so that the gathers spread evenly over the lanes
        warp_list_positions(word, lane, list);
        for (uint32_t t = lane; t < cnt; t += 32) {
            const float xs = __fmul_rn(scale, x[base + list[t]]);
            const uint32_t a = __float_as_uint(xs) & 0x7FFFFFFFu;
            if (P == NC_P_INF) vmax = max(vmax, a);
            else if (P == 1) dsum += (double)__uint_as_float(a);
            else dsum = fma((double)xs, (double)xs, dsum);
        }
    }
    uint64_t part;
    if (P == NC_P_INF) part = (uint64_t)warp_max_u(vmax);
    else part = (uint64_t)__double_as_longlong(warp_sum_d(dsum));
    if (lane == 0) {
        s_cnt[threadIdx.x >> 5] = cnt;
        s_part[threadIdx.x >> 5] = part;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t c = 0, m = 0;
        double sum = 0.0;
        for (int w = 0; w < kWarpsPerBlock; ++w) {     // fixed order
            c += s_cnt[w];
            if (P == NC_P_INF) m = max(m, (uint32_t)s_part[w]);
            else sum += __longlong_as_double((long long)s_part[w]);
        }
        block_count[blockIdx.x] = c;
        block_partial[blockIdx.x] =
            (P == NC_P_INF) ? (uint64_t)m : (uint64_t)__double_as_longlong(sum);
    }
}

// drop <- 2 * drop + carry(word + neg_thr): shifts in a 1 iff word >= 2^32 - neg_thr, i.e. iff the
// coordinate's stream word is not below the keep threshold
__device__ __forceinline__ void shift_in_drop_bit(uint32_t& drop, uint32_t word, uint32_t neg_thr) {
    asm("{\n\t.reg .u32 t;\n\tadd.cc.u32 t, %1, %2;\n\taddc.u32 %0, %0, %0;\n\t}"
        : "+r"(drop)
        : "r"(word), "r"(neg_thr));
}

struct Scale {
    float pre;       // 1, or 2^24 when the norm is subnormal (its reciprocal would overflow)
    float rinv;      // fl32(1 / (norm * pre)), or 0 for a degenerate norm
    uint32_t smax;   // s, or 0 for a degenerate norm (0 or not finite: every code is 0)
};

__device__ __forceinline__ Scale make_scale(float norm, int s) {
    Scale r;
    const bool ok = (norm > 0.f) && (norm <= 3.40282347e38f);
    r.pre = norm < 1.17549435e-38f ? 16777216.f : 1.f;
    r.rinv = ok ? __fdiv_rn(1.0f, __fmul_rn(norm, r.pre)) : 0.f;
    r.smax = ok ? (uint32_t)s : 0u;
    return r;
}

// same rounding rule as the dense dithering kernel (Def. 3, natural levels)
__device__ __forceinline__ uint32_t sparse_level_code(uint32_t bits, uint32_t rnd, const Scale sc,
                                                      float pow2s) {
    const float ax = __uint_as_float(bits & 0x7FFFFFFFu);
    const float y = __fmul_rn(__fmul_rn(ax, sc.pre), sc.rinv);   // the scaling by pre is exact
    const float z = __fmul_rn(y, pow2s);
    // below 2 the bottom interval [0, 2^(1-s)] is mapped onto [1, 2): w = 1 + z/2 (> z there);
    // from 2 on 1 + z/2 <= z, so one max selects the right branch
    const float w = fmaxf(z, __fmaf_rz(z, 0.5f, 1.0f));
    const uint32_t t = __float_as_uint(w) + (~rnd & 0x7FFFFFu) - 0x3F800000u;
    return min(t >> 23, sc.smax);
}

__host__ __device__ inline int code_value_bits(int s) {
    int nb = 0;
    while ((1 << nb) < s) ++nb;
    return nb;
}

// the stream word of element j (any domain), for gathered entries
__device__ __forceinline__ uint32_t stream_word_at(uint64_t j, uint32_t worker, uint32_t domain,
                                                   const PhiloxKeys& keys) {
    uint32_t r4[4];
    stream_words4(j >> 2, worker, domain, keys, r4);
    return (j & 3) == 0 ? r4[0] : (j & 3) == 1 ? r4[1] : (j & 3) == 2 ? r4[2] : r4[3];
}

// One block of kScanThreads threads: in-place exclusive scan of counts[0, n); every thread gets
// the total.  Chunks of 4 * kScanThreads values, one coalesced 16-byte load per thread and chunk
// (the array is 16-byte aligned and allocated up to a multiple of 4 entries).
__device__ __forceinline__ uint32_t block_exclusive_scan_inplace(uint32_t* __restrict__ counts,
                                                                 const uint64_t n) {
    __shared__ uint32_t s_warp[32];
    const int t = threadIdx.x;
    const int lane = t & 31;
    const int warp = t >> 5;
    uint32_t carry = 0;
    for (uint64_t c0 = 0; c0 < n; c0 += 4ull * kScanThreads) {
        const uint64_t i = c0 + 4ull * t;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (i < n) v = *reinterpret_cast<const uint4*>(counts + i);
        if (i + 1 >= n) v.y = 0u;
        if (i + 2 >= n) v.z = 0u;
        if (i + 3 >= n) v.w = 0u;
        const uint32_t sum = v.x + v.y + v.z + v.w;
        uint32_t incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += u;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            uint32_t w = s_warp[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, w, o);
                if (lane >= o) w += u;
            }
            s_warp[lane] = w;
        }
        __syncthreads();
        const uint32_t run = carry + (warp ? s_warp[warp - 1] : 0u) + incl - sum;
        if (i < n) {
            uint4 o;
            o.x = run;
            o.y = o.x + v.x;
            o.z = o.y + v.y;
            o.w = o.z + v.z;
            *reinterpret_cast<uint4*>(counts + i) = o;
        }
        carry += s_warp[31];
        __syncthreads();
    }
    return carry;
}

// Given, per worker, the selection bitmask, the per-block kept counts and the norm partials in
// the workspace (what the select kernels leave): norm, level rounding, dropping of level-0
// entries, index list and code planes of the compact format.  Defined with the sparsifier
// kernels; launches only.
void sparse_compact_finish(const SparseBatch& batch, uint64_t d, float scale, int p, int s,
                           const PhiloxKeys& keys, uint64_t cap, char* ws, uint64_t ws_stride,
                           int n, cudaStream_t stream);

}  // namespace natcomp

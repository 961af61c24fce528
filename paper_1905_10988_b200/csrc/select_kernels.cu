// Selection of exactly q coordinates on the device, for sm_100a:
//   * the sparsifier with exactly q non-zeros (the paper's S^q: a uniformly random subset of
//     size q; here the q coordinates with the smallest selection-stream words), followed by
//     D_nat^{p,s} of Def. 3 in the compact list format;
//   * TopK followed by C_nat (the "TopK-C_nat" composition of the experiments): the K entries of
//     largest magnitude, each with the 9-bit code of Def. 1.
//
// Both are "the q smallest 32-bit keys, equal keys by ascending index" (key = the stream word,
// or the complemented magnitude bits).  Most-significant-digit radix select, no sort and no
// waiting between blocks:
//   hist x3   : histogram of the next digit (11, 11, 10 bits) over the keys that match the
//               digits fixed so far; per-block shared-memory histogram, flushed with integer atomics
//   choose x3 : one block finds the digit bin holding the q-th key and fixes it
//               (if few keys share the digits fixed after pass 0 or 1, the later passes are
//               skipped on the device and those keys are collected as candidates instead)
//   mark      : per 1024-element tile the masks "key < T" and "key == T" (T = the q-th key)
//   candidates: one block finishes the selection on the collected (key, coordinate) pairs
//   scan      : exclusive offsets of the per-block counts of "== T"
//   resolve   : final mask = "< T" plus the first r of the "== T" in index order; per-block
//               kept counts (and norm partials for the sparsifier)
// then the compaction kernels shared with the independent-selection sparsifier, or the TopK emit.
// Keys are recomputed (Philox) or re-read (x) in every pass; nothing of size d except the two
// bit masks is stored.
#include "sparse_common.cuh"

namespace natcomp {

constexpr int kSelBins = 2048;
constexpr int kSelPasses = 3;

__host__ __device__ constexpr int sel_shift(int pass) { return pass == 0 ? 21 : pass == 1 ? 10 : 0; }
__host__ __device__ constexpr int sel_bins(int pass) { return pass == 2 ? 1024 : 2048; }
// mask of the key bits fixed before this pass
__host__ __device__ constexpr uint32_t sel_fixed(int pass) {
    return pass == 0 ? 0u : pass == 1 ? 0xFFE00000u : 0xFFFFFC00u;
}

constexpr uint32_t kCandCap = 1u << 18;      // candidate list entries (8 bytes each)

struct SelectState {
    uint32_t prefix;        // digits fixed so far; after the last pass the q-th smallest key T
    uint32_t mode;          // 0: all three digit passes; 1 / 2: candidates collected after pass 0 / 1
    uint64_t remaining;     // how many keys to take among those matching the prefix
};

struct SelectWorkspace {
    uint32_t* eqmask;       // tiles * 32 words
    uint32_t* eq_block;     // one per block of 8 tiles
    uint32_t* hist;         // kSelPasses * kSelBins
    uint32_t* hist2;        // 3 * kSelBins: second digit of the keys in the three guessed first bins
    SelectState* state;
    uint32_t* count;        // listed entries (TopK)
    uint32_t* cand_count;
    uint2* cand;            // kCandCap pairs (key, coordinate)
};

inline size_t select_extra_bytes(uint64_t d) {
    const uint64_t t = sparse_tiles(d);
    return round_up16(t * 128) + round_up16(t * 4) + (size_t)(kSelPasses + 3) * kSelBins * 4 + 64 +
           (size_t)kCandCap * 8;
}

__host__ __device__ inline SelectWorkspace select_ws_carve(char* p, uint64_t d) {
    const uint64_t t = sparse_tiles(d);
    SelectWorkspace w;
    w.eqmask = reinterpret_cast<uint32_t*>(p);   p += round_up16(t * 128);
    w.eq_block = reinterpret_cast<uint32_t*>(p); p += round_up16(t * 4);
    w.hist = reinterpret_cast<uint32_t*>(p);     p += (size_t)kSelPasses * kSelBins * 4;
    w.hist2 = reinterpret_cast<uint32_t*>(p);    p += (size_t)3 * kSelBins * 4;
    w.state = reinterpret_cast<SelectState*>(p);
    w.count = reinterpret_cast<uint32_t*>(p + 32);
    w.cand_count = reinterpret_cast<uint32_t*>(p + 36);
    w.cand = reinterpret_cast<uint2*>(p + 64);
    return w;
}

// ---- key sources: load(k) gives the 4 keys of in-tile positions pos(lane, k, 0..3) ------------
// Stream keys are computed, not loaded, so a lane takes 32 consecutive coordinates and its 32
// per-key bits are a word of the tile mask as they are; keys read from memory keep the coalesced
// layout of the other kernels and their bits are transposed.
struct StreamKeys {          // selection-stream word of the coordinate
    static constexpr bool kCanonical = true;
    uint32_t worker;
    PhiloxKeys keys;
    struct Tile {
        PhiloxTile pt;
        uint32_t q_lo;
    };
    __device__ __forceinline__ Tile tile(uint64_t base, int lane) const {
        Tile t;
        t.pt = philox_tile((uint32_t)(base >> 34), worker, kDomainSelect, keys);
        t.q_lo = (uint32_t)(base >> 2) + (uint32_t)(lane * 8);
        return t;
    }
    __device__ __forceinline__ void load(const Tile& t, uint64_t, int, int k, uint64_t,
                                         uint32_t (&out)[4]) const {
        stream_words4_tile(t.q_lo + (uint32_t)k, t.pt, keys, out);
    }
    // the key of element k*128 + 4*lane + c of the tile alone (recomputed)
    __device__ __forceinline__ uint32_t key_at(const Tile& t, uint64_t, int, int k, int c) const {
        uint32_t out[4];
        stream_words4_tile(t.q_lo + (uint32_t)k, t.pt, keys, out);
        return c == 0 ? out[0] : c == 1 ? out[1] : c == 2 ? out[2] : out[3];
    }
};

struct MagnitudeKeys {       // largest |x| first: complement of the magnitude bits
    static constexpr bool kCanonical = false;
    const float* x;
    struct Tile {};
    __device__ __forceinline__ Tile tile(uint64_t, int) const { return Tile(); }
    __device__ __forceinline__ void load(const Tile&, uint64_t base, int lane, int k, uint64_t d,
                                         uint32_t (&out)[4]) const {
        const uint64_t j = base + (uint64_t)(k * 128 + lane * 4);
        if (j + 4 <= d) {
            const uint4 v = ld_stream_u4(x + j);
            out[0] = ~(v.x & 0x7FFFFFFFu);
            out[1] = ~(v.y & 0x7FFFFFFFu);
            out[2] = ~(v.z & 0x7FFFFFFFu);
            out[3] = ~(v.w & 0x7FFFFFFFu);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                out[c] = (j + c < d) ? ~(__float_as_uint(x[j + c]) & 0x7FFFFFFFu) : 0xFFFFFFFFu;
        }
    }
    __device__ __forceinline__ uint32_t key_at(const Tile&, uint64_t base, int lane, int k,
                                               int c) const {
        return ~(__float_as_uint(x[base + (uint64_t)(k * 128 + lane * 4 + c)]) & 0x7FFFFFFFu);
    }
};

// in-tile position of key c of load k
template <class Src>
__device__ __forceinline__ int key_pos(int lane, int k, int c) {
    return Src::kCanonical ? lane * 32 + 4 * k + c : k * 128 + lane * 4 + c;
}

// bits 4k+c of a lane whose keys lie inside [0, d)
template <class Src>
__device__ __forceinline__ uint32_t valid_nibbles(uint64_t base, int lane, uint64_t d) {
    if (base + kTile <= d) return 0xFFFFFFFFu;
    uint32_t v = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (base + (uint64_t)key_pos<Src>(lane, k, c) < d) v |= 1u << (4 * k + c);
    }
    return v;
}

// per-key bits of a lane -> word `lane` of the tile mask
template <class Src>
__device__ __forceinline__ uint32_t mask_word(uint32_t nib, int lane) {
    return Src::kCanonical ? nib : canonical_mask_word(nib, lane);
}

__global__ void select_init_kernel(SelectWorkspace ws, const uint64_t q) {
    for (int i = threadIdx.x; i < (kSelPasses + 3) * kSelBins; i += blockDim.x) ws.hist[i] = 0u;
    if (threadIdx.x == 0) {
        ws.state->prefix = 0u;
        ws.state->mode = 0u;
        ws.state->remaining = q;
        *ws.count = 0u;
        *ws.cand_count = 0u;
    }
}

// persistent blocks: block b takes the groups of 8 tiles b, b + gridDim.x, ...
// With a guess g of the first digit of the q-th key (stream keys are uniform, so g = q * 2048 / d
// is right to within one bin), pass 0 also counts the second digit of the keys whose first digit
// is g - 1, g or g + 1: the choose kernel can then fix 22 key bits at once and the candidate list
// shrinks from d / 2^11 to d / 2^22 keys.  A wrong guess only loses that shortcut.
template <class Src, int PASS, bool kGuess = false>
__global__ void __launch_bounds__(kBlockThreads)
select_hist_kernel(const Src src, const uint64_t d, const SelectWorkspace ws, const int guess = 0) {
    constexpr int bins = sel_bins(PASS);
    constexpr int shift = sel_shift(PASS);
    constexpr uint32_t fixed = sel_fixed(PASS);
    // candidates already collected: the remaining digits are found on the candidate list
    if (PASS > 0 && ws.state->mode != 0u) return;
    __shared__ uint32_t s_hist[bins];
    __shared__ uint32_t s_hist2[kGuess ? 3 * kSelBins : 1];
    for (int i = threadIdx.x; i < bins; i += kBlockThreads) s_hist[i] = 0u;
    if (kGuess)
        for (int i = threadIdx.x; i < 3 * kSelBins; i += kBlockThreads) s_hist2[i] = 0u;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const uint32_t prefix = PASS == 0 ? 0u : ws.state->prefix;
    const uint32_t guess_lo = kGuess ? (uint32_t)(guess - 1) << 21 : 0u;    // first key of bin g - 1
    const uint64_t groups = (sparse_tiles(d) + kWarpsPerBlock - 1) / kWarpsPerBlock;
    for (uint64_t g = blockIdx.x; g < groups; g += gridDim.x) {
        const uint64_t base = (g * kWarpsPerBlock + (threadIdx.x >> 5)) * kTile;
        if (base >= d) continue;
        const typename Src::Tile t = src.tile(base, lane);
        if (Src::kCanonical && base + kTile <= d) {
            // computed keys, full tile: no validity test (this variant is bound by instruction
            // issue; the loaded-key variant is bound by memory and keeps the smaller code)
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                uint32_t key[4];
                src.load(t, base, lane, k, d, key);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if ((key[c] & fixed) == prefix)
                        atomicAdd(&s_hist[(key[c] >> shift) & (uint32_t)(bins - 1)], 1u);
                    if (kGuess && key[c] - guess_lo < (3u << 21))
                        atomicAdd(&s_hist2[(key[c] - guess_lo) >> 10], 1u);
                }
            }
            continue;
        }
        const uint32_t valid = valid_nibbles<Src>(base, lane, d);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t key[4];
            src.load(t, base, lane, k, d, key);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if ((key[c] & fixed) == prefix && ((valid >> (4 * k + c)) & 1u)) {
                    atomicAdd(&s_hist[(key[c] >> shift) & (uint32_t)(bins - 1)], 1u);
                    if (kGuess && key[c] - guess_lo < (3u << 21))
                        atomicAdd(&s_hist2[(key[c] - guess_lo) >> 10], 1u);
                }
            }
        }
    }
    __syncthreads();
    uint32_t* __restrict__ hist = ws.hist + PASS * kSelBins;
    for (int i = threadIdx.x; i < bins; i += kBlockThreads) {
        const uint32_t v = s_hist[i];
        if (v) atomicAdd(&hist[i], v);
    }
    if (kGuess) {
        for (int i = threadIdx.x; i < 3 * kSelBins; i += kBlockThreads) {
            const uint32_t v = s_hist2[i];
            if (v) atomicAdd(&ws.hist2[i], v);
        }
    }
}

// one block of 1024 threads, two bins each: the bin in which the cumulative count reaches
// `remaining` becomes the next digit.  If few enough keys share the digits fixed so far (passes 0
// and 1), the remaining passes over all d keys are skipped: the mark kernel collects those keys
// and the candidate kernel finishes the selection on the list.
template <int PASS>
__global__ void __launch_bounds__(kScanThreads)
select_choose_kernel(const SelectWorkspace ws, const int guess = -1) {
    constexpr int bins = sel_bins(PASS);
    if (PASS > 0 && ws.state->mode != 0u) return;
    const uint32_t* __restrict__ hist = ws.hist + PASS * kSelBins;
    __shared__ uint64_t s_sum[kScanThreads];
    __shared__ int s_pick;
    const int t = threadIdx.x;
    uint32_t h0 = (2 * t < bins) ? hist[2 * t] : 0u;
    uint32_t h1 = (2 * t + 1 < bins) ? hist[2 * t + 1] : 0u;
    if (t == 0) s_pick = -1;
    s_sum[t] = (uint64_t)h0 + h1;
    __syncthreads();
    for (int o = 1; o < kScanThreads; o <<= 1) {
        const uint64_t v = (t >= o) ? s_sum[t - o] : 0ull;
        __syncthreads();
        s_sum[t] += v;
        __syncthreads();
    }
    uint64_t remaining = ws.state->remaining;
    uint64_t before = s_sum[t] - h0 - h1;               // keys in lower bins
    __syncthreads();                                    // everyone has read the state
    int pick = -1;
    if (remaining > before && remaining <= before + h0) pick = 0;
    else if (remaining > before + h0 && remaining <= before + h0 + h1) pick = 1;
    if (pick >= 0) {
        ws.state->prefix |= (uint32_t)(2 * t + pick) << sel_shift(PASS);
        ws.state->remaining = remaining - before - (pick ? h0 : 0u);
        if (PASS < 2 && (pick ? h1 : h0) <= kCandCap) ws.state->mode = (uint32_t)(PASS + 1);
        s_pick = 2 * t + pick;
    }
    if (PASS != 0 || guess < 0) return;
    // second digit from the guessed rows, if the first digit is one of the three guessed bins
    __syncthreads();
    const int row = s_pick - (guess - 1);
    if (s_pick < 0 || row < 0 || row > 2) return;
    const uint32_t* __restrict__ hist2 = ws.hist2 + row * kSelBins;
    h0 = hist2[2 * t];
    h1 = hist2[2 * t + 1];
    s_sum[t] = (uint64_t)h0 + h1;
    __syncthreads();
    for (int o = 1; o < kScanThreads; o <<= 1) {
        const uint64_t v = (t >= o) ? s_sum[t - o] : 0ull;
        __syncthreads();
        s_sum[t] += v;
        __syncthreads();
    }
    remaining = ws.state->remaining;                    // what is left inside the first bin
    before = s_sum[t] - h0 - h1;
    __syncthreads();
    pick = -1;
    if (remaining > before && remaining <= before + h0) pick = 0;
    else if (remaining > before + h0 && remaining <= before + h0 + h1) pick = 1;
    if (pick >= 0 && (pick ? h1 : h0) <= kCandCap) {
        ws.state->prefix |= (uint32_t)(2 * t + pick) << sel_shift(1);
        ws.state->remaining = remaining - before - (pick ? h0 : 0u);
        ws.state->mode = 2u;                            // candidates share 22 fixed bits
    }
}

// grid: ceil(tiles / warps per block); one tile per warp.  With sh = 0 (all digits fixed) the
// masks are "key < T" and "key == T"; with candidates (sh = 21 or 10 undecided low bits) they are
// "fixed digits below the prefix" and, instead of a tie mask, the keys whose fixed digits equal
// the prefix go to the candidate list: one reservation on the global counter per block, the
// (rare) candidate keys recomputed one by one.
template <class Src>
__global__ void __launch_bounds__(kBlockThreads)
select_mark_kernel(const Src src, const uint64_t d, uint32_t* __restrict__ less_mask,
                   const SelectWorkspace ws) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + warp;
    const uint64_t base = tile * kTile;
    const bool active = base < d;
    const uint32_t mode = ws.state->mode;
    const int sh = mode == 0u ? 0 : mode == 1u ? 21 : 10;
    const uint32_t T = ws.state->prefix >> sh;
    __shared__ uint32_t s_eq[kWarpsPerBlock];
    __shared__ uint32_t s_base;
    // "fixed digits >= T" is "key >= T << sh", "fixed digits > T" is "key >= (T + 1) << sh"; both
    // comparisons are the carry of key + (2^32 - bound), shifted straight into a bit register
    // (two integer instructions each).  T << sh = 0 never carries and means "always"; a second
    // bound of 2^32 gives the addend 0, which never carries, as it should.
    const uint32_t lo_bound = T << sh;
    const uint32_t neg_lo = 0u - lo_bound;
    const uint32_t neg_hi = (uint32_t)(0ull - (((unsigned long long)T + 1ull) << sh));
    uint32_t less = 0, equal = 0;
    typename Src::Tile t;
    if (active) {
        t = src.tile(base, lane);
        const uint32_t valid = valid_nibbles<Src>(base, lane, d);
        if (Src::kCanonical) {
            // computed keys: the pass is bound by instruction issue, the carry form is shorter
            uint32_t ge_lo = 0, ge_hi = 0;
#pragma unroll
            for (int k = 7; k >= 0; --k) {
                uint32_t key[4];
                src.load(t, base, lane, k, d, key);
#pragma unroll
                for (int c = 3; c >= 0; --c) {
                    shift_in_drop_bit(ge_lo, key[c], neg_lo);
                    shift_in_drop_bit(ge_hi, key[c], neg_hi);
                }
            }
            if (lo_bound == 0u) ge_lo = 0xFFFFFFFFu;
            less = ~ge_lo & valid;
            equal = ge_lo & ~ge_hi & valid;
        } else {
            // loaded keys: the pass is bound by memory; plain comparisons, loads in ascending order
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                uint32_t key[4];
                src.load(t, base, lane, k, d, key);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t hi = key[c] >> sh;
                    less |= (hi < T ? 1u : 0u) << (4 * k + c);
                    equal |= (hi == T ? 1u : 0u) << (4 * k + c);
                }
            }
            less &= valid;
            equal &= valid;
        }
    }
    const uint32_t lw = mask_word<Src>(less, lane);
    const uint32_t ew = (mode == 0u) ? mask_word<Src>(equal, lane) : 0u;
    if (active) {
        less_mask[tile * 32 + lane] = lw;
        ws.eqmask[tile * 32 + lane] = ew;
    }
    // ties (mode 0) or candidates (modes 1, 2) of this lane, then of the warps before it
    const uint32_t mine = __popc(equal);
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_eq[warp] = incl;
    __syncthreads();
    uint32_t block_total = 0, before = incl - mine;
    for (int w = 0; w < kWarpsPerBlock; ++w) {
        if (w < warp) before += s_eq[w];
        block_total += s_eq[w];
    }
    if (mode == 0u) {
        if (threadIdx.x == 0) ws.eq_block[blockIdx.x] = block_total;
        return;
    }
    if (threadIdx.x == 0) {
        ws.eq_block[blockIdx.x] = 0u;
        s_base = block_total ? atomicAdd(ws.cand_count, block_total) : 0u;
    }
    __syncthreads();
    uint32_t at = s_base + before;
    while (equal) {
        const int bit = __ffs(equal) - 1;
        equal &= equal - 1;
        if (at < kCandCap)
            ws.cand[at] = make_uint2(src.key_at(t, base, lane, bit >> 2, bit & 3),
                                     (uint32_t)(base + (uint64_t)key_pos<Src>(lane, bit >> 2, bit & 3)));
        ++at;
    }
}

// One block.  Finishes the selection on the candidate list: the `remaining` smallest pairs
// (key, coordinate) among the candidates are selected, digit by digit over the undecided key bits
// and then, only while equal keys remain undecided, over the coordinate bits; stops as soon as a
// digit bin is taken whole.  Selected coordinates are set in the mask.
__global__ void __launch_bounds__(kScanThreads)
select_candidates_kernel(uint32_t* __restrict__ mask, const SelectWorkspace ws) {
    const uint32_t mode = ws.state->mode;
    if (mode == 0u) return;
    __shared__ uint32_t s_hist[kSelBins];
    __shared__ uint32_t s_scan[kScanThreads];
    __shared__ unsigned long long s_prefix;
    __shared__ uint32_t s_remaining, s_done;
    const int t = threadIdx.x;
    const uint32_t n = min(*ws.cand_count, kCandCap);
    const uint2* __restrict__ cand = ws.cand;
    if (t == 0) {
        s_prefix = (unsigned long long)ws.state->prefix << 32;
        s_remaining = (uint32_t)ws.state->remaining;
        s_done = 0u;
    }
    __syncthreads();
    // digit positions in the 64-bit pair (key << 32 | coordinate): shift, width
    const int shifts[5] = {42, 32, 21, 10, 0};
    const int widths[5] = {11, 10, 11, 11, 10};
    int final_shift = 0;
    for (int pass = (mode == 1u ? 0 : 1); pass < 5; ++pass) {
        const int shift = shifts[pass];
        const int bins = 1 << widths[pass];
        for (int i = t; i < kSelBins; i += kScanThreads) s_hist[i] = 0u;
        __syncthreads();
        const unsigned long long prefix = s_prefix;
        const int above = shift + widths[pass];
        for (uint32_t i0 = t; i0 < n; i0 += 8 * kScanThreads) {      // 8 loads in flight
            uint2 e[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t i = i0 + u * kScanThreads;
                e[u] = (i < n) ? cand[i] : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned long long v = ((unsigned long long)e[u].x << 32) | e[u].y;
                if (i0 + u * kScanThreads < n && (v >> above) == (prefix >> above))
                    atomicAdd(&s_hist[(uint32_t)(v >> shift) & (uint32_t)(bins - 1)], 1u);
            }
        }
        __syncthreads();
        const uint32_t h0 = (2 * t < bins) ? s_hist[2 * t] : 0u;
        const uint32_t h1 = (2 * t + 1 < bins) ? s_hist[2 * t + 1] : 0u;
        s_scan[t] = h0 + h1;
        __syncthreads();
        for (int o = 1; o < kScanThreads; o <<= 1) {
            const uint32_t v = (t >= o) ? s_scan[t - o] : 0u;
            __syncthreads();
            s_scan[t] += v;
            __syncthreads();
        }
        const uint32_t remaining = s_remaining;
        const uint32_t before = s_scan[t] - h0 - h1;
        __syncthreads();
        int pick = -1;
        if (remaining > before && remaining <= before + h0) pick = 0;
        else if (remaining > before + h0 && remaining <= before + h0 + h1) pick = 1;
        if (pick >= 0) {
            const uint32_t lower = before + (pick ? h0 : 0u);
            s_prefix = prefix | ((unsigned long long)(2 * t + pick) << shift);
            s_remaining = remaining - lower;
            if ((pick ? h1 : h0) == remaining - lower) s_done = 1u;      // the bin is taken whole
        }
        __syncthreads();
        final_shift = shift;
        if (s_done) break;
    }
    // pairs are distinct, so the loop ends with s_done set at the latest after the last pass
    const unsigned long long limit = s_prefix >> final_shift;
    const unsigned long long fixed_hi = s_prefix >> (mode == 1u ? 53 : 42);
    for (uint32_t i0 = t; i0 < n; i0 += 8 * kScanThreads) {
        uint2 e[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t i = i0 + u * kScanThreads;
            e[u] = (i < n) ? cand[i] : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const unsigned long long v = ((unsigned long long)e[u].x << 32) | e[u].y;
            if (i0 + u * kScanThreads < n && (v >> (mode == 1u ? 53 : 42)) == fixed_hi &&
                (v >> final_shift) <= limit)
                atomicOr(&mask[e[u].y >> 5], 1u << (e[u].y & 31u));
        }
    }
}

// one block: in-place exclusive scan of n counts; the total goes to *total if it is not null
__global__ void __launch_bounds__(kScanThreads)
select_scan_counts_kernel(uint32_t* __restrict__ counts, const uint64_t n,
                          uint32_t* __restrict__ total, const SelectState* skip_unless_mode0) {
    // the tie counts are only needed when all three digit passes ran
    if (skip_unless_mode0 && skip_unless_mode0->mode != 0u) return;
    const uint32_t sum = block_exclusive_scan_inplace(counts, n);
    if (threadIdx.x == 0 && total) *total = sum;
}

// grid: ceil(tiles / warps per block).  Only when all three digit passes ran (mode 0): mask <-
// "< T" | the first r of "== T" in index order.  In the candidate modes the candidate kernel has
// already set the selected candidates in the mask and there is nothing to do.
__global__ void __launch_bounds__(kBlockThreads)
select_resolve_kernel(const uint64_t d, const SparseWorkspace sp, const SelectWorkspace ws) {
    if (ws.state->mode != 0u) return;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    __shared__ uint32_t s_eq[kWarpsPerBlock];
    const uint64_t r = ws.state->remaining;
    const uint64_t groups = (sparse_tiles(d) + kWarpsPerBlock - 1) / kWarpsPerBlock;
    for (uint64_t g = blockIdx.x; g < groups; g += gridDim.x) {      // a few blocks: the usual
        const uint64_t tile = g * kWarpsPerBlock + warp;             // early exit costs nothing
        const uint64_t base = tile * kTile;
        const bool active = base < d;
        uint32_t word = active ? sp.bitmask[tile * 32 + lane] : 0u;
        uint32_t ew = active ? ws.eqmask[tile * 32 + lane] : 0u;
        const uint32_t ne = __popc(ew);
        uint32_t incl = ne;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        __syncthreads();                                             // s_eq of the last round is read
        if (lane == 31) s_eq[warp] = incl;
        __syncthreads();
        uint64_t rank0 = (uint64_t)ws.eq_block[g] + (incl - ne);     // rank of this lane's first
        for (int w = 0; w < warp; ++w) rank0 += s_eq[w];
        const uint32_t allowed = (r > rank0) ? (uint32_t)min((uint64_t)ne, r - rank0) : 0u;
        uint32_t left = ne;
        while (left > allowed) {             // drop the highest-index ties beyond the first r
            ew &= ~(0x80000000u >> __clz(ew));
            --left;
        }
        word |= ew;
        if (active) sp.bitmask[tile * 32 + lane] = word;
    }
}

// grid: ceil(tile groups / warps per block); one warp per group of 8 tiles.  Per-group kept count
// of the final mask and, with kNorm, the norm partial of the scaled kept entries (P as in the
// sparsifier): what the compaction kernels shared with the sparsifier expect from a select pass.
template <int P, bool kNorm>
__global__ void __launch_bounds__(kBlockThreads)
select_group_partial_kernel(const float* __restrict__ x, const uint64_t d, const float scale,
                            const SparseWorkspace sp) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint64_t tiles = sparse_tiles(d);
    const uint64_t groups = (tiles + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const uint64_t grp = (uint64_t)blockIdx.x * kWarpsPerBlock + warp;
    if (grp >= groups) return;
    const uint64_t tile0 = grp * kWarpsPerBlock;
    const uint64_t gbase = tile0 * kTile;
    __shared__ uint16_t s_list[kNorm ? kWarpsPerBlock : 1][kNorm ? kGroupListCap : 1];
    uint32_t word[kWarpsPerBlock];
#pragma unroll
    for (int w = 0; w < kWarpsPerBlock; ++w)
        word[w] = (tile0 + w < tiles) ? sp.bitmask[(tile0 + w) * 32 + lane] : 0u;
    uint32_t kept = 0;
    double dsum = 0.0;
    uint32_t vmax = 0;
    if (kNorm) {
        uint16_t* list = s_list[warp];
        auto take = [&](float xv) {
            const float xs = __fmul_rn(scale, xv);
            const uint32_t a = __float_as_uint(xs) & 0x7FFFFFFFu;
            if (P == NC_P_INF) vmax = max(vmax, a);
            else if (P == 1) dsum += (double)__uint_as_float(a);
            else dsum = fma((double)xs, (double)xs, dsum);
        };
        auto flush = [&](uint32_t cnt) {
            __syncwarp();
            if (cnt <= 4u * 32u) {
                float xv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t t = (uint32_t)(e * 32 + lane);
                    xv[e] = (t < cnt) ? x[gbase + list[t]] : 0.f;   // +0 adds nothing to any norm
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) take(xv[e]);
            } else {
                for (uint32_t t = lane; t < cnt; t += 32) take(x[gbase + list[t]]);
            }
            __syncwarp();
        };
        uint32_t cnt = 0;
#pragma unroll
        for (int w = 0; w < kWarpsPerBlock; ++w) {
            const uint32_t tile_cnt = warp_sum_u(__popc(word[w]));
            if (cnt + tile_cnt > kGroupListCap) {
                flush(cnt);
                cnt = 0;
            }
            group_list_append(word[w], lane, w, list, cnt);
            cnt += tile_cnt;
            kept += tile_cnt;
        }
        flush(cnt);
    } else {
#pragma unroll
        for (int w = 0; w < kWarpsPerBlock; ++w) kept += __popc(word[w]);
        kept = warp_sum_u(kept);
    }
    uint64_t part = 0;
    if (kNorm) {
        if (P == NC_P_INF) part = (uint64_t)warp_max_u(vmax);
        else part = (uint64_t)__double_as_longlong(warp_sum_d(dsum));
    }
    if (lane == 0) {
        sp.block_count[grp] = kept;
        if (kNorm) sp.block_partial[grp] = part;
    }
}

// grid: ceil(tiles / warps per block).  Lists the selected entries in index order: index, the
// exponent byte of C_nat(x_j) (Def. 1; stream of coordinate j) and one sign byte for the packer.
__global__ void __launch_bounds__(kBlockThreads)
topk_emit_kernel(const float* __restrict__ x, const uint64_t d, const uint32_t worker,
                 const __grid_constant__ PhiloxKeys keys, const uint64_t cap,
                 uint32_t* __restrict__ idx, uint8_t* __restrict__ exp, const SparseWorkspace sp) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint64_t tile = (uint64_t)blockIdx.x * kWarpsPerBlock + warp;
    const uint64_t base = tile * kTile;
    const bool active = base < d;
    __shared__ uint32_t s_tile[kWarpsPerBlock];
    __shared__ uint16_t s_list[kWarpsPerBlock][kTile];
    uint16_t* list = s_list[warp];
    const uint32_t word = active ? sp.bitmask[tile * 32 + lane] : 0u;
    const uint32_t cnt = warp_list_positions(word, lane, list);
    if (lane == 0) s_tile[warp] = cnt;
    __syncthreads();
    uint64_t k0 = (uint64_t)sp.block_count[blockIdx.x];
    for (int w = 0; w < warp; ++w) k0 += s_tile[w];
    for (uint32_t t = lane; t < cnt; t += 32) {
        const uint64_t k = k0 + t;
        if (k >= cap) break;
        const uint64_t j = base + list[t];
        const uint32_t bits = __float_as_uint(x[j]);
        const uint32_t r23 = stream_word_at(j, worker, kDomainCnat, keys) & 0x7FFFFFu;
        const uint32_t e = (bits >> 23) & 0xFFu;
        const uint32_t m = bits & 0x7FFFFFu;
        // up with probability m / 2^23; 2^127 and above saturate, inf and NaN give byte 255
        const uint32_t byte = (e >= 254u) ? e : e + (r23 < m ? 1u : 0u);
        idx[k] = (uint32_t)j;
        exp[k] = (uint8_t)byte;
        sp.tmp_codes[k] = (uint8_t)(bits >> 31);
    }
}

// one warp per 32 listed entries: sign bytes -> one word of the sign plane
__global__ void __launch_bounds__(kBlockThreads)
topk_pack_sign_kernel(const uint8_t* __restrict__ sign_bytes, const uint64_t listed,
                      uint32_t* __restrict__ sign) {
    const int lane = threadIdx.x & 31;
    const uint64_t group = (uint64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (group * 32 >= listed) return;
    const uint64_t k = group * 32 + lane;
    const uint32_t b = (k < listed) ? sign_bytes[k] : 0u;
    const uint32_t wv = __ballot_sync(0xFFFFFFFFu, b & 1u);
    if (lane == 0) sign[group] = wv;
}

// grid: ceil(count / threads)
__global__ void __launch_bounds__(kBlockThreads)
topk_decode_accumulate_kernel(const uint32_t* __restrict__ idx, const uint8_t* __restrict__ exp,
                              const uint32_t* __restrict__ sign, const uint64_t count,
                              const uint64_t d, float* __restrict__ acc) {
    const uint64_t k = (uint64_t)blockIdx.x * kBlockThreads + threadIdx.x;
    if (k >= count) return;
    const uint32_t j = idx[k];
    if (j >= d) return;
    const uint32_t bits = ((uint32_t)exp[k] << 23) | (((sign[k >> 5] >> (k & 31)) & 1u) << 31);
    acc[j] = __fadd_rn(acc[j], __uint_as_float(bits));
}

// zero count, norm and planes: the q = 0 sparsifier
__global__ void __launch_bounds__(kBlockThreads)
select_empty_kernel(uint32_t* __restrict__ planes, const uint64_t words,
                    uint32_t* __restrict__ count, float* __restrict__ norm) {
    const uint64_t i = (uint64_t)blockIdx.x * kBlockThreads + threadIdx.x;
    if (i < words) planes[i] = 0u;
    if (i == 0) {
        *count = 0u;
        *norm = 0.f;
    }
}

// hist/choose passes, mark, scan of the tie counts: leaves T and r in the state, "< T" in the
// sparsifier bitmask and "== T" in the tie mask
template <class Src>
static void run_select(const Src& src, uint64_t d, uint64_t q, const SparseWorkspace& sp,
                       const SelectWorkspace& ws, int sm_count, cudaStream_t stream,
                       int guess = -1) {
    const uint64_t groups = (sparse_tiles(d) + kWarpsPerBlock - 1) / kWarpsPerBlock;
    // persistent grid: exactly the blocks that are resident together (a partial second wave would
    // run at the end with most SMs idle)
    static int per_sm[64] = {0};
    int dev = 0;
    int resident = 4;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        if (per_sm[dev] == 0) {
            int v = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, select_hist_kernel<Src, 0>,
                                                              kBlockThreads, 0) != cudaSuccess ||
                v < 1)
                v = 4;
            per_sm[dev] = v;
        }
        resident = per_sm[dev];
    }
    const uint64_t cap_blocks = (uint64_t)sm_count * (uint64_t)resident;
    const unsigned pgrid = (unsigned)(groups < cap_blocks ? groups : cap_blocks);
    select_init_kernel<<<1, kScanThreads, 0, stream>>>(ws, q);
    if (guess >= 0)
        select_hist_kernel<Src, 0, true><<<pgrid, kBlockThreads, 0, stream>>>(src, d, ws, guess);
    else
        select_hist_kernel<Src, 0><<<pgrid, kBlockThreads, 0, stream>>>(src, d, ws);
    select_choose_kernel<0><<<1, kScanThreads, 0, stream>>>(ws, guess);
    select_hist_kernel<Src, 1><<<pgrid, kBlockThreads, 0, stream>>>(src, d, ws);
    select_choose_kernel<1><<<1, kScanThreads, 0, stream>>>(ws);
    select_hist_kernel<Src, 2><<<pgrid, kBlockThreads, 0, stream>>>(src, d, ws);
    select_choose_kernel<2><<<1, kScanThreads, 0, stream>>>(ws);
    select_mark_kernel<Src><<<(unsigned)groups, kBlockThreads, 0, stream>>>(src, d, sp.bitmask, ws);
    select_candidates_kernel<<<1, kScanThreads, 0, stream>>>(sp.bitmask, ws);
    select_scan_counts_kernel<<<1, kScanThreads, 0, stream>>>(ws.eq_block, groups, nullptr,
                                                              ws.state);
}

static int sm_count_of_current_device() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1)
            v = 148;
        cached[dev] = v;
    }
    return cached[dev];
}

}  // namespace natcomp

using namespace natcomp;

extern "C" {

size_t nc_select_workspace_bytes(size_t d, size_t cap) {
    return sparse_ws_bytes(d, cap) + select_extra_bytes(d);
}

nc_status nd_sparse_exact_compress(const float* x, size_t d, uint64_t q, float scale, int p, int s,
                                   uint64_t seed, uint32_t worker, uint32_t* idx,
                                   uint32_t* planes, uint32_t* count, float* norm, size_t cap,
                                   void* workspace, size_t workspace_bytes, cudaStream_t stream) {
    if (!x || !idx || !planes || !count || !norm || s < 1 || s > 8 || cap < 1)
        return NC_ERR_INVALID;
    if (p != 1 && p != 2 && p != NC_P_INF) return NC_ERR_UNSUPPORTED;
    if (d == 0) return NC_OK;
    if (d > 0xFFFFFFFFull) return NC_ERR_INVALID;
    if (!workspace) return NC_ERR_INVALID;
    if (!aligned16(workspace)) return NC_ERR_ALIGN;
    if (!aligned32(x) || !aligned16(idx) || !aligned16(planes) || !aligned4(count) ||
        !aligned4(norm))
        return NC_ERR_ALIGN;
    if (workspace_bytes < nc_select_workspace_bytes(d, cap)) return NC_ERR_WORKSPACE;
    if (q > d) q = d;
    if (q == 0) {
        const uint64_t words = ((cap + 31) / 32) * (uint64_t)(code_value_bits(s) + 1);
        select_empty_kernel<<<(unsigned)((words + kBlockThreads - 1) / kBlockThreads),
                              kBlockThreads, 0, stream>>>(planes, words, count, norm);
        return launch_status();
    }
    char* wsp = reinterpret_cast<char*>(workspace);
    const SparseWorkspace sp = sparse_ws_carve(wsp, d);
    const SelectWorkspace ws = select_ws_carve(wsp + sparse_ws_bytes(d, cap), d);
    const PhiloxKeys keys = make_philox_keys(seed);
    StreamKeys src;
    src.worker = worker;
    src.keys = keys;
    // stream keys are uniform: the q-th smallest lies in first-digit bin q * 2048 / d, give or take one
    int guess = (int)((unsigned __int128)q * 2048u / d);
    guess = guess < 1 ? 1 : (guess > 2046 ? 2046 : guess);
    run_select(src, d, q, sp, ws, sm_count_of_current_device(), stream, guess);
    const unsigned grid = (unsigned)((sparse_tiles(d) + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const uint64_t tile_groups = (sparse_tiles(d) + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const unsigned ggrid = (unsigned)((tile_groups + kWarpsPerBlock - 1) / kWarpsPerBlock);
    select_resolve_kernel<<<min(grid, 4u * (unsigned)sm_count_of_current_device()), kBlockThreads, 0,
                            stream>>>(d, sp, ws);
    if (p == 1)
        select_group_partial_kernel<1, true><<<ggrid, kBlockThreads, 0, stream>>>(x, d, scale, sp);
    else if (p == 2)
        select_group_partial_kernel<2, true><<<ggrid, kBlockThreads, 0, stream>>>(x, d, scale, sp);
    else
        select_group_partial_kernel<NC_P_INF, true><<<ggrid, kBlockThreads, 0, stream>>>(x, d,
                                                                                        scale, sp);
    SparseBatch batch;
    batch.x[0] = x;
    batch.idx[0] = idx;
    batch.codes[0] = reinterpret_cast<uint8_t*>(planes);
    batch.count[0] = count;
    batch.norm[0] = norm;
    batch.worker[0] = worker;
    sparse_compact_finish(batch, d, scale, p, s, keys, cap, wsp, sparse_ws_bytes(d, cap), 1,
                          stream);
    return launch_status();
}

nc_status nc_topk_compress(const float* x, size_t d, uint64_t K, uint64_t seed, uint32_t worker,
                           uint32_t* idx, uint8_t* exp, uint32_t* sign, void* workspace,
                           size_t workspace_bytes, cudaStream_t stream) {
    if (!x || !idx || !exp || !sign) return NC_ERR_INVALID;
    if (d > 0xFFFFFFFFull) return NC_ERR_INVALID;
    if (K > d) K = d;
    if (d == 0 || K == 0) return NC_OK;
    if (!workspace) return NC_ERR_INVALID;
    if (!aligned16(workspace)) return NC_ERR_ALIGN;
    if (!aligned32(x) || !aligned16(idx) || !aligned16(exp) || !aligned16(sign))
        return NC_ERR_ALIGN;
    if (workspace_bytes < nc_select_workspace_bytes(d, K)) return NC_ERR_WORKSPACE;
    char* wsp = reinterpret_cast<char*>(workspace);
    const SparseWorkspace sp = sparse_ws_carve(wsp, d);
    const SelectWorkspace ws = select_ws_carve(wsp + sparse_ws_bytes(d, K), d);
    MagnitudeKeys src;
    src.x = x;
    run_select(src, d, K, sp, ws, sm_count_of_current_device(), stream);
    const uint64_t groups = (sparse_tiles(d) + kWarpsPerBlock - 1) / kWarpsPerBlock;
    select_resolve_kernel<<<(unsigned)min(groups, (uint64_t)(4 * sm_count_of_current_device())),
                            kBlockThreads, 0, stream>>>(d, sp, ws);
    select_group_partial_kernel<NC_P_INF, false>
        <<<(unsigned)((groups + kWarpsPerBlock - 1) / kWarpsPerBlock), kBlockThreads, 0, stream>>>(
            x, d, 1.0f, sp);
    select_scan_counts_kernel<<<1, kScanThreads, 0, stream>>>(sp.block_count, groups, ws.count,
                                                              nullptr);
    topk_emit_kernel<<<(unsigned)groups, kBlockThreads, 0, stream>>>(
        x, d, worker, make_philox_keys(seed), K, idx, exp, sp);
    const uint64_t sgroups = (K + 31) / 32;
    topk_pack_sign_kernel<<<(unsigned)((sgroups + kWarpsPerBlock - 1) / kWarpsPerBlock),
                            kBlockThreads, 0, stream>>>(sp.tmp_codes, K, sign);
    return launch_status();
}

nc_status nc_topk_decode_accumulate(const uint32_t* idx, const uint8_t* exp, const uint32_t* sign,
                                    size_t count, size_t d, float* acc, cudaStream_t stream) {
    if (!idx || !exp || !sign || !acc) return NC_ERR_INVALID;
    if (d > 0xFFFFFFFFull || count > 0xFFFFFFFFull) return NC_ERR_INVALID;
    if (count == 0 || d == 0) return NC_OK;
    if (!aligned16(idx) || !aligned16(exp) || !aligned16(sign) || !aligned32(acc))
        return NC_ERR_ALIGN;
    const unsigned grid = (unsigned)((count + kBlockThreads - 1) / kBlockThreads);
    topk_decode_accumulate_kernel<<<grid, kBlockThreads, 0, stream>>>(idx, exp, sign, count, d,
                                                                      acc);
    return launch_status();
}

}  // extern "C"

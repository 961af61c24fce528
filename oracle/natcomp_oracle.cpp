// CPU oracle for the natural-compression hot path.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, scalar restatement of what the operators compute, written from
// the paper's definitions (arXiv 1905.10988).  It exists so that the CUDA library
// can be checked against something that is obviously the definition; it is never
// part of the product path, shares no code with the CUDA sources, and nothing in
// the package imports it.  Floating point is done in double unless a step is
// pinned to binary32 (the decoded values, the fixed-order fp32 sum, and the
// "given-norm" dithering mode).  Build: g++ -O2 -ffp-contract=off (no fast-math,
// no flush-to-zero), optional OpenMP over independent elements.
//
// Every function below is pinned by tests/test_oracle_*.py against values the
// paper prints, closed forms, exhaustive enumeration of the 2^23 random
// thresholds, or library routines (numpy); there is no "parity unpinned" function.
//
// Random numbers.  The paper only says that the rounding is randomised; this
// library fixes the random stream as Philox4x32-10 (Salmon, Moraes, Dror, Shaw,
// "Parallel random numbers: as easy as 1, 2, 3", SC'11):
//   key     = (low 32 bits of seed, high 32 bits of seed)
//   counter = (low 32 bits of q, high 32 bits of q, worker, domain),  q = j / 4
//   element j of a worker's vector uses output word (j mod 4), and of that word
//   the low 23 bits r23.
// domain: 0 = natural compression, 1 = natural-dithering rounding, 2 = sparsifier.
//
// Edge policy for binary32 inputs the paper does not discuss (Sec. 2 assumes a
// normal number with an implicit leading one):
//   +-0            -> +-0 (sign kept), Def. 1 "C_nat(0) = 0"
//   subnormal t    -> +-0 or +-2^-126, up-probability |t| / 2^-126 (unbiased; the
//                     9/8 second-moment bound of Thm. 1 does not hold here)
//   2^127<|t|<inf  -> never rounded up: +-2^127 (saturation, biased)
//   +-inf, NaN     -> +-inf (exponent byte 255, sign bit kept)

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <cstddef>
#include <limits>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------- Philox4x32-10
// One round: two 32x32->64 multiplies; the high halves are mixed with the other
// two counter words and the round key, the low halves pass through (SC'11, Sec. 4).
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {            // Weyl key schedule between rounds
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        const uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(prod1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)prod1;
        const uint32_t n2 = (uint32_t)(prod0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)prod0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

uint32_t stream_word(uint64_t seed, uint32_t worker, uint32_t domain, uint64_t j) {
    const uint64_t q = j / 4;
    const uint32_t ctr[4] = {(uint32_t)(q & 0xFFFFFFFFu), (uint32_t)(q >> 32), worker, domain};
    const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return out[j % 4];
}

const double TWO23 = 8388608.0;

// ------------------------------------------------------- natural compression
// Def. 1: t != 0 is rounded to sign(t) 2^floor(log2|t|) with probability p(t) and
// to sign(t) 2^ceil(log2|t|) with probability 1 - p(t),
// p(t) = (2^ceil - |t|) / 2^floor.  The draw: "up" iff r23 < (1 - p(t)) * 2^23.
// For a binary32 t the product is the integer mantissa field (Sec. 2:
// p(t) = 1 - m), so the rule is exact, not an approximation.
double cnat_value(float t, uint32_t r23) {
    if (t == 0.0f) return (double)t;                                  // keeps -0
    if (std::isnan(t) || std::isinf(t))
        return std::copysign(std::numeric_limits<double>::infinity(), (double)t);
    const double a = std::fabs((double)t);
    double lo, hi;
    if (a < 0x1p-126) {               // subnormal: bracket [0, 2^-126]
        lo = 0.0;
        hi = 0x1p-126;
    } else {
        const int fl = std::ilogb(a);              // floor(log2 |t|)
        lo = std::ldexp(1.0, fl);
        hi = std::ldexp(1.0, fl + 1);
        if (fl >= 127) return std::copysign(lo, (double)t);           // saturate
    }
    const double p_floor = (hi - a) / (hi - lo);   // p(t) of Def. 1 (hi - lo = 2^floor)
    const double p_up = 1.0 - p_floor;
    const bool up = (double)r23 < p_up * TWO23;
    return std::copysign(up ? hi : lo, (double)t);
}

// The paper's "deterministic" control variant (experimental set-up appendix): t is rounded to
// the nearest power of two, no randomness (biased).  Nearest in absolute distance, the midpoint
// 1.5 * 2^floor going up; zeros, subnormals, overflow and non-finite inputs as for C_nat
// (a subnormal goes to 0 or 2^-126, whichever is nearer).
double nearest_pow2_value(float t) {
    if (t == 0.0f) return (double)t;
    if (std::isnan(t) || std::isinf(t))
        return std::copysign(std::numeric_limits<double>::infinity(), (double)t);
    const double a = std::fabs((double)t);
    double lo, hi;
    if (a < 0x1p-126) {
        lo = 0.0;
        hi = 0x1p-126;
    } else {
        const int fl = std::ilogb(a);
        lo = std::ldexp(1.0, fl);
        hi = std::ldexp(1.0, fl + 1);
        if (fl >= 127) return std::copysign(lo, (double)t);
    }
    const bool up = (a - lo) >= (hi - a);
    return std::copysign(up ? hi : lo, (double)t);
}

// 9-bit code of a value of the form +-0, +-2^k, +-inf: biased exponent + sign bit.
void cnat_code(double value, uint8_t* exp_byte, uint32_t* sign_bit) {
    *sign_bit = std::signbit(value) ? 1u : 0u;
    const double a = std::fabs(value);
    if (a == 0.0) *exp_byte = 0;
    else if (std::isinf(a)) *exp_byte = 255;
    else *exp_byte = (uint8_t)(std::ilogb(a) + 127);
}

float cnat_decode(uint8_t exp_byte, uint32_t sign_bit) {
    double a;
    if (exp_byte == 0) a = 0.0;
    else if (exp_byte == 255) a = std::numeric_limits<double>::infinity();
    else a = std::ldexp(1.0, (int)exp_byte - 127);
    return (float)(sign_bit ? -a : a);
}

// ------------------------------------------------------------------- norms
// ||x||_p of Def. 3 for p in {1, 2, inf (encoded 0)}; double accumulation in index
// order, rounded once to binary32.  A NaN entry makes every norm NaN.
float norm_p(const float* x, uint64_t len, int p) {
    double acc = 0.0;
    bool saw_nan = false;
    for (uint64_t i = 0; i < len; ++i) {
        const double a = std::fabs((double)x[i]);
        if (std::isnan(a)) saw_nan = true;
        if (p == 1) acc += a;
        else if (p == 2) acc += a * a;
        else if (a > acc) acc = a;
    }
    if (saw_nan) return std::numeric_limits<float>::quiet_NaN();
    if (p == 2) acc = std::sqrt(acc);
    return (float)acc;
}

bool norm_degenerate(float norm) {
    // x = 0 gives D(x) = 0 (Def. 3).  A norm that is not finite has no ratio |x| / norm to
    // round either: such a bucket gets level code 0 everywhere, and its norm is still stored,
    // which is how the receiver can tell.  A subnormal norm is an ordinary norm.
    return !(norm > 0.0f) || std::isinf(norm);
}

// y = |x| / norm of Def. 3 in the pinned binary32 arithmetic of the "given norm" mode: one
// reciprocal per bucket, one multiply per entry.  The reciprocal of a subnormal norm would
// overflow, so below 2^-126 both operands are first multiplied by 2^24; that scaling is exact
// (norm * 2^24 is a normal number and so is |x| * 2^24 for any |x| <= norm), hence y is the
// same ratio and E xi(y) = y keeps the operator unbiased for buckets of tiny entries.
float ratio_given_norm(float ax, float norm) {
    if (norm < 0x1p-126f) {
        ax = ax * 0x1p24f;
        norm = norm * 0x1p24f;
    }
    const float rinv = 1.0f / norm;
    return ax * rinv;
}

// ------------------------------------------------------- natural dithering
// Def. 3 with the natural levels l_u = 2^-u (u = 0..s-1), l_s = 0.  For
// l_{u+1} <= y <= l_u, xi(y) = l_u with probability (y - l_{u+1}) / (l_u - l_{u+1}).
// Returns the level code c in 0..s:  c = 0 <-> 0,  c = k <-> 2^(k-s).
// The draw: "up" iff r23 < floor(probability * 2^23).
int nd_level_code(double y, int s, uint32_t r23) {
    if (y >= 1.0) return s;                       // y = l_0 (or a rounding excess)
    // xi is defined on [0, 1] (Def. 3).  A ratio outside it can only come from a norm that is not
    // the norm of these entries (norms given by the caller): y > 1 takes the top level above, and
    // so does a ratio that is not a number (a NaN entry against a finite norm).
    if (std::isnan(y)) return s;
    for (int u = 0; u < s; ++u) {
        const double upper = std::ldexp(1.0, -u);
        const double lower = (u + 1 == s) ? 0.0 : std::ldexp(1.0, -(u + 1));
        if (y >= lower) {
            const double p_up = (y - lower) / (upper - lower);
            const double thr = std::floor(p_up * TWO23);
            const bool up = (double)r23 < thr;
            return up ? (s - u) : (s - u - 1);
        }
    }
    return 0;   // not reached for y >= 0
}

// Decoded value of level code c under norm (Def. 3: ||x|| * sign * xi with xi = 2^(c-s), and
// xi = 0 for c = 0): one binary32 multiply by an exact power of two.  c = 0 contributes a zero
// whatever the norm is; for c > 0 the product is taken as it comes, so a norm that is not
// finite gives a value that is not finite.
float nd_decode_value(int c, int s, float norm, uint32_t sign_bit) {
    float mag;
    if (c == 0) mag = 0.0f;
    else mag = norm * (float)std::ldexp(1.0, c - s);
    return sign_bit ? -mag : mag;
}

}  // namespace

extern "C" {

void orc_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

int orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}

// out[i] = the 32-bit stream word of element j0 + i
void orc_stream_words(uint64_t seed, uint32_t worker, uint32_t domain, uint64_t j0,
                      uint64_t count, uint32_t* out) {
    for (uint64_t i = 0; i < count; ++i) out[i] = stream_word(seed, worker, domain, j0 + i);
}

// Scalar C_nat with explicit random thresholds: out[i] = C_nat(t[i]; r23[i]).
void orc_cnat_values(const float* t, const uint32_t* r23, uint64_t count, double* out) {
    for (uint64_t i = 0; i < count; ++i) out[i] = cnat_value(t[i], r23[i] & 0x7FFFFFu);
}

// 9-bit codes with explicit random thresholds (exhaustive bit-pattern parity).
void orc_cnat_codes(const float* t, const uint32_t* r23, uint64_t count, uint8_t* exp_bytes,
                    uint8_t* sign_bits) {
    for (uint64_t i = 0; i < count; ++i) {
        uint32_t sb;
        cnat_code(cnat_value(t[i], r23[i] & 0x7FFFFFu), &exp_bytes[i], &sb);
        sign_bits[i] = (uint8_t)sb;
    }
}

void orc_cnat_decode(const uint8_t* exp_bytes, const uint8_t* sign_bits, uint64_t count, float* out) {
    for (uint64_t i = 0; i < count; ++i) out[i] = cnat_decode(exp_bytes[i], sign_bits[i]);
}

// Worker-side C_nat of x[0..d) whose first entry is element j0 of the worker's
// vector (j0 a multiple of 32).  exp: d bytes; sign: ceil(d/32) words, bit (j mod 32)
// of word (j / 32), unused high bits of the last word zero.
void orc_nc_compress(const float* x, uint64_t d, uint64_t j0, uint64_t seed, uint32_t worker,
                     uint8_t* exp, uint32_t* sign) {
    const int64_t words = (int64_t)((d + 31) / 32);
#pragma omp parallel for schedule(static)
    for (int64_t w = 0; w < words; ++w) {
        uint32_t bits = 0;
        const uint64_t end = ((uint64_t)w * 32 + 32 < d) ? (uint64_t)w * 32 + 32 : d;
        for (uint64_t i = (uint64_t)w * 32; i < end; ++i) {
            const uint32_t r23 = stream_word(seed, worker, 0u, j0 + i) & 0x7FFFFFu;
            uint32_t sb;
            cnat_code(cnat_value(x[i], r23), &exp[i], &sb);
            bits |= sb << (i % 32);
        }
        sign[w] = bits;
    }
}

// Deterministic variant of orc_nc_compress: codes of the nearest power of two.
void orc_nc_compress_nearest(const float* x, uint64_t d, uint8_t* exp, uint32_t* sign) {
    const int64_t words = (int64_t)((d + 31) / 32);
#pragma omp parallel for schedule(static)
    for (int64_t w = 0; w < words; ++w) {
        uint32_t bits = 0;
        const uint64_t end = ((uint64_t)w * 32 + 32 < d) ? (uint64_t)w * 32 + 32 : d;
        for (uint64_t i = (uint64_t)w * 32; i < end; ++i) {
            uint32_t sb;
            cnat_code(nearest_pow2_value(x[i]), &exp[i], &sb);
            bits |= sb << (i % 32);
        }
        sign[w] = bits;
    }
}

// Master side, one worker: acc[j] = acc[j] + decode(code_j) in binary32.
void orc_nc_decode_accumulate(const uint8_t* exp, const uint32_t* sign, uint64_t d, float* acc) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)d; ++i) {
        const float v = cnat_decode(exp[i], (sign[i / 32] >> (i % 32)) & 1u);
        acc[i] = acc[i] + v;
    }
}

// Master side (Algorithm 1, "aggregate"): out[j] = sum over workers i = 0..n-1 of
// decode(code_{i,j}), accumulated left to right in binary32 starting from +0.
void orc_nc_aggregate(const uint8_t* const* exp, const uint32_t* const* sign, int n, uint64_t d,
                      float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)d; ++j) {
        float acc = 0.0f;
        for (int i = 0; i < n; ++i) {
            const float v = cnat_decode(exp[i][j], (sign[i][j / 32] >> (j % 32)) & 1u);
            acc = acc + v;
        }
        out[j] = acc;
    }
}

// The uncompressed reference point: out[j] = ((+0 + x_0[j]) + x_1[j]) + ... in binary32.
void orc_sum_fp32(const float* const* xs, int n, uint64_t d, float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)d; ++j) {
        float acc = 0.0f;
        for (int i = 0; i < n; ++i) acc = acc + xs[i][j];
        out[j] = acc;
    }
}

// Per-bucket norms; bucket_off has B+1 entries relative to x, bucket b = [off[b], off[b+1]).
void orc_norms(const float* x, const uint64_t* bucket_off, int B, int p, float* norms) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        norms[b] = norm_p(x + bucket_off[b], bucket_off[b + 1] - bucket_off[b], p);
}

// Level codes for explicit y and thresholds (enumeration pins).
void orc_nd_level_codes(const double* y, const uint32_t* r23, uint64_t count, int s, int32_t* codes) {
    for (uint64_t i = 0; i < count; ++i) codes[i] = nd_level_code(y[i], s, r23[i] & 0x7FFFFFu);
}

// Standard dithering D_sta^{p,u} (Def. 3 with the linear levels k/u, C = identity), oracle side
// only: it is the comparison operator of the empirical-variance experiment (Appendix A.2) and of
// Thm. 5, not part of the CUDA path.  Level index of y in [0, 1]: floor(y u) or that plus one,
// the upper one with probability y u - floor(y u); the draw is "up iff r23 < floor(p 2^23)".
void orc_dsta_level_index(const double* y, const uint32_t* r23, uint64_t count, int u,
                          int32_t* index) {
    for (uint64_t i = 0; i < count; ++i) {
        double yy = y[i];
        if (yy >= 1.0) { index[i] = u; continue; }
        const double scaled = yy * (double)u;
        const double k = std::floor(scaled);
        const double thr = std::floor((scaled - k) * TWO23);
        index[i] = (int32_t)k + (((double)(r23[i] & 0x7FFFFFu) < thr) ? 1 : 0);
    }
}

// out[i] = D_sta^{p,u}(x)_i = ||x||_p sign(x_i) xi(|x_i| / ||x||_p), one bucket, norm and y in
// double, random thresholds from the domain-1 stream of (seed, worker).
void orc_dsta_apply(const float* x, uint64_t d, int p, int u, uint64_t seed, uint32_t worker,
                    double* out) {
    const float norm_f = norm_p(x, d, p);
    const double norm = (double)norm_f;
    for (uint64_t i = 0; i < d; ++i) {
        if (!(norm > 0.0) || std::isinf(norm)) { out[i] = 0.0; continue; }
        const double y = std::fabs((double)x[i]) / norm;
        const uint32_t r = stream_word(seed, worker, 1u, i) & 0x7FFFFFu;
        int32_t idx;
        orc_dsta_level_index(&y, &r, 1, u, &idx);
        out[i] = std::copysign(norm * (double)idx / (double)u, (double)x[i]);
    }
}

// Natural dithering D_nat^{p,s} of x[0..d) split into B buckets, one norm each.
//   mode 0 (definition): norms are computed here (double accumulation); y = |x| / norm in double.
//   mode 1 (given norm): norms[] is an input; y = fl32(|x| * fl32(1 / norm)), all in binary32.
// domain selects the random stream (1 for the product; 0 lets a test compare with C_nat).
// level: one 4-bit code per entry, entry j in bits 4*(j mod 2).. of byte j/2 (s <= 15);
// sign: as for C_nat (sign bit of x).  x[0] is element j0 of the worker's vector
// (j0 a multiple of 32); ceil(d/2) level bytes and ceil(d/32) sign words are written.
void orc_nd_compress(const float* x, uint64_t d, uint64_t j0, const uint64_t* bucket_off, int B,
                     int p, int s, uint64_t seed, uint32_t worker, uint32_t domain, int mode,
                     float* norms, uint8_t* level, uint32_t* sign) {
    if (mode == 0) orc_norms(x, bucket_off, B, p, norms);
    // Bucket starts need not be even or multiples of 32, so a level byte or a sign word can
    // belong to two buckets: the codes are first worked out entry by entry (buckets are
    // independent of each other), then packed.
    std::vector<uint8_t> code(d), sbit(d);
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const float norm = norms[b];
        const bool degenerate = norm_degenerate(norm);
        for (uint64_t i = bucket_off[b]; i < bucket_off[b + 1]; ++i) {
            const float t = x[i];
            int c = 0;
            if (!degenerate) {
                double y;
                if (mode == 0) {
                    y = std::fabs((double)t) / (double)norm;
                } else {
                    y = (double)ratio_given_norm(std::fabs(t), norm);
                }
                const uint32_t r23 = stream_word(seed, worker, domain, j0 + i) & 0x7FFFFFu;
                c = nd_level_code(y, s, r23);
            }
            code[i] = (uint8_t)c;
            sbit[i] = std::signbit(t) ? 1 : 0;
        }
    }
    const int64_t level_bytes = (int64_t)((d + 1) / 2), sign_words = (int64_t)((d + 31) / 32);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < level_bytes; ++k) {
        const uint64_t i = 2 * (uint64_t)k;
        level[k] = (uint8_t)(code[i] | (i + 1 < d ? code[i + 1] << 4 : 0));
    }
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < sign_words; ++k) {
        uint32_t w = 0;
        for (uint64_t i = 32 * (uint64_t)k; i < 32 * (uint64_t)k + 32 && i < d; ++i)
            w |= (uint32_t)sbit[i] << (i % 32);
        sign[k] = w;
    }
}

void orc_nd_decode_accumulate(const float* norms, const uint8_t* level, const uint32_t* sign,
                              uint64_t d, const uint64_t* bucket_off, int B, int s, float* acc) {
    (void)d;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (uint64_t i = bucket_off[b]; i < bucket_off[b + 1]; ++i) {
            const int c = (level[i / 2] >> (4 * (i % 2))) & 0xF;
            const float v = nd_decode_value(c, s, norms[b], (sign[i / 32] >> (i % 32)) & 1u);
            acc[i] = acc[i] + v;
        }
    }
}

void orc_nd_aggregate(const float* const* norms, const uint8_t* const* level,
                      const uint32_t* const* sign, int n, uint64_t d, const uint64_t* bucket_off,
                      int B, int s, float* out) {
    (void)d;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (uint64_t j = bucket_off[b]; j < bucket_off[b + 1]; ++j) {
            float acc = 0.0f;
            for (int i = 0; i < n; ++i) {
                const int c = (level[i][j / 2] >> (4 * (j % 2))) & 0xF;
                const float v =
                    nd_decode_value(c, s, norms[i][b], (sign[i][j / 32] >> (j % 32)) & 1u);
                acc = acc + v;
            }
            out[j] = acc;
        }
    }
}

// Random sparsification followed by natural dithering, on one bucket (the whole vector).
// Coordinate j is kept iff its domain-2 stream word is below keep_threshold
// (independent Bernoulli selection with probability keep_threshold / 2^32; the special
// value keep_threshold = 2^32 keeps everything), and a kept entry becomes
// x'_j = fl32(scale * x_j).  Then D_nat^{p,s} of the kept entries with norm
// ||x'||_p over the kept entries, given-norm arithmetic (mode 1 above) and the
// domain-1 stream at the dense index j.
// Output: ascending indices, one byte-packed 4-bit code per kept entry
// (bit 3 = sign, bits 0..2 = level 0..s, s <= 7; entry k in bits 4*(k mod 2).. of byte k/2),
// the count and the norm.  Returns the count; entries beyond cap are counted but not stored.
uint64_t orc_sparse_compress(const float* x, uint64_t d, uint64_t keep_threshold, float scale,
                             int p, int s, uint64_t seed, uint32_t worker, uint32_t* idx,
                             uint8_t* codes, uint64_t cap, float* norm_out,
                             const float* given_norm) {
    // pass 1: selection and the norm of the kept, scaled entries (double accumulation)
    double acc = 0.0;
    bool saw_nan = false;
    uint64_t count = 0;
    for (uint64_t j = 0; j < d; ++j) {
        if ((uint64_t)stream_word(seed, worker, 2u, j) >= keep_threshold) continue;
        const float xs = scale * x[j];
        const double a = std::fabs((double)xs);
        if (std::isnan(a)) saw_nan = true;
        if (p == 1) acc += a;
        else if (p == 2) acc += a * a;
        else if (a > acc) acc = a;
        ++count;
    }
    if (p == 2) acc = std::sqrt(acc);
    float norm = saw_nan ? std::numeric_limits<float>::quiet_NaN() : (float)acc;
    if (given_norm) norm = *given_norm;      // pins the rounding independently of the summation
    *norm_out = norm;
    const bool degenerate = norm_degenerate(norm);
    // pass 2: level codes of the kept entries, in ascending index order
    uint64_t k = 0;
    const uint64_t stored = count < cap ? count : cap;
    std::memset(codes, 0, (size_t)((stored + 1) / 2));
    for (uint64_t j = 0; j < d && k < stored; ++j) {
        if ((uint64_t)stream_word(seed, worker, 2u, j) >= keep_threshold) continue;
        const float xs = scale * x[j];
        int c = 0;
        if (!degenerate) {
            const float yf = ratio_given_norm(std::fabs(xs), norm);
            const uint32_t r23 = stream_word(seed, worker, 1u, j) & 0x7FFFFFu;
            c = nd_level_code((double)yf, s, r23);
        }
        const uint32_t sb = std::signbit(xs) ? 1u : 0u;
        idx[k] = (uint32_t)j;
        codes[k / 2] |= (uint8_t)(((sb << 3) | (uint32_t)c) << (4 * (k % 2)));
        ++k;
    }
    return count;
}

// acc[idx[k]] = acc[idx[k]] + sign * norm * 2^(c-s) for the listed entries.
void orc_sparse_decode_accumulate(const uint32_t* idx, const uint8_t* codes, uint64_t count,
                                  float norm, int s, float* acc) {
    for (uint64_t k = 0; k < count; ++k) {
        const uint32_t code = (codes[k / 2] >> (4 * (k % 2))) & 0xFu;
        const float v = nd_decode_value((int)(code & 7u), s, norm, code >> 3);
        acc[idx[k]] = acc[idx[k]] + v;
    }
}

// The compact form of the sparsified + dithered vector: entries whose level rounds to 0 carry no
// information and are left out of the list.  Same selection, scaling, norm (over all kept
// entries) and rounding as orc_sparse_compress.  A listed entry has level 1..s and the code
// (sign << nb) | (level - 1) with nb = bits needed for s - 1 (2 for s <= 4, so 3-bit codes).
// Codes are stored as bit planes: for the g-th group of 32 listed entries, word
// planes[g * (nb + 1) + b] holds bit b of the 32 codes (entry k in bit k mod 32).
// Returns the number of listed entries (those beyond cap are counted, not stored).
static int bits_for(int s) {
    int nb = 0;
    while ((1 << nb) < s) ++nb;
    return nb;
}

uint64_t orc_sparse_compact_compress(const float* x, uint64_t d, uint64_t keep_threshold,
                                     float scale, int p, int s, uint64_t seed, uint32_t worker,
                                     uint32_t* idx, uint32_t* planes, uint64_t cap,
                                     float* norm_out) {
    // pass 1: the norm of the kept, scaled entries.  Sums are taken in index order; the maximum
    // does not depend on the order, so that case may be split over threads.
    double acc = 0.0;
    bool saw_nan = false;
    if (p == 0) {
#pragma omp parallel for schedule(static) reduction(max : acc) reduction(|| : saw_nan)
        for (int64_t j = 0; j < (int64_t)d; ++j) {
            if ((uint64_t)stream_word(seed, worker, 2u, (uint64_t)j) >= keep_threshold) continue;
            const float xs = scale * x[j];
            const double a = std::fabs((double)xs);
            if (std::isnan(a)) saw_nan = true;
            else if (a > acc) acc = a;
        }
    } else {
        for (uint64_t j = 0; j < d; ++j) {
            if ((uint64_t)stream_word(seed, worker, 2u, j) >= keep_threshold) continue;
            const float xs = scale * x[j];
            const double a = std::fabs((double)xs);
            if (std::isnan(a)) saw_nan = true;
            if (p == 1) acc += a;
            else acc += a * a;
        }
    }
    if (p == 2) acc = std::sqrt(acc);
    const float norm = saw_nan ? std::numeric_limits<float>::quiet_NaN() : (float)acc;
    *norm_out = norm;
    const int nb = bits_for(s);
    const uint64_t groups = (cap + 31) / 32;
    std::memset(planes, 0, (size_t)(groups * (uint64_t)(nb + 1)) * 4);
    if (norm_degenerate(norm)) return 0;            // every level is 0: nothing to list
    // pass 2: per coordinate, 0 = not listed, else code + 1 (coordinates are independent);
    // then the list is written in ascending index order
    std::vector<uint8_t> entry(d);
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)d; ++j) {
        entry[j] = 0;
        if ((uint64_t)stream_word(seed, worker, 2u, (uint64_t)j) >= keep_threshold) continue;
        const float xs = scale * x[j];
        const float yf = ratio_given_norm(std::fabs(xs), norm);
        const uint32_t r23 = stream_word(seed, worker, 1u, (uint64_t)j) & 0x7FFFFFu;
        const int c = nd_level_code((double)yf, s, r23);
        if (c == 0) continue;
        entry[j] = (uint8_t)((((std::signbit(xs) ? 1u : 0u) << nb) | (uint32_t)(c - 1)) + 1u);
    }
    uint64_t k = 0;
    for (uint64_t j = 0; j < d; ++j) {
        if (!entry[j]) continue;
        if (k < cap) {
            const uint32_t code = (uint32_t)entry[j] - 1u;
            idx[k] = (uint32_t)j;
            for (int b = 0; b <= nb; ++b)
                planes[(k / 32) * (uint64_t)(nb + 1) + (uint64_t)b] |= ((code >> b) & 1u) << (k % 32);
        }
        ++k;
    }
    return k;
}

void orc_sparse_compact_decode_accumulate(const uint32_t* idx, const uint32_t* planes,
                                          uint64_t count, float norm, int s, float* acc) {
    const int nb = bits_for(s);
    for (uint64_t k = 0; k < count; ++k) {
        uint32_t code = 0;
        for (int b = 0; b <= nb; ++b)
            code |= ((planes[(k / 32) * (uint64_t)(nb + 1) + (uint64_t)b] >> (k % 32)) & 1u) << b;
        const int level = (int)(code & ((1u << nb) - 1u)) + 1;
        const float v = nd_decode_value(level, s, norm, code >> nb);
        acc[idx[k]] = acc[idx[k]] + v;
    }
}

// ---- the paper's 8-bit wire format and integer aggregation ---------------------------------
// Experimental set-up appendix: 1 sign bit, exponents clipped to [-50, 10] (6 bits), one bit
// that flags zeros; the aggregator restores the values as 64-bit integers and adds them.
// Byte layout chosen here: bit 7 sign, bit 6 zero flag, bits 0..5 exponent + 50.
static uint8_t code8_of_value(double value) {
    const uint8_t sign = std::signbit(value) ? 0x80 : 0x00;
    const double a = std::fabs(value);
    if (a == 0.0) return (uint8_t)(sign | 0x40);
    int e = std::isinf(a) ? 1000 : std::ilogb(a);
    if (e < -50) e = -50;
    if (e > 10) e = 10;
    return (uint8_t)(sign | (uint8_t)(e + 50));
}

static long long restore8_int(uint8_t c) {
    if (c & 0x40) return 0;
    const long long v = (long long)1 << (c & 0x3F);
    return (c & 0x80) ? -v : v;
}

void orc_nc8_compress(const float* x, uint64_t d, uint64_t j0, uint64_t seed, uint32_t worker,
                      uint8_t* code) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)d; ++i) {
        const uint32_t r23 = stream_word(seed, worker, 0u, j0 + (uint64_t)i) & 0x7FFFFFu;
        code[i] = code8_of_value(cnat_value(x[i], r23));
    }
}

// decoded values +-2^(e-50) (0 for the zero flag)
void orc_nc8_decode(const uint8_t* code, uint64_t d, float* out) {
    for (uint64_t i = 0; i < d; ++i)
        out[i] = (float)std::ldexp((double)restore8_int(code[i]), -50);
}

// exact integer sums (returned as well, for the pins) and their fp32 value fl32(sum) * 2^-50
void orc_nc8_aggregate(const uint8_t* const* codes, int n, uint64_t d, float* out,
                       int64_t* sums) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)d; ++j) {
        long long acc = 0;
        for (int i = 0; i < n; ++i) acc += restore8_int(codes[i][j]);
        if (sums) sums[j] = acc;
        out[j] = (float)acc * 0x1p-50f;
    }
}

// C_nat of the integer sum S (value S 2^-50), Def. 1 on exact integers: floor power 2^e, ceil
// power 2^(e+1), up-probability (|S| - 2^e) / 2^e, the draw "up iff r23 < floor(p 2^23)".
void orc_nc8_aggregate_compress(const uint8_t* const* codes, int n, uint64_t d, uint64_t seed,
                                uint32_t master, uint8_t* out_code) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)d; ++j) {
        long long acc = 0;
        for (int i = 0; i < n; ++i) acc += restore8_int(codes[i][j]);
        if (acc == 0) { out_code[j] = 0x40; continue; }
        const bool neg = acc < 0;
        const unsigned __int128 a = neg ? (unsigned __int128)(-(__int128)acc) : (unsigned __int128)acc;
        int e = 0;
        while ((a >> (e + 1)) != 0) ++e;
        const unsigned __int128 lo = (unsigned __int128)1 << e;
        const uint64_t thr = (uint64_t)(((a - lo) << 23) >> e);       // floor(p_up * 2^23)
        const uint32_t r23 = stream_word(seed, master, 0u, (uint64_t)j) & 0x7FFFFFu;
        const int e_out = e + ((uint64_t)r23 < thr ? 1 : 0);
        const double value = std::ldexp(neg ? -1.0 : 1.0, e_out - 50);
        out_code[j] = code8_of_value(value);
    }
}

// ---- selection of exactly q coordinates -----------------------------------------------------
// mask[j] = 1 for the q coordinates with the smallest keys, ties going to the lower index.
// With i.i.d. uniform keys this is a uniformly random subset of size q, which is the mask xi of
// the sparsifier definition (S^q: exactly q non-zeros).  Written as the definition: sort.
void orc_select_smallest(const uint32_t* keys, uint64_t d, uint64_t q, uint8_t* mask) {
    std::vector<uint64_t> order(d);
    for (uint64_t j = 0; j < d; ++j) order[j] = j;
    std::stable_sort(order.begin(), order.end(),
                     [&](uint64_t a, uint64_t b) { return keys[a] < keys[b]; });
    std::memset(mask, 0, (size_t)d);
    for (uint64_t k = 0; k < q && k < d; ++k) mask[order[k]] = 1;
}

// S^q with exactly q kept coordinates (keys = the domain-2 stream words), x' = (d / q) x on the
// kept coordinates (scale passed in as binary32), then D_nat^{p,s} in the compact form of
// orc_sparse_compact_compress.  Returns the number of listed entries.
uint64_t orc_sparse_exact_compress(const float* x, uint64_t d, uint64_t q, float scale, int p,
                                   int s, uint64_t seed, uint32_t worker, uint32_t* idx,
                                   uint32_t* planes, uint64_t cap, float* norm_out,
                                   const float* given_norm) {
    std::vector<uint32_t> keys(d);
    for (uint64_t j = 0; j < d; ++j) keys[j] = stream_word(seed, worker, 2u, j);
    std::vector<uint8_t> mask(d);
    orc_select_smallest(keys.data(), d, q, mask.data());
    double acc = 0.0;
    bool saw_nan = false;
    for (uint64_t j = 0; j < d; ++j) {
        if (!mask[j]) continue;
        const float xs = scale * x[j];
        const double a = std::fabs((double)xs);
        if (std::isnan(a)) saw_nan = true;
        if (p == 1) acc += a;
        else if (p == 2) acc += a * a;
        else if (a > acc) acc = a;
    }
    if (p == 2) acc = std::sqrt(acc);
    // given_norm: round against a norm computed elsewhere (binary32), for checking the level
    // codes of an implementation whose norm differs in the last bits by summation order
    const float norm = given_norm ? *given_norm
                     : saw_nan ? std::numeric_limits<float>::quiet_NaN() : (float)acc;
    *norm_out = norm;
    const int nb = bits_for(s);
    std::memset(planes, 0, (size_t)(((cap + 31) / 32) * (uint64_t)(nb + 1)) * 4);
    if (norm_degenerate(norm)) return 0;
    uint64_t k = 0;
    for (uint64_t j = 0; j < d; ++j) {
        if (!mask[j]) continue;
        const float xs = scale * x[j];
        const float yf = ratio_given_norm(std::fabs(xs), norm);
        const uint32_t r23 = stream_word(seed, worker, 1u, j) & 0x7FFFFFu;
        const int c = nd_level_code((double)yf, s, r23);
        if (c == 0) continue;
        if (k < cap) {
            const uint32_t code = ((std::signbit(xs) ? 1u : 0u) << nb) | (uint32_t)(c - 1);
            idx[k] = (uint32_t)j;
            for (int b = 0; b <= nb; ++b)
                planes[(k / 32) * (uint64_t)(nb + 1) + (uint64_t)b] |= ((code >> b) & 1u) << (k % 32);
        }
        ++k;
    }
    return k;
}

// TopK followed by C_nat (the paper's TopK-C_nat of the experiments section): the K entries of
// largest magnitude (compared as binary32 bit patterns with the sign cleared, so NaN patterns
// rank above inf; equal magnitudes: lower index first), listed in ascending index order, each
// with the 9-bit code of C_nat(x_j) drawn from the stream (seed, worker, j).
// exp: one byte per listed entry; sign: bit (k mod 32) of word k / 32.
void orc_topk_compress(const float* x, uint64_t d, uint64_t K, uint64_t seed, uint32_t worker,
                       uint32_t* idx, uint8_t* exp, uint32_t* sign) {
    std::vector<uint32_t> keys(d);
    for (uint64_t j = 0; j < d; ++j) {
        uint32_t bits;
        std::memcpy(&bits, &x[j], 4);
        keys[j] = ~(bits & 0x7FFFFFFFu);            // largest magnitude = smallest key
    }
    std::vector<uint8_t> mask(d);
    orc_select_smallest(keys.data(), d, K, mask.data());
    const uint64_t listed = K < d ? K : d;
    std::memset(sign, 0, (size_t)((listed + 31) / 32) * 4);
    uint64_t k = 0;
    for (uint64_t j = 0; j < d; ++j) {
        if (!mask[j]) continue;
        const uint32_t r23 = stream_word(seed, worker, 0u, j) & 0x7FFFFFu;
        uint32_t sb;
        cnat_code(cnat_value(x[j], r23), &exp[k], &sb);
        idx[k] = (uint32_t)j;
        sign[k / 32] |= sb << (k % 32);
        ++k;
    }
}

void orc_topk_decode_accumulate(const uint32_t* idx, const uint8_t* exp, const uint32_t* sign,
                                uint64_t count, float* acc) {
    for (uint64_t k = 0; k < count; ++k) {
        const float v = cnat_decode(exp[k], (sign[k / 32] >> (k % 32)) & 1u);
        acc[idx[k]] = acc[idx[k]] + v;
    }
}

// ---- 16-bit inputs ----------------------------------------------------------------------
// The real value of a bfloat16 (8-bit exponent, 7-bit mantissa) or binary16 (5-bit exponent,
// 10-bit mantissa) pattern, by the format definition.  Both are exactly representable in binary32.
static float value_of_16bit(uint16_t h, int dtype) {
    const int sign = h >> 15;
    double a;
    if (dtype == 1) {                                   // bfloat16
        const int e = (h >> 7) & 0xFF, m = h & 0x7F;
        if (e == 0xFF) a = m ? std::numeric_limits<double>::quiet_NaN()
                             : std::numeric_limits<double>::infinity();
        else if (e == 0) a = std::ldexp((double)m / 128.0, -126);
        else a = std::ldexp(1.0 + (double)m / 128.0, e - 127);
    } else {                                            // binary16
        const int e = (h >> 10) & 0x1F, m = h & 0x3FF;
        if (e == 0x1F) a = m ? std::numeric_limits<double>::quiet_NaN()
                             : std::numeric_limits<double>::infinity();
        else if (e == 0) a = std::ldexp((double)m / 1024.0, -14);
        else a = std::ldexp(1.0 + (double)m / 1024.0, e - 15);
    }
    return (float)(sign ? -a : a);
}

// C_nat (Def. 1) of 16-bit inputs: the operator on the real value, coded as for binary32.
void orc_nc_compress_typed(const uint16_t* x, int dtype, uint64_t d, uint64_t seed,
                           uint32_t worker, uint8_t* exp, uint32_t* sign) {
    std::memset(sign, 0, (size_t)((d + 31) / 32) * 4);
    for (uint64_t j = 0; j < d; ++j) {
        const float t = value_of_16bit(x[j], dtype);
        const uint32_t r23 = stream_word(seed, worker, 0u, j) & 0x7FFFFFu;
        uint32_t sb;
        cnat_code(cnat_value(t, r23), &exp[j], &sb);
        sign[j / 32] |= sb << (j % 32);
    }
}

// C_nat (Def. 1) of bfloat16 inputs with a short random threshold.  A bfloat16 value has 7
// mantissa bits, so its up-probability m = 1 - p(t) is a multiple of 1/128 and 7 random bits
// decide the rounding exactly: "up" iff r7 < m * 128.  The draw is r7 = low 7 bits of byte
// (j mod 4) of the stream word with index j / 4 in domain 4 (so one generator block of four words
// serves 16 entries).  Written as the binary32 rule with r23 = r7 * 2^16: the threshold
// m * 2^23 of a bfloat16 value is a multiple of 2^16.  Codes and edge cases as for binary32.
void orc_nc_compress_bf16_r8(const uint16_t* x, uint64_t d, uint64_t seed, uint32_t worker,
                             uint8_t* exp, uint32_t* sign) {
    std::memset(sign, 0, (size_t)((d + 31) / 32) * 4);
    for (uint64_t j = 0; j < d; ++j) {
        const float t = value_of_16bit(x[j], 1);
        const uint32_t word = stream_word(seed, worker, 4u, j / 4);
        const uint32_t r7 = (word >> (8 * (j % 4))) & 0x7Fu;
        uint32_t sb;
        cnat_code(cnat_value(t, r7 << 16), &exp[j], &sb);
        sign[j / 32] |= sb << (j % 32);
    }
}

// C_nat (Def. 1) of binary16 inputs with a short random threshold.  A binary16 value has 10
// mantissa bits (a subnormal has fewer), so its up-probability m = 1 - p(t) is a multiple of
// 1/1024 and 10 random bits decide the rounding exactly: "up" iff r10 < m * 1024.  The draw is
// r10 = low 10 bits of half-word (j mod 2) of the stream word with index j / 2 in domain 5 (one
// generator block of four words serves 8 entries).  Written as the binary32 rule with
// r23 = r10 * 2^13: the threshold m * 2^23 of a binary16 value is a multiple of 2^13.
void orc_nc_compress_f16_r16(const uint16_t* x, uint64_t d, uint64_t seed, uint32_t worker,
                             uint8_t* exp, uint32_t* sign) {
    std::memset(sign, 0, (size_t)((d + 31) / 32) * 4);
    for (uint64_t j = 0; j < d; ++j) {
        const float t = value_of_16bit(x[j], 2);
        const uint32_t word = stream_word(seed, worker, 5u, j / 2);
        const uint32_t r10 = (word >> (16 * (j % 2))) & 0x3FFu;
        uint32_t sb;
        cnat_code(cnat_value(t, r10 << 13), &exp[j], &sb);
        sign[j / 32] |= sb << (j % 32);
    }
}

void orc_values_of_16bit(const uint16_t* x, int dtype, uint64_t d, float* out) {
    for (uint64_t j = 0; j < d; ++j) out[j] = value_of_16bit(x[j], dtype);
}

// ---- binary64 inputs: 11-bit exponent + sign ---------------------------------------------
// Def. 1 on a binary64 t ("11 bits for the exponent and 1 for the sign", Sec. 2).  The mantissa has
// 52 bits, so the threshold needs 52 random bits: r52 = (low 23 bits of the domain-0 word of
// element j) * 2^29 + (domain-3 word of element j) / 8, "up" iff r52 < (1 - p(t)) * 2^52.
// Edge policy as for binary32 with the binary64 limits (subnormals bracket [0, 2^-1022],
// 2^1023 and above never round up, inf / NaN give exponent field 2047).
static double cnat64_value(double t, uint64_t r52) {
    if (t == 0.0) return t;
    if (std::isnan(t) || std::isinf(t))
        return std::copysign(std::numeric_limits<double>::infinity(), t);
    const double a = std::fabs(t);
    double lo, hi;
    if (a < 0x1p-1022) {
        lo = 0.0;
        hi = 0x1p-1022;
    } else {
        const int fl = std::ilogb(a);
        lo = std::ldexp(1.0, fl);
        if (fl >= 1023) return std::copysign(lo, t);
        hi = std::ldexp(1.0, fl + 1);
    }
    const double p_up = (a - lo) / (hi - lo);            // exact: a - lo and a power of two
    const bool up = (double)r52 < p_up * 0x1p52;          // both sides exact integers below 2^53
    return std::copysign(up ? hi : lo, t);
}

static uint64_t stream_r52(uint64_t seed, uint32_t worker, uint64_t j) {
    const uint64_t top = stream_word(seed, worker, 0u, j) & 0x7FFFFFu;
    const uint64_t low = stream_word(seed, worker, 3u, j) >> 3;
    return (top << 29) | low;
}

// 12-bit code of +-0, +-2^k, +-inf: 11-bit biased exponent and the sign
static void cnat64_code(double value, uint32_t* e11, uint32_t* sign_bit) {
    *sign_bit = std::signbit(value) ? 1u : 0u;
    const double a = std::fabs(value);
    if (a == 0.0) *e11 = 0;
    else if (std::isinf(a)) *e11 = 2047;
    else *e11 = (uint32_t)(std::ilogb(a) + 1023);
}

// exp_lo[j] = low 8 bits of the exponent field; nibble (j mod 2) of hi[j / 2] = sign * 8 +
// (exponent field >> 8)
void orc_nc64_compress(const double* x, uint64_t d, uint64_t seed, uint32_t worker,
                       uint8_t* exp_lo, uint8_t* hi) {
    std::memset(hi, 0, (size_t)((d + 1) / 2));
    for (uint64_t j = 0; j < d; ++j) {
        uint32_t e11, sb;
        cnat64_code(cnat64_value(x[j], stream_r52(seed, worker, j)), &e11, &sb);
        exp_lo[j] = (uint8_t)(e11 & 0xFFu);
        hi[j / 2] |= (uint8_t)(((sb << 3) | (e11 >> 8)) << (4 * (j % 2)));
    }
}

static double cnat64_decode(uint32_t e11, uint32_t sign_bit) {
    double a;
    if (e11 == 0) a = 0.0;
    else if (e11 == 2047) a = std::numeric_limits<double>::infinity();
    else a = std::ldexp(1.0, (int)e11 - 1023);
    return sign_bit ? -a : a;
}

// out[j] = sum over the workers, in worker order, of the decoded values (binary64 adds from +0)
void orc_nc64_aggregate(const uint8_t* const* exp_lo, const uint8_t* const* hi, int n, uint64_t d,
                        double* out) {
    for (uint64_t j = 0; j < d; ++j) {
        double acc = 0.0;
        for (int i = 0; i < n; ++i) {
            const uint32_t nib = (hi[i][j / 2] >> (4 * (j % 2))) & 0xFu;
            acc = acc + cnat64_decode(((nib & 7u) << 8) | exp_lo[i][j], nib >> 3);
        }
        out[j] = acc;
    }
}

void orc_cnat64_values(const double* t, const uint64_t* r52, uint64_t n, double* out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = cnat64_value(t[i], r52[i]);
}

// ---- receiver-side regeneration of the kept set --------------------------------------------
// With independent selection the kept set is a function of (seed, worker, threshold) alone, so
// the index list need not travel: the receiver walks the coordinates, regenerates "kept iff
// stream word (domain 2, j) < threshold" and pairs the k-th kept coordinate with the k-th code of
// the listed 4-bit form (orc_sparse_compress).  Only the first `count` kept coordinates are applied.
void orc_sparse_regen_decode_accumulate(const uint8_t* codes, uint64_t count, float norm,
                                        uint64_t d, uint64_t keep_threshold, int s, uint64_t seed,
                                        uint32_t worker, float* acc) {
    uint64_t k = 0;
    for (uint64_t j = 0; j < d && k < count; ++j) {
        if ((uint64_t)stream_word(seed, worker, 2u, j) >= keep_threshold) continue;
        const uint32_t code = (codes[k / 2] >> (4 * (k % 2))) & 0xFu;
        acc[j] = acc[j] + nd_decode_value((int)(code & 7u), s, norm, code >> 3);
        ++k;
    }
}

}  // extern "C"

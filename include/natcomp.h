/* natcomp.h -- C ABI of the natural-compression hot path for NVIDIA B200 (sm_100a).
 *
 * The operators are those of "Natural Compression for Distributed Deep Learning"
 * (arXiv 1905.10988): the per-entry compressor C_nat (Def. 1, Sec. 2), natural
 * dithering D_nat^{p,s} (Def. 3), random sparsification composed with dithering
 * (appendix "Sparsification - Formal Definition", Thm. 3) and the master-side
 * aggregation  Delta = sum_i C(g_i)  of Algorithm 1.
 *
 * Conventions shared by every call
 *   - Pointers are DEVICE pointers unless a parameter is documented as a host array.
 *     "host array of device pointers" arguments hold at most NC_MAX_WORKERS entries
 *     and are copied into the kernel's parameters before the call returns.
 *   - The caller owns every buffer; the library allocates and frees nothing.  Scratch
 *     memory is passed in as `workspace`; its size is queried with the
 *     *_workspace_bytes helpers.
 *   - fp32 vectors (x, acc, out) must be 32-byte aligned; exp, sign, level, idx, codes and
 *     workspace 16-byte aligned; bucket_off 8-byte, norms and count 4-byte aligned
 *     (NC_ERR_ALIGN otherwise).
 *   - Calls are asynchronous on `stream`, never synchronise, and return after the
 *     launch.  The return value covers argument validation and the launch status.
 *   - d == 0 returns NC_OK and launches nothing.
 *   - Packed planes are written including their zero padding up to the size the
 *     *_bytes helpers return; padding is ignored on decode.
 *
 * Random stream (the paper fixes none): Philox4x32-10 with
 *   key = (low32(seed), high32(seed)), counter = (low32(q), high32(q), worker, domain),
 *   q = j / 4; element j of a worker's vector uses output word j mod 4, low 23 bits.
 *   domain 0: C_nat, 1: D_nat rounding, 2: sparsifier selection, 3: low bits of binary64
 *   thresholds, 4: byte-wide draws of nc_compress_bf16_r8, 5: half-word draws of
 *   nc_compress_f16_r16.
 * The stream depends on (seed, worker, j) only, so outputs are reproducible and
 * independent of launch geometry.
 *
 * Packed formats
 *   C_nat, 9 bits per entry (Sec. 2, "From 32 to 9 bits"):
 *     exp[j]        biased binary32 exponent of C_nat(x_j)   (uint8; 0 encodes +-0, 255 +-inf)
 *     sign[j / 32]  bit (j mod 32) = sign bit of x_j          (uint32 words)
 *   D_nat^{p,s}, s <= 15: per bucket one fp32 norm; per entry a level code c in 0..s
 *     (c = 0 <-> 0, c = k <-> 2^(k-s)) in bits 4*(j mod 2).. of level[j / 2], plus the
 *     same sign plane.
 *   Sparse D_nat, s <= 7: ascending uint32 indices; codes[k / 2] bits 4*(k mod 2)..:
 *     bit 3 = sign, bits 0..2 = level code of the k-th kept entry.
 *
 * Inputs the paper does not discuss: +-0 keeps its sign and encodes as exponent 0;
 * a subnormal x is rounded to +-0 or +-2^-126 with up-probability |x| / 2^-126;
 * 2^127 < |x| < inf is never rounded up; +-inf and NaN encode as +-inf.
 */
#ifndef NATCOMP_H_
#define NATCOMP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#ifndef __DRIVER_TYPES_H__
typedef struct CUstream_st* cudaStream_t;
#endif

typedef enum {
    NC_OK = 0,
    NC_ERR_INVALID = -1,     /* null pointer, n or s or p out of range, inconsistent sizes */
    NC_ERR_ALIGN = -2,       /* a pointer is not aligned as required */
    NC_ERR_UNSUPPORTED = -3, /* p other than 1, 2, NC_P_INF */
    NC_ERR_WORKSPACE = -4,   /* workspace_bytes smaller than the query helper's answer */
    NC_ERR_CUDA = -5,        /* the CUDA runtime reported an error at launch */
    NC_ERR_TOO_LARGE = -6    /* the problem does not fit the fixed scratch of a *_static call */
} nc_status;

#define NC_MAX_WORKERS 64
#define NC_P_INF 0 /* value of `p` that selects the max-norm */

/* Human-readable name of a status code (static string). */
const char* nc_status_string(int status);

/* ---- sizes (host-only arithmetic, no CUDA calls) -------------------------------- */
size_t nc_exp_bytes(size_t d);   /* d rounded up to a multiple of 16 */
size_t nc_sign_bytes(size_t d);  /* 4 * ceil(d / 32) rounded up to a multiple of 16 */
size_t nd_level_bytes(size_t d); /* ceil(d / 2) rounded up to a multiple of 16 */
size_t nd_workspace_bytes(size_t d, int num_buckets);
size_t nd_sparse_workspace_bytes(size_t d, size_t cap);

/* ---- C_nat (Def. 1; binary32 form in Sec. 2) ----------------------------------- */

/* Worker side: exp/sign <- code of C_nat(x_j), j = 0..d-1, with the stream (seed, worker, j).
 * x: fp32[d].  exp: nc_exp_bytes(d).  sign: nc_sign_bytes(d).  Bit-exact w.r.t. Def. 1. */
nc_status nc_compress(const float* x, size_t d, uint64_t seed, uint32_t worker, uint8_t* exp,
                      uint32_t* sign, cudaStream_t stream);

/* The same for n workers' vectors of equal length d in one launch.  xs, exps, signs are host
 * arrays of n device pointers, workers a host array of n worker ids (1 <= n <= NC_MAX_WORKERS). */
nc_status nc_compress_batch(const float* const* xs, size_t d, uint64_t seed,
                            const uint32_t* workers, uint8_t* const* exps,
                            uint32_t* const* signs, int n, cudaStream_t stream);

/* The paper's deterministic control variant (experimental set-up appendix; there it exposes the
 * cost of sampling): the same 9-bit code,
 * but every entry goes to the nearer of its two neighbouring powers of two (the midpoint
 * 1.5 * 2^k goes up), with no random numbers.  Biased.  Edge cases as for nc_compress. */
nc_status nc_compress_nearest(const float* x, size_t d, uint8_t* exp, uint32_t* sign,
                              cudaStream_t stream);
nc_status nc_compress_nearest_batch(const float* const* xs, size_t d, uint8_t* const* exps,
                                    uint32_t* const* signs, int n, cudaStream_t stream);

/* Master side, one worker (Algorithm 1, aggregation step): acc[j] <- acc[j] + decode(code_j),
 * one binary32 addition per entry.  acc: fp32[d], read and written. */
nc_status nc_decode_accumulate(const uint8_t* exp, const uint32_t* sign, size_t d, float* acc,
                               cudaStream_t stream);

/* Master side, n workers (Algorithm 1: Delta = sum_i Delta_i):
 * out[j] <- (((+0 + v_0j) + v_1j) + ... + v_{n-1,j}) in binary32, v_ij = decode(code of worker i).
 * exps, signs: host arrays of n device pointers.  out: fp32[d], overwritten.
 * Identical to zero-filling out and calling nc_decode_accumulate for i = 0..n-1. */
nc_status nc_aggregate(const uint8_t* const* exps, const uint32_t* const* signs, int n, size_t d,
                       float* out, cudaStream_t stream);

/* Master side with compression of the aggregate (Algorithm 1, "compress g = C_M(Delta)", with
 * C_M = C_nat; the bidirectional-compression models of the speed-up appendix): the 9-bit code of
 * C_nat(sum_i v_ij), the sum taken as in nc_aggregate and never written to memory.  The rounding
 * uses the C_nat stream of (seed, worker = master, j).  out_exp: nc_exp_bytes(d), out_sign:
 * nc_sign_bytes(d).  Identical to nc_aggregate followed by nc_compress(.., seed, master, ..). */
nc_status nc_aggregate_compress(const uint8_t* const* exps, const uint32_t* const* signs, int n,
                                size_t d, uint64_t seed, uint32_t master, uint8_t* out_exp,
                                uint32_t* out_sign, cudaStream_t stream);

/* The same for a shard of a longer vector (the master's work split over several devices, each
 * owning a range of coordinates): the d entries are the coordinates first_index .. first_index+d-1
 * of the whole vector and the rounding uses the stream of (seed, master, first_index + j), so the
 * shards' outputs put side by side equal one nc_aggregate_compress over the whole vector.
 * first_index must be a multiple of 1024 (NC_ERR_INVALID otherwise); every pointer addresses the
 * shard's own first entry. */
nc_status nc_aggregate_compress_shard(const uint8_t* const* exps, const uint32_t* const* signs,
                                      int n, size_t d, uint64_t first_index, uint64_t seed,
                                      uint32_t master, uint8_t* out_exp, uint32_t* out_sign,
                                      cudaStream_t stream);

/* Reference point (the "no compression" baseline of Table 1): out[j] <- ((+0 + x_0j) + x_1j) + ...
 * xs: host array of n device pointers to fp32[d]. */
nc_status nc_sum_fp32(const float* const* xs, int n, size_t d, float* out, cudaStream_t stream);

/* ---- D_nat^{p,s} (Def. 3 with levels 2^-u) -------------------------------------- */

/* Worker side.  bucket_off: device array of B+1 ascending element offsets, off[0] = 0, off[B] = d;
 * bucket b = [off[b], off[b+1]) has its own norm ||x_b||_p, p in {1, 2, NC_P_INF}, 1 <= s <= 15.
 * norms: fp32[B] out.  level: nd_level_bytes(d).  sign: nc_sign_bytes(d).
 * workspace: nd_workspace_bytes(d, B) bytes of scratch (contents undefined afterwards).
 * Arithmetic: norm accumulated in binary64 from per-thread binary32 partial sums, rounded once;
 * y = fl32(|x| * fl32(1 / norm)); above 2^(1-s) the up-probability is the mantissa fraction of y
 * (as in C_nat), below it is y * 2^(s-1), both at 2^-23 resolution.  For a subnormal norm, whose
 * reciprocal would overflow, |x| and the norm are both multiplied by 2^24 first (exact, y
 * unchanged).  Given the stored norms the codes are bit-exact w.r.t. Def. 3 in that arithmetic.
 * Degenerate buckets: norm 0 (x = 0 gives D(x) = 0) and a norm that is inf or NaN (the bucket
 * holds an inf or a NaN; Def. 3 has no ratio |x| / norm to round then) get level code 0
 * everywhere, and the norm is stored as it is.  Such a bucket decodes to zeros, so the stored
 * norm is how a receiver sees it; on the worker side `status` reports it:
 * status: optional (may be NULL) device uint32, 4-byte aligned; the call adds 1 to it for every
 * bucket whose norm is inf or NaN.  The caller zeroes it and reads it back when it likes. */
nc_status nd_compress(const float* x, size_t d, const uint64_t* bucket_off, int B, int p, int s,
                      uint64_t seed, uint32_t worker, float* norms, uint8_t* level,
                      uint32_t* sign, void* workspace, size_t workspace_bytes, uint32_t* status,
                      cudaStream_t stream);

/* The same for n workers' vectors of equal length d and one shared bucket table, in three launches
 * in total.  xs, norms, levels, signs: host arrays of n device pointers; workers: host array of n
 * worker ids.  workspace: nd_batch_workspace_bytes(d, B, n). */
size_t nd_batch_workspace_bytes(size_t d, int num_buckets, int n);
nc_status nd_compress_batch(const float* const* xs, size_t d, const uint64_t* bucket_off, int B,
                            int p, int s, uint64_t seed, const uint32_t* workers,
                            float* const* norms, uint8_t* const* levels, uint32_t* const* signs,
                            int n, void* workspace, size_t workspace_bytes, uint32_t* status,
                            cudaStream_t stream);

/* The two halves of nd_compress_batch as calls of their own: the per-bucket norms, and the level
 * rounding against norms that are given (for example after partial norms of a bucket that is
 * split over several devices were combined, or norms that were compressed and decoded again).
 * nd_compress_batch(..) gives exactly what nd_norms_batch(..) followed by nd_round_batch(..)
 * with the same arguments gives.  Arguments as for nd_compress_batch; `norms` is written by the
 * first call and read by the second; workspace: nd_batch_workspace_bytes(d, B, n).
 * Against norms that are not the entries' own, a ratio |x| / norm above 1 (or NaN: a NaN entry
 * under a finite norm) takes the top level s; a norm that is 0, negative, inf or NaN gives level 0
 * for its whole bucket. */
nc_status nd_norms_batch(const float* const* xs, size_t d, const uint64_t* bucket_off, int B, int p,
                         float* const* norms, int n, void* workspace, size_t workspace_bytes,
                         uint32_t* status, cudaStream_t stream);
nc_status nd_round_batch(const float* const* xs, size_t d, const uint64_t* bucket_off, int B, int s,
                         uint64_t seed, const uint32_t* workers, const float* const* norms,
                         uint8_t* const* levels, uint32_t* const* signs, int n,
                         cudaStream_t stream);

/* The same count for norms that are already stored (n workers' norm arrays of B entries each;
 * host array of n device pointers): *status += number of norms that are inf or NaN.  For the
 * master before it aggregates received buffers, and for the sparse calls (B = 1, their `norm`
 * output).  Def. 3 leaves a norm that is not finite undefined; this is how it is made visible. */
nc_status nd_norm_status(const float* const* norms, int n, int B, uint32_t* status,
                         cudaStream_t stream);

/* nd_compress for callers that have no device memory to hand over as workspace and may not
 * allocate any.  (The paper has no counterpart; this is a deployment convenience.)  Typical
 * cases: a gradient hook running while a framework's caching allocator owns all device memory
 * and communication kernels are in flight, where a cudaMalloc would synchronise the device or
 * simply fail; or a process whose memory budget was fixed at start-up.  Such callers still pass
 * the input and every output buffer, but the scratch the kernels need lives in a fixed array
 * inside the library image: nd_static_scratch_bytes() bytes (1 MiB), present on every GPU that
 * loads the library for as long as the process runs.
 *   - Accepted sizes: nd_workspace_bytes(d, B) <= nd_static_scratch_bytes(), i.e. roughly
 *     d <= 89 million entries for a few hundred buckets; anything larger returns
 *     NC_ERR_TOO_LARGE and launches nothing.
 *   - Results are identical to nd_compress with the same arguments.
 *   - The call allocates and frees nothing.  The first call on each device looks up the device
 *     address of the array (a CUDA runtime query, made with that device current); make that
 *     first call before starting any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the previous call left in
 *     it.  Nothing in it needs to start at zero (every slot is written before it is read), but
 *     two calls that overlap on the GPU (different streams, or several host threads) race on
 *     it: serialise them, or use nd_compress with separate workspaces. */
size_t nd_static_scratch_bytes(void);
nc_status nd_compress_static(const float* x, size_t d, const uint64_t* bucket_off, int B, int p,
                             int s, uint64_t seed, uint32_t worker, float* norms, uint8_t* level,
                             uint32_t* sign, uint32_t* status, cudaStream_t stream);

/* Master side, one worker: acc[j] <- acc[j] + sign_j * fl32(norm_b * 2^(c_j - s)); c = 0 adds +-0
 * whatever the norm.  For c > 0 the product is taken as it comes (Def. 3: norm * sign * xi), so
 * a norm that is inf or NaN gives an entry that is not finite. */
nc_status nd_decode_accumulate(const float* norms, const uint8_t* level, const uint32_t* sign,
                               size_t d, const uint64_t* bucket_off, int B, int s, float* acc,
                               cudaStream_t stream);

/* Master side, n workers, fixed order 0..n-1 starting from +0 (see nc_aggregate).
 * norms, levels, signs: host arrays of n device pointers. */
nc_status nd_aggregate(const float* const* norms, const uint8_t* const* levels,
                       const uint32_t* const* signs, int n, size_t d, const uint64_t* bucket_off,
                       int B, int s, float* out, cudaStream_t stream);

/* ---- random sparsification composed with D_nat (Thm. 3; one bucket = the whole vector) ----- */

/* Keep coordinate j iff its domain-2 stream word < keep_threshold (probability
 * keep_threshold / 2^32; keep_threshold = 2^32 keeps all), x'_j = fl32(scale * x_j), then
 * D_nat^{p,s} of the kept entries (norm over kept entries; 1 <= s <= 7).
 * idx: uint32[cap], ascending.  codes: ceil(cap / 2) bytes rounded up to 16.
 * count: device uint32, number of kept entries (may exceed cap; only cap are stored).
 * norm: device fp32.  workspace: nd_sparse_workspace_bytes(d, cap).  d < 2^32. */
nc_status nd_sparse_compress(const float* x, size_t d, uint64_t keep_threshold, float scale,
                             int p, int s, uint64_t seed, uint32_t worker, uint32_t* idx,
                             uint8_t* codes, uint32_t* count, float* norm, size_t cap,
                             void* workspace, size_t workspace_bytes, cudaStream_t stream);

/* The same for n workers' vectors of equal length d in four launches in total.  xs, idxs, codes,
 * counts, norms: host arrays of n device pointers (each worker has its own list of `cap` entries);
 * workspace: nd_sparse_batch_workspace_bytes(d, cap, n). */
size_t nd_sparse_batch_workspace_bytes(size_t d, size_t cap, int n);
nc_status nd_sparse_compress_batch(const float* const* xs, size_t d, uint64_t keep_threshold,
                                   float scale, int p, int s, uint64_t seed,
                                   const uint32_t* workers, uint32_t* const* idxs,
                                   uint8_t* const* codes, uint32_t* const* counts,
                                   float* const* norms, size_t cap, int n, void* workspace,
                                   size_t workspace_bytes, cudaStream_t stream);

/* acc[idx[k]] <- acc[idx[k]] + decoded value, k < min(*count, cap).  Indices are unique within
 * one worker's list, so one call needs no atomics; calls for different workers are applied in
 * the order they are enqueued on the stream. */
nc_status nd_sparse_decode_accumulate(const uint32_t* idx, const uint8_t* codes,
                                      const uint32_t* count, const float* norm, int s, size_t d,
                                      size_t cap, float* acc, cudaStream_t stream);

/* ---- sparse update without an index list --------------------------------------------------
 * With independent selection the kept set is a function of (seed, worker, keep_threshold), so a
 * receiver that knows them can regenerate it instead of receiving idx: the wire carries count,
 * norm and the 4-bit codes only, 0.5 byte per kept entry.
 * Applies the output of nd_sparse_compress made with the same d, keep_threshold, seed and worker:
 * the k-th code goes to the k-th kept coordinate in ascending order, k < min(*count, cap);
 * acc[j] <- acc[j] + sign * fl32(norm * 2^(c - s)).  Cost: one pass of the selection generator
 * over d.  workspace: nd_sparse_regen_workspace_bytes(d) bytes, 16-byte aligned. */
size_t nd_sparse_regen_workspace_bytes(size_t d);
nc_status nd_sparse_regen_decode_accumulate(const uint8_t* codes, const uint32_t* count,
                                            const float* norm, size_t d, uint64_t keep_threshold,
                                            int s, uint64_t seed, uint32_t worker, size_t cap,
                                            float* acc, void* workspace, size_t workspace_bytes,
                                            cudaStream_t stream);

/* ---- compact sparse format: zero levels dropped, codes as bit planes ------------------------
 * Same operator as nd_sparse_compress (sparsifier definition + Def. 3, composition of Thm. 3), in
 * the format "index list + log2(s)+1 bits per listed entry" that the paper's bit counts for
 * sparsified dithering assume: a kept coordinate whose level rounds to 0 decodes to +-0 and is
 * left out of the list.  Listed entry k has level 1..s and code (sign << nb) | (level - 1),
 * nb = ceil(log2 s) (s <= 4: 3-bit codes; s <= 8 supported).  For the g-th group of 32 listed
 * entries, word planes[g * (nb + 1) + b] holds bit b of the 32 codes (entry k in bit k mod 32).
 * idx: uint32[cap]; planes: nd_sparse_plane_bytes(cap, s) bytes, written for all ceil(cap/32)
 * groups (zero beyond the count); count: listed entries (may exceed cap); norm: p-norm over ALL
 * kept entries, as in nd_sparse_compress; workspace: nd_sparse_batch_workspace_bytes(d, cap, n). */
size_t nd_sparse_plane_bytes(size_t cap, int s);
nc_status nd_sparse_compact_compress(const float* x, size_t d, uint64_t keep_threshold,
                                     float scale, int p, int s, uint64_t seed, uint32_t worker,
                                     uint32_t* idx, uint32_t* planes, uint32_t* count, float* norm,
                                     size_t cap, void* workspace, size_t workspace_bytes,
                                     cudaStream_t stream);
nc_status nd_sparse_compact_compress_batch(const float* const* xs, size_t d,
                                           uint64_t keep_threshold, float scale, int p, int s,
                                           uint64_t seed, const uint32_t* workers,
                                           uint32_t* const* idxs, uint32_t* const* planes,
                                           uint32_t* const* counts, float* const* norms,
                                           size_t cap, int n, void* workspace,
                                           size_t workspace_bytes, cudaStream_t stream);
/* acc[idx[k]] <- acc[idx[k]] + sign * fl32(norm * 2^(level - s)) for the listed entries. */
nc_status nd_sparse_compact_decode_accumulate(const uint32_t* idx, const uint32_t* planes,
                                              const uint32_t* count, const float* norm, int s,
                                              size_t d, size_t cap, float* acc,
                                              cudaStream_t stream);

/* Master side, all workers in one call (Algorithm 1, aggregate): out[j] = sum over the n workers,
 * in that order and starting from +0, of their decoded entries at coordinate j; coordinates no
 * list mentions get +0.  Every index list must be ascending (as the compressors write it);
 * entries k >= min(*count, cap) are ignored.  out: float[d], 32-byte aligned, overwritten. */
nc_status nd_sparse_compact_aggregate(const uint32_t* const* idxs, const uint32_t* const* planes,
                                      const uint32_t* const* counts, const float* const* norms,
                                      int n, int s, size_t d, size_t cap, float* out,
                                      cudaStream_t stream);

/* ---- the paper's 8-bit wire format and integer aggregation ----------------------------------
 * Experimental set-up appendix: an 8-bit code made of a sign bit, a flag for zero and a 6-bit
 * exponent clipped to [-50, 10], summed at the aggregator in 64-bit integers; and the "fast
 * aggregation" appendix (values restored as integers with one non-zero bit).
 * Code byte: bit 7 sign, bit 6 zero flag, bits 0..5 = exponent + 50 of C_nat(x) with the
 * exponent clipped to [-50, 10] (+-inf and NaN clip to +-2^10).  Planes hold nc_exp_bytes(d) bytes. */

/* Worker side: code[j] <- 8-bit code of C_nat(x_j) with the stream (seed, worker, j). */
nc_status nc8_compress(const float* x, size_t d, uint64_t seed, uint32_t worker, uint8_t* code,
                       cudaStream_t stream);
nc_status nc8_compress_batch(const float* const* xs, size_t d, uint64_t seed,
                             const uint32_t* workers, uint8_t* const* codes, int n,
                             cudaStream_t stream);

/* Master side: every code is restored as the 64-bit integer +-2^(exponent + 50) (0 for the zero
 * flag), the n integers are added, out[j] <- fl32(sum) * 2^-50.  The result does not depend on the
 * order of the workers.  Exact while |sum| < 2^63 (any n <= 7; any n if no entry is at 2^10). */
nc_status nc8_aggregate(const uint8_t* const* codes, int n, size_t d, float* out,
                        cudaStream_t stream);

/* The same sum, compressed again by C_nat into the 8-bit format (Algorithm 1, g = C_M(Delta)):
 * for the integer S with 2^e <= |S| < 2^(e+1) the code of +-2^(e-50) or +-2^(e+1-50), the upper one
 * iff r23 < floor((|S| - 2^e) 2^23 / 2^e), r23 from the C_nat stream of (seed, master, j). */
nc_status nc8_aggregate_compress(const uint8_t* const* codes, int n, size_t d, uint64_t seed,
                                 uint32_t master, uint8_t* out_code, cudaStream_t stream);

/* ---- 16-bit inputs ---------------------------------------------------------------------------
 * C_nat (Def. 1) of a bfloat16 or binary16 vector.  Such a value is a binary32 value, so the
 * operator is the binary32 rule of Sec. 2 on the exactly converted input: same 9-bit code, same
 * planes and same stream (seed, worker, domain 0, j) as nc_compress; the up-probability is the
 * 7- or 10-bit mantissa fraction (for a binary16 subnormal: its fraction of the binade).
 * x: device pointer to 16-bit patterns, 16-byte aligned.  dtype NC_DTYPE_F32 forwards to
 * nc_compress; other values give NC_ERR_UNSUPPORTED. */
enum { NC_DTYPE_F32 = 0, NC_DTYPE_BF16 = 1, NC_DTYPE_F16 = 2 };
nc_status nc_compress_typed(const void* x, int dtype, size_t d, uint64_t seed, uint32_t worker,
                            uint8_t* exp, uint32_t* sign, cudaStream_t stream);
nc_status nc_compress_typed_batch(const void* const* xs, int dtype, size_t d, uint64_t seed,
                                  const uint32_t* workers, uint8_t* const* exps,
                                  uint32_t* const* signs, int n, cudaStream_t stream);

/* bfloat16 inputs with 7-bit thresholds (Def. 1: a bfloat16 value has 7 mantissa bits, so its
 * up-probability is a multiple of 1/128 and 7 random bits decide the rounding exactly).  Entry j
 * draws the low 7 bits of byte (j mod 4) of stream word j / 4 of domain 4 and is rounded up iff
 * the draw is below its mantissa field: one generator block serves 16 entries, which makes the
 * call memory-bound.  Unbiased like nc_compress_typed, but a different draw, so the two calls give
 * different (equally distributed) codes.  x: d bfloat16 bit patterns, 32-byte aligned.  Planes,
 * edge cases and errors as for nc_compress. */
nc_status nc_compress_bf16_r8(const void* x, size_t d, uint64_t seed, uint32_t worker,
                              uint8_t* exp, uint32_t* sign, cudaStream_t stream);
nc_status nc_compress_bf16_r8_batch(const void* const* xs, size_t d, uint64_t seed,
                                    const uint32_t* workers, uint8_t* const* exps,
                                    uint32_t* const* signs, int n, cudaStream_t stream);

/* binary16 inputs with 10-bit thresholds (Def. 1: a binary16 value has at most 10 mantissa bits,
 * so its up-probability is a multiple of 1/1024).  Entry j draws the low 10 bits of half-word
 * (j mod 2) of stream word j / 2 of domain 5 and is rounded up iff draw / 1024 is below its
 * mantissa fraction (for a subnormal: the fraction above its leading bit): one generator block
 * serves 8 entries.  Same law as nc_compress_typed with NC_DTYPE_F16, a different draw.
 * x: d binary16 bit patterns, 32-byte aligned.  Planes, edge cases and errors as for nc_compress. */
nc_status nc_compress_f16_r16(const void* x, size_t d, uint64_t seed, uint32_t worker,
                              uint8_t* exp, uint32_t* sign, cudaStream_t stream);
nc_status nc_compress_f16_r16_batch(const void* const* xs, size_t d, uint64_t seed,
                                    const uint32_t* workers, uint8_t* const* exps,
                                    uint32_t* const* signs, int n, cudaStream_t stream);

/* ---- binary64 inputs: 12-bit codes -------------------------------------------------------------
 * Sec. 2 gives the code size for binary64: an 11-bit exponent and a sign bit.  C_nat (Def. 1) of a
 * binary64 vector with
 * a 52-bit threshold: r52 = (low 23 bits of the stream word (seed, worker, domain 0, j)) << 29 |
 * (stream word (seed, worker, domain 3, j) >> 3); round up iff r52 < the 52-bit mantissa field.
 * Planes: exp_lo[j] = low 8 bits of the rounded 11-bit exponent field (nc_exp_bytes(d) bytes);
 * hi: 4 bits per entry, (sign << 3) | (exponent field >> 8), entry j in nibble j mod 2 of byte
 * j / 2 (nd_level_bytes(d) bytes).  Padding bytes are written as 0.  Subnormals round to +-0 or
 * +-2^-1022, 2^1023 and above stay, +-inf and NaN give exponent field 2047.  x 32-byte aligned. */
nc_status nc64_compress(const double* x, size_t d, uint64_t seed, uint32_t worker, uint8_t* exp_lo,
                        uint8_t* hi, cudaStream_t stream);
nc_status nc64_compress_batch(const double* const* xs, size_t d, uint64_t seed,
                              const uint32_t* workers, uint8_t* const* exp_los,
                              uint8_t* const* his, int n, cudaStream_t stream);
/* Master side (Algorithm 1, aggregate): out[j] = sum over the n workers, in that order, of the
 * decoded values, binary64 adds starting from +0.  out: double[d], 32-byte aligned. */
nc_status nc64_aggregate(const uint8_t* const* exp_los, const uint8_t* const* his, int n, size_t d,
                         double* out, cudaStream_t stream);

/* ---- exactly q kept coordinates: S^q then D_nat, and TopK then C_nat -------------------------
 * The sparsifier definition of the appendix with exactly q non-zeros ("S^q": xi a uniformly random
 * subset of size q, probabilities q/d), composed with D_nat^{p,s} (Def. 3, Thm. 3), and the
 * TopK-C_nat composition of the experiments.  The random subset is the q coordinates with the
 * smallest words of the selection stream (seed, worker, domain 2, j), equal words by ascending j;
 * TopK takes the K largest |x_j| compared as binary32 bit patterns with the sign cleared (NaN
 * patterns rank above inf), equal magnitudes by ascending j.  Device pointers; x 32-byte aligned,
 * the other buffers 16-byte; workspace: nc_select_workspace_bytes(d, cap) (cap = K for TopK). */
size_t nc_select_workspace_bytes(size_t d, size_t cap);

/* S^q then D_nat^{p,s}: x'_j = scale * x_j on the q selected coordinates (the caller passes
 * scale = fl32(d / q)), norm = ||x'||_p over the selected entries, levels drawn from the dithering
 * stream (domain 1) of coordinate j.  Output in the compact format of nd_sparse_compact_compress
 * (idx, planes, count, norm, cap with the same meaning), decoded by
 * nd_sparse_compact_decode_accumulate.  q > d is taken as d; q = 0 gives count 0 and norm 0. */
nc_status nd_sparse_exact_compress(const float* x, size_t d, uint64_t q, float scale, int p, int s,
                                   uint64_t seed, uint32_t worker, uint32_t* idx,
                                   uint32_t* planes, uint32_t* count, float* norm, size_t cap,
                                   void* workspace, size_t workspace_bytes, cudaStream_t stream);

/* TopK then C_nat (Def. 1): min(K, d) entries listed by ascending coordinate: idx[k] = j,
 * exp[k] = exponent byte of C_nat(x_j) drawn from the stream (seed, worker, domain 0, j) (the
 * same draw nc_compress makes for coordinate j), sign: bit k mod 32 of word k / 32.
 * idx: uint32[K]; exp: K bytes; sign: ceil(K / 32) words.  K = 0 or d = 0 writes nothing. */
nc_status nc_topk_compress(const float* x, size_t d, uint64_t K, uint64_t seed, uint32_t worker,
                           uint32_t* idx, uint8_t* exp, uint32_t* sign, void* workspace,
                           size_t workspace_bytes, cudaStream_t stream);

/* Master side: acc[idx[k]] <- acc[idx[k]] + decoded value, k < count (host integer); indices
 * >= d are skipped.  Indices of one list are distinct, so no atomics are needed. */
nc_status nc_topk_decode_accumulate(const uint32_t* idx, const uint8_t* exp, const uint32_t* sign,
                                    size_t count, size_t d, float* acc, cudaStream_t stream);

/* ---- debug build (no counterpart in the paper) ------------------------------------------------
 * `python paper_1905_10988_b200/build.py --bounds` builds libnatcomp_bounds.so with -DNC_BOUNDS:
 * the same entry points, but every global store of the C_nat and D_nat kernels (nc_compress*,
 * nc_aggregate*, nc_decode_accumulate, nc_sum_fp32, nd_compress*, nd_norms_batch, nd_round_batch,
 * nd_aggregate, nd_decode_accumulate) first checks its address against the ranges the call may
 * write (its outputs and workspace, sized by the *_bytes helpers).  A store outside them is
 * skipped and counted; the kernel runs on and nothing traps.  Calls must not overlap on the GPU in
 * that build (the range table is shared), and it is several times slower.
 * nc_debug_bounds_status: synchronises the device, then *violations = skipped stores since the
 * last reset, *first_address = address of the first one (0 if none); reset != 0 clears the count.
 * nc_debug_bounds_selftest: aims one store 64 bytes past a 16-byte range at the start of
 * `scratch` (device memory, >= 128 bytes, 16-byte aligned), which the check must skip and count:
 * shows that the mechanism is alive without any invalid access.
 * In the regular library both return NC_ERR_UNSUPPORTED. */
nc_status nc_debug_bounds_status(uint64_t* violations, uint64_t* first_address, int reset);
nc_status nc_debug_bounds_selftest(void* scratch, cudaStream_t stream);

/* ---- host-buffer plumbing (no counterpart in the paper, where workers and master exchange
 * these buffers over a network) ------------------------------------------------------------- */

/* Asynchronous copies on `stream` between host memory (pinned for real overlap) and device
 * memory, so that a caller holding gradients on the host can drive the whole path through this
 * ABI.  bytes == 0 is NC_OK. */
nc_status nc_copy_to_device(void* dst_device, const void* src_host, size_t bytes,
                            cudaStream_t stream);
nc_status nc_copy_to_host(void* dst_host, const void* src_device, size_t bytes,
                          cudaStream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* NATCOMP_H_ */

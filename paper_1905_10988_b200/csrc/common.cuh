// Shared device/host helpers of the natcomp CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/natcomp.h"

namespace natcomp {

constexpr int kWarp = 32;
constexpr int kTile = 1024;           // elements one warp handles per tile (8 x float4 per lane)
constexpr int kBlockThreads = 256;    // 8 warps
constexpr int kWarpsPerBlock = kBlockThreads / kWarp;

// Round keys of Philox4x32-10 for one seed: the Weyl sequence is the same for every
// thread, so the host computes it once and the kernels read it from parameter space.
struct PhiloxKeys {
    uint32_t k0[10];
    uint32_t k1[10];
};

inline PhiloxKeys make_philox_keys(uint64_t seed) {
    PhiloxKeys k;
    uint32_t a = (uint32_t)(seed & 0xFFFFFFFFu), b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = a;
        k.k1[r] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return k;
}

inline bool aligned32(const void* p) { return ((uintptr_t)p & 31u) == 0; }
inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }
inline bool aligned4(const void* p) { return ((uintptr_t)p & 3u) == 0; }

__host__ __device__ inline size_t round_up16(size_t v) { return (v + 15) & ~(size_t)15; }

// SM count of the current device (looked up once per device)
inline int device_sm_count() {
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

inline nc_status launch_status() {
    return cudaPeekAtLastError() == cudaSuccess ? NC_OK : NC_ERR_CUDA;
}

// ---- debug build (-DNC_BOUNDS) --------------------------------------------------------------
// Every global store of the C_nat and D_nat kernels first checks its address against the table of
// output ranges that the entry point filled in for this call (outputs and workspace, as sized by
// the *_bytes helpers).  A store outside every range is skipped and recorded in a device status
// block that nc_debug_bounds_status reads: the kernel goes on, nothing traps.  The table and the
// record exist once per translation unit; calls of one unit must not overlap on the GPU in this
// build.  Without NC_BOUNDS all of this compiles to nothing.
struct BoundsRecord {
    unsigned long long violations;     // stores that were skipped
    unsigned long long first_address;  // address of the first one
    unsigned int first_bytes, first_block, first_thread, pad;
};

#ifdef NC_BOUNDS
constexpr int kBoundsRanges = 4 * NC_MAX_WORKERS + 8;
struct BoundsTable {
    unsigned long long lo[kBoundsRanges];
    unsigned long long hi[kBoundsRanges];
    int count;
};
static __device__ BoundsTable g_bounds_table;
static __device__ BoundsRecord g_bounds_record;

static __device__ __noinline__ bool nc_store_ok(const void* p, unsigned bytes) {
    const unsigned long long a = (unsigned long long)p;
    const int n = g_bounds_table.count;
    if (n == 0) return true;           // a unit whose entry points fill in no table checks nothing
    for (int i = 0; i < n; ++i)
        if (a >= g_bounds_table.lo[i] && a + bytes <= g_bounds_table.hi[i]) return true;
    if (atomicAdd(&g_bounds_record.violations, 1ull) == 0ull) {
        g_bounds_record.first_address = a;
        g_bounds_record.first_bytes = bytes;
        g_bounds_record.first_block = blockIdx.x;
        g_bounds_record.first_thread = threadIdx.x;
    }
    return false;
}
#define NC_STORE_OK(p, bytes) nc_store_ok((p), (bytes))

typedef cudaError_t (*BoundsFetch)(BoundsRecord* out, bool reset);
void nc_bounds_register(BoundsFetch fetch);          // api_misc.cu keeps the list of units

static cudaError_t bounds_fetch_this_unit(BoundsRecord* out, bool reset) {
    cudaError_t e = cudaMemcpyFromSymbol(out, g_bounds_record, sizeof(BoundsRecord));
    if (e == cudaSuccess && reset) {
        const BoundsRecord zero = {};
        e = cudaMemcpyToSymbol(g_bounds_record, &zero, sizeof(BoundsRecord));
    }
    return e;
}
static struct BoundsRegistrar {
    BoundsRegistrar() { nc_bounds_register(&bounds_fetch_this_unit); }
} g_bounds_registrar;

// Host side: the ranges a call may write, sent to the device in stream order before its launches.
struct BoundsScope {
    BoundsTable t;
    BoundsScope() { t.count = 0; }
    void add(const void* p, size_t bytes) {
        if (!p || !bytes || t.count >= kBoundsRanges) return;
        t.lo[t.count] = (unsigned long long)(uintptr_t)p;
        t.hi[t.count] = t.lo[t.count] + bytes;
        ++t.count;
    }
    void commit(cudaStream_t stream) {
        cudaMemcpyToSymbolAsync(g_bounds_table, &t, sizeof(BoundsTable), 0, cudaMemcpyHostToDevice,
                                stream);
    }
};
#else
#define NC_STORE_OK(p, bytes) true
struct BoundsScope {
    void add(const void*, size_t) {}
    void commit(cudaStream_t) {}
};
#endif

// a plain store through the same check
#define NC_STORE(ptr, value)                                        \
    do {                                                            \
        if (NC_STORE_OK((ptr), (unsigned)sizeof(*(ptr)))) *(ptr) = (value); \
    } while (0)

// ---- streaming loads / stores: every plane is touched once, keep it out of L1 and
// mark it evict-first in L2.
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
    return __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ uint32_t ld_stream_u32(const void* p) {
    return __ldcs(reinterpret_cast<const unsigned int*>(p));
}
__device__ __forceinline__ void st_stream_u4(void* p, uint4 v) {
    if (NC_STORE_OK(p, 16u)) __stcs(reinterpret_cast<uint4*>(p), v);
}
__device__ __forceinline__ void st_stream_u32(void* p, uint32_t v) {
    if (NC_STORE_OK(p, 4u)) __stcs(reinterpret_cast<unsigned int*>(p), v);
}
__device__ __forceinline__ void st_stream_f4(void* p, float4 v) {
    if (NC_STORE_OK(p, 16u)) __stcs(reinterpret_cast<float4*>(p), v);
}

// 4x4 transpose of bytes across each aligned group of 4 lanes: lane i holds bytes b[i][t]
// (t = 0..3) -> lane t holds bytes b[i][t] (i = 0..3, byte i).
__device__ __forceinline__ uint32_t transpose_bytes_4x4(uint32_t v, int lane) {
    uint32_t t = __shfl_xor_sync(0xFFFFFFFFu, v, 2);
    v = __byte_perm(v, t, (lane & 2) ? 0x3276 : 0x5410);
    t = __shfl_xor_sync(0xFFFFFFFFu, v, 1);
    v = __byte_perm(v, t, (lane & 1) ? 0x3715 : 0x6240);
    return v;
}

// 8x8 transpose of 4-bit fields across each aligned group of 8 lanes.
// In: lane i of a group holds nibbles n[i][k], k = 0..7 (nibble k in bits 4k..4k+3).
// Out: lane k of the group holds nibbles n[i][k], i = 0..7 (nibble i in bits 4i..4i+3).
__device__ __forceinline__ uint32_t transpose_nibbles_8x8(uint32_t v, int lane) {
    uint32_t t = __shfl_xor_sync(0xFFFFFFFFu, v, 4);
    v = __byte_perm(v, t, (lane & 4) ? 0x3276 : 0x5410);
    t = __shfl_xor_sync(0xFFFFFFFFu, v, 2);
    v = __byte_perm(v, t, (lane & 2) ? 0x3715 : 0x6240);
    t = __shfl_xor_sync(0xFFFFFFFFu, v, 1);
    const uint32_t m = 0x0F0F0F0Fu;
    v = (lane & 1) ? (((t >> 4) & m) | (v & ~m)) : ((v & m) | ((t & m) << 4));
    return v;
}

}  // namespace natcomp

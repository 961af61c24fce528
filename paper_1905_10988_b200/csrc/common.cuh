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

// ---- streaming loads / stores: every plane is touched once, keep it out of L1 and
// mark it evict-first in L2.
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
    return __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ uint32_t ld_stream_u32(const void* p) {
    return __ldcs(reinterpret_cast<const unsigned int*>(p));
}
__device__ __forceinline__ void st_stream_u4(void* p, uint4 v) {
    __stcs(reinterpret_cast<uint4*>(p), v);
}
__device__ __forceinline__ void st_stream_u32(void* p, uint32_t v) {
    __stcs(reinterpret_cast<unsigned int*>(p), v);
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

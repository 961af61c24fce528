// Host-only helpers of the C ABI: status strings and packed-plane sizes.
#include "common.cuh"

using namespace natcomp;

extern "C" {

const char* nc_status_string(int status) {
    switch (status) {
        case NC_OK: return "NC_OK";
        case NC_ERR_INVALID: return "NC_ERR_INVALID";
        case NC_ERR_ALIGN: return "NC_ERR_ALIGN";
        case NC_ERR_UNSUPPORTED: return "NC_ERR_UNSUPPORTED";
        case NC_ERR_WORKSPACE: return "NC_ERR_WORKSPACE";
        case NC_ERR_CUDA: return "NC_ERR_CUDA";
        case NC_ERR_TOO_LARGE: return "NC_ERR_TOO_LARGE";
        default: return "NC_ERR_UNKNOWN";
    }
}

size_t nc_exp_bytes(size_t d) { return round_up16(d); }

size_t nc_sign_bytes(size_t d) { return round_up16(4 * ((d + 31) / 32)); }

size_t nd_level_bytes(size_t d) { return round_up16((d + 1) / 2); }

}  // extern "C"

// ---- debug build: the list of translation units that keep a bounds record -----------------
#ifdef NC_BOUNDS
namespace natcomp {
namespace {
struct BoundsUnits {
    BoundsFetch fetch[32];
    int count = 0;
};
BoundsUnits& bounds_units() {
    static BoundsUnits units;        // constructed on first use, before any registrar needs it
    return units;
}
}  // namespace
void nc_bounds_register(BoundsFetch fetch) {
    BoundsUnits& u = bounds_units();
    if (u.count < 32) u.fetch[u.count++] = fetch;
}

__global__ void bounds_selftest_kernel(unsigned int* p) {
    // the address lies outside the one range of the table: the store is skipped and recorded
    st_stream_u32(p, 0xDEADBEEFu);
}
}  // namespace natcomp
#endif

extern "C" {

nc_status nc_debug_bounds_status(uint64_t* violations, uint64_t* first_address, int reset) {
#ifdef NC_BOUNDS
    if (!violations || !first_address) return NC_ERR_INVALID;
    if (cudaDeviceSynchronize() != cudaSuccess) return NC_ERR_CUDA;
    *violations = 0;
    *first_address = 0;
    for (int i = 0; i < bounds_units().count; ++i) {
        BoundsRecord r;
        if (bounds_units().fetch[i](&r, reset != 0) != cudaSuccess) return NC_ERR_CUDA;
        if (r.violations && !*violations) *first_address = r.first_address;
        *violations += r.violations;
    }
    return NC_OK;
#else
    (void)violations; (void)first_address; (void)reset;
    return NC_ERR_UNSUPPORTED;
#endif
}

nc_status nc_debug_bounds_selftest(void* scratch, cudaStream_t stream) {
#ifdef NC_BOUNDS
    if (!scratch || !aligned16(scratch)) return NC_ERR_INVALID;
    // the table admits the first 16 bytes of `scratch`; the kernel aims at byte 64
    BoundsScope scope;
    scope.add(scratch, 16);
    scope.commit(stream);
    bounds_selftest_kernel<<<1, 1, 0, stream>>>(reinterpret_cast<unsigned int*>(scratch) + 16);
    return launch_status();
#else
    (void)scratch; (void)stream;
    return NC_ERR_UNSUPPORTED;
#endif
}

nc_status nc_copy_to_device(void* dst_device, const void* src_host, size_t bytes,
                            cudaStream_t stream) {
    if (bytes == 0) return NC_OK;
    if (!dst_device || !src_host) return NC_ERR_INVALID;
    return cudaMemcpyAsync(dst_device, src_host, bytes, cudaMemcpyHostToDevice, stream) ==
                   cudaSuccess ? NC_OK : NC_ERR_CUDA;
}

nc_status nc_copy_to_host(void* dst_host, const void* src_device, size_t bytes,
                          cudaStream_t stream) {
    if (bytes == 0) return NC_OK;
    if (!dst_host || !src_device) return NC_ERR_INVALID;
    return cudaMemcpyAsync(dst_host, src_device, bytes, cudaMemcpyDeviceToHost, stream) ==
                   cudaSuccess ? NC_OK : NC_ERR_CUDA;
}

}  // extern "C"

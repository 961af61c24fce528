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

extern "C" {

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

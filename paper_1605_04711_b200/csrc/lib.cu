// Library-level entry points: device query, status text, status read-back.
#include "common.cuh"

int twn_current_device(twn_device_info *info)
{
    static twn_device_info cache[64];
    static bool have[64] = {false};
    int dev = 0;
    TWN_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return TWN_ERR_CUDA;
    if (!have[dev]) {
        twn_device_info d;
        d.ordinal = dev;
        TWN_CUDA_OK(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
        TWN_CUDA_OK(cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
        TWN_CUDA_OK(cudaDeviceGetAttribute(&d.cc_minor, cudaDevAttrComputeCapabilityMinor, dev));
        cache[dev] = d;
        have[dev] = true;
    }
    *info = cache[dev];
    if (info->cc_major != 10) return TWN_ERR_UNSUPPORTED_ARCH;
    return TWN_OK;
}

extern "C" const char *twn_strerror(int status)
{
    switch (status) {
        case TWN_OK: return "ok";
        case TWN_ERR_INVALID_ARG: return "invalid argument";
        case TWN_ERR_MISALIGNED: return "pointer or leading dimension not aligned as required";
        case TWN_ERR_WORKSPACE: return "workspace missing or too small";
        case TWN_ERR_NONFINITE: return "a master weight is NaN or infinite";
        case TWN_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case TWN_ERR_CUDA: return "a CUDA call failed";
        case TWN_ERR_UNSUPPORTED_ARCH: return "the current device is not sm_100";
        case TWN_ERR_BAD_CODE: return "a ternary code outside {-1,0,+1}";
        case TWN_ERR_TOO_LARGE: return "size beyond the fixed capacity of this entry point";
        default: return "unknown status";
    }
}

extern "C" int twn_read_status(const int32_t *dev_status, int32_t *host_out, twn_stream_t stream)
{
    TWN_REQUIRE(dev_status != nullptr && host_out != nullptr, TWN_ERR_INVALID_ARG);
    TWN_CUDA_OK(cudaMemcpyAsync(host_out, dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, twn_cu(stream)));
    TWN_CUDA_OK(cudaStreamSynchronize(twn_cu(stream)));
    return TWN_OK;
}

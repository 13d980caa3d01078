// Shared host/device helpers of the CUDA library (not used by the CPU oracle).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "twn.h"

#define TWN_CUDA_OK(expr)                                   \
    do {                                                    \
        cudaError_t twn_e_ = (expr);                        \
        if (twn_e_ != cudaSuccess) return TWN_ERR_CUDA;     \
    } while (0)

#define TWN_REQUIRE(cond, code) \
    do {                        \
        if (!(cond)) return (code); \
    } while (0)

// Properties of the current device, cached per device ordinal.
struct twn_device_info {
    int ordinal;
    int sm_count;
    int cc_major;
    int cc_minor;
};

// TWN_OK and *info filled, TWN_ERR_CUDA, or TWN_ERR_UNSUPPORTED_ARCH when the
// current device is not compute capability 10.x.
int twn_current_device(twn_device_info *info);

static inline bool twn_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static inline cudaStream_t twn_cu(twn_stream_t s) { return reinterpret_cast<cudaStream_t>(s); }

// Launch with programmatic stream serialization: the kernel may start while the kernel before it in the stream
// is still draining (see pdl_wait in tc_ptx.cuh); its blocks run their set-up and wait there.
template <typename... KArgs, typename... Args>
static inline cudaError_t twn_launch_pdl(bool allow, void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t s,
                                         Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = allow ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

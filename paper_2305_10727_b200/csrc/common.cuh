// Shared host-side helpers of libgpusq (argument checks, launch error mapping).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "gpusq.h"
#include "gpusq_testing.h"

namespace gpusq {

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// The compute calls run on compute capability 10.x only; there is no fallback.
inline int check_arch()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPUSQ_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return GPUSQ_ERR_CUDA;
    return major == 10 ? GPUSQ_OK : GPUSQ_ERR_UNSUPPORTED_ARCH;
}

inline int num_sms()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        return 148;
    return n;
}

inline int launch_status()
{
    return cudaGetLastError() == cudaSuccess ? GPUSQ_OK : GPUSQ_ERR_CUDA;
}

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int round_up(int a, int b) { return (a + b - 1) / b * b; }

}  // namespace gpusq

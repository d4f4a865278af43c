// Shared host/device helpers of the library: status plumbing and launch checks.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "war.h"

// Sticky device status word: the first device-side problem since the last war_device_status() call.
// It is one __device__ variable defined in war_api.cu; kernels of other translation units receive its
// address as an argument (war_status_word() resolves it once per device).
int* war_status_word();

__device__ __forceinline__ void war_set_device_status(int* status_word, int code) {
    atomicCAS(status_word, 0, code);
}

#define WAR_CUDA_TRY(expr)                                     \
    do {                                                       \
        cudaError_t e__ = (expr);                              \
        if (e__ != cudaSuccess) {                              \
            (void)cudaGetLastError();                          \
            return e__ == cudaErrorMemoryAllocation ? WAR_ERR_OOM : WAR_ERR_CUDA; \
        }                                                      \
    } while (0)

#define WAR_LAUNCH_CHECK()                                     \
    do {                                                       \
        cudaError_t e__ = cudaGetLastError();                  \
        if (e__ != cudaSuccess) return WAR_ERR_CUDA;           \
    } while (0)

static inline int64_t war_ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Shared host/device helpers of the PODS CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/pods.h"

#define PODS_FULL_MASK 0xffffffffu

#define PODS_RETURN_IF_CUDA_ERROR(expr)              \
    do {                                             \
        cudaError_t err__ = (expr);                  \
        if (err__ != cudaSuccess) return PODS_ERR_CUDA; \
    } while (0)

static inline cudaStream_t pods_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

static inline bool pods_aligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0;
}

// Number of SMs of the current device (148 on B200); queried per call, it is cheap.
static inline int pods_sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
    return sms;
}

__device__ __forceinline__ void pods_raise(uint32_t* status, uint32_t bit) {
    if (status != nullptr) atomicOr(status, bit);
}

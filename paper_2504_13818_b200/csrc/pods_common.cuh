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

// Checked build (-DPODS_BOUNDS_CHECK, a separate library used by the tests in place of a memory checker): an index
// that the kernels compute is compared with the extent it must stay inside; a violation ORs PODS_STATUS_INTERNAL
// into the status word and the access is skipped - never a trap.  In the normal build the test is the constant
// true and costs nothing.
#ifdef PODS_BOUNDS_CHECK
__device__ __forceinline__ bool pods_index_ok(long long i, long long extent, uint32_t* status) {
    if (i >= 0 && i < extent) return true;
    pods_raise(status, PODS_STATUS_INTERNAL);
    return false;
}
#define PODS_INDEX_OK(i, extent, status) pods_index_ok((long long)(i), (long long)(extent), (status))
// the index itself if it is inside its extent, else 0 (with the bit raised): for loads whose value feeds warp-wide
// operations, where skipping is not an option
#define PODS_CLAMPED(i, extent, status) (pods_index_ok((long long)(i), (long long)(extent), (status)) ? (i) : 0)
#else
#define PODS_INDEX_OK(i, extent, status) true
#define PODS_CLAMPED(i, extent, status) (i)
#endif

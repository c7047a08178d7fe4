// Library-level entry points: version, status strings, status read-back.

#include "pods_common.cuh"

extern "C" const char* pods_version(void) { return "pods-b200 0.1.0 (sm_100a)"; }

extern "C" const char* pods_status_string(int status) {
    switch (status) {
        case PODS_OK: return "ok";
        case PODS_ERR_INVALID_ARG: return "invalid argument";
        case PODS_ERR_UNSUPPORTED: return "unsupported size or rule";
        case PODS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case PODS_ERR_CUDA: return "CUDA runtime error";
        case PODS_ERR_STATIC_CAPACITY: return "chunk has more rows than the built-in scratch array holds";
        default: return "unknown status";
    }
}

extern "C" int pods_read_status(const uint32_t* status, uint32_t* host_value, void* stream) {
    if (status == nullptr || host_value == nullptr) return PODS_ERR_INVALID_ARG;
    cudaStream_t s = pods_stream(stream);
    PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(host_value, status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    PODS_RETURN_IF_CUDA_ERROR(cudaStreamSynchronize(s));
    return PODS_OK;
}

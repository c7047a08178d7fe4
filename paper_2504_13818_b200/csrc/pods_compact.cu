// pods_compact: concatenate the kept rollouts of every prompt group (text after Algorithm 1).
//   scan kernel   - exclusive prefix sums of the kept rollouts' lengths -> cu_seqlens [M+1]
//   gather kernel - copy each kept rollout's token ids and per-token fp32 streams from the
//                   padded all-rollouts storage to their packed position
// grpo_seq_weights: the 1/(M |o_i|) factors of L_PODS (Section 3.2).

#include "pods_common.cuh"

namespace {

constexpr int kScanThreads = 1024;
constexpr int kMaxStreams = 4;

struct StreamPtrs {
    const float* src[kMaxStreams];
    float* dst[kMaxStreams];
};

// idx[i] as a rollout number of its group: a value outside [0, n) (the caller handed over something that is not
// pods_select's output) raises PODS_STATUS_INDEX_RANGE and is read as rollout 0, so that no address leaves the storage.
__device__ __forceinline__ int32_t kept_rollout(const int32_t* idx, int64_t i, int n, uint32_t* status) {
    const int32_t j = idx[i];
    if (j >= 0 && j < n) return j;
    pods_raise(status, PODS_STATUS_INDEX_RANGE);
    return 0;
}

// One CTA walks the M kept rollouts in tiles of 1024, carrying the running total: M is the number
// of kept rollouts of a training batch (hundreds to thousands), far too few to need a
// multi-CTA scan.
__global__ void __launch_bounds__(kScanThreads)
compact_scan_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ lengths, int64_t M, int n,
                    int m, int64_t src_ld, int64_t* __restrict__ cu_seqlens, uint32_t* status) {
    __shared__ int64_t warp_tot[32];
    __shared__ int64_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int64_t tile = 0; tile < M; tile += kScanThreads) {
        const int64_t i = tile + tid;
        int64_t len = 0;
        if (i < M) {
            const int64_t g = i / m;
            int32_t l = lengths[g * n + kept_rollout(idx, i, n, status)];
            if (l < 0) { l = 0; pods_raise(status, PODS_STATUS_NEG_LENGTH); }
            if (l > src_ld) { l = (int32_t)src_ld; pods_raise(status, PODS_STATUS_CAPACITY); }   // longer than its storage row
            len = l;
        }
        int64_t inc = len;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int64_t t = __shfl_up_sync(PODS_FULL_MASK, inc, d);
            if (lane >= d) inc += t;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            int64_t w = warp_tot[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int64_t t = __shfl_up_sync(PODS_FULL_MASK, w, d);
                if (lane >= d) w += t;
            }
            warp_tot[lane] = w;                      // inclusive over warps
        }
        __syncthreads();
        const int64_t carry = carry_s;
        const int64_t before = carry + (warp > 0 ? warp_tot[warp - 1] : 0) + inc - len;
        if (i < M) cu_seqlens[i] = before;
        __syncthreads();
        if (tid == kScanThreads - 1) carry_s = carry + warp_tot[31];
        __syncthreads();
    }
    if (tid == 0) cu_seqlens[M] = carry_s;
}

// One CTA per kept rollout.
__global__ void __launch_bounds__(256)
compact_gather_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ lengths, int n, int m,
                      const int32_t* __restrict__ src_tokens, int64_t src_ld, StreamPtrs streams, int n_f32,
                      const int64_t* __restrict__ cu_seqlens, int32_t* __restrict__ dst_tokens, int64_t T_cap,
                      uint32_t* status) {
    const int64_t i = blockIdx.x;
    const int64_t g = i / m;
    const int64_t row = g * n + kept_rollout(idx, i, n, nullptr);     // the scan kernel has raised the bit already
    const int64_t begin = cu_seqlens[i];
    int64_t len = cu_seqlens[i + 1] - begin;
    if (begin + len > T_cap) {
        if (threadIdx.x == 0) pods_raise(status, PODS_STATUS_CAPACITY);
        len = T_cap > begin ? T_cap - begin : 0;
    }
    const int32_t* st = src_tokens + row * src_ld;
    for (int64_t t = threadIdx.x; t < len; t += blockDim.x)
        if (PODS_INDEX_OK(begin + t, T_cap, status) && PODS_INDEX_OK(t, src_ld, status)) dst_tokens[begin + t] = st[t];
    for (int s = 0; s < n_f32; ++s) {
        const float* sp = streams.src[s] + row * src_ld;
        float* dp = streams.dst[s] + begin;
        for (int64_t t = threadIdx.x; t < len; t += blockDim.x)
            if (PODS_INDEX_OK(begin + t, T_cap, status) && PODS_INDEX_OK(t, src_ld, status)) dp[t] = sp[t];
    }
    (void)lengths;
}

// One warp per kept rollout: |o_i| = number of unmasked tokens.
__global__ void __launch_bounds__(128)
seq_weights_kernel(const uint8_t* __restrict__ mask, const int64_t* __restrict__ cu_seqlens, int64_t M,
                   double* __restrict__ seq_weight) {
    const int64_t i = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (i >= M) return;
    const int64_t b = cu_seqlens[i], e = cu_seqlens[i + 1];
    int64_t count = 0;
    if (mask == nullptr) {
        count = e - b;
    } else {
        int c = 0;
        for (int64_t t = b + lane; t < e; t += 32) c += mask[t] ? 1 : 0;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(PODS_FULL_MASK, c, d);
        count = c;
    }
    if (lane == 0) seq_weight[i] = count > 0 ? 1.0 / ((double)M * (double)count) : 0.0;
}

}  // namespace

extern "C" int pods_compact(const int32_t* idx, int64_t G, int32_t n, int32_t m, const int32_t* lengths,
                            const int32_t* src_tokens, int64_t src_ld, const float* const* src_f32,
                            int32_t n_f32, int64_t* cu_seqlens, int32_t* dst_tokens, float* const* dst_f32,
                            int64_t T_cap, uint32_t* status, void* stream) {
    if (G < 0 || n < 1 || m < 1 || m > n || src_ld < 0 || T_cap < 0) return PODS_ERR_INVALID_ARG;
    if (n_f32 < 0 || n_f32 > kMaxStreams) return PODS_ERR_INVALID_ARG;
    if (cu_seqlens == nullptr || !pods_aligned(cu_seqlens, 8)) return PODS_ERR_INVALID_ARG;
    const int64_t M = G * (int64_t)m;
    if (M > 0x7fffffff) return PODS_ERR_UNSUPPORTED;
    if (M > 0 && (idx == nullptr || lengths == nullptr || src_tokens == nullptr || dst_tokens == nullptr))
        return PODS_ERR_INVALID_ARG;
    if (n_f32 > 0 && (src_f32 == nullptr || dst_f32 == nullptr)) return PODS_ERR_INVALID_ARG;
    StreamPtrs sp = {};
    for (int s = 0; s < n_f32; ++s) {
        if (src_f32[s] == nullptr || dst_f32[s] == nullptr) return PODS_ERR_INVALID_ARG;
        sp.src[s] = src_f32[s];
        sp.dst[s] = dst_f32[s];
    }
    cudaStream_t s = pods_stream(stream);
    compact_scan_kernel<<<1, kScanThreads, 0, s>>>(idx, lengths, M, n, m, src_ld, cu_seqlens, status);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    if (M > 0) {
        compact_gather_kernel<<<(unsigned)M, 256, 0, s>>>(idx, lengths, n, m, src_tokens, src_ld, sp, n_f32,
                                                          cu_seqlens, dst_tokens, T_cap, status);
        PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    }
    return PODS_OK;
}

extern "C" int grpo_seq_weights(const uint8_t* mask, const int64_t* cu_seqlens, int64_t M, double* seq_weight,
                                void* stream) {
    if (M < 0) return PODS_ERR_INVALID_ARG;
    if (M == 0) return PODS_OK;
    if (cu_seqlens == nullptr || seq_weight == nullptr) return PODS_ERR_INVALID_ARG;
    if (!pods_aligned(cu_seqlens, 8) || !pods_aligned(seq_weight, 8)) return PODS_ERR_INVALID_ARG;
    const int64_t blocks = (M + 3) / 4;
    if (blocks > 0x7fffffff) return PODS_ERR_UNSUPPORTED;
    seq_weights_kernel<<<(unsigned)blocks, 128, 0, pods_stream(stream)>>>(mask, cu_seqlens, M, seq_weight);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

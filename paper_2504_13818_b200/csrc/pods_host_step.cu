// pods_host_step: one whole step of the hot path for callers whose data lives in HOST memory:
// rewards and rollout storage in, loss / log-probs / kept indices out, the gradient left on the
// device.  The object owns its device buffers and two streams; the bf16 logits, by far the
// largest input, are uploaded in row chunks through two staging buffers so that the copy of chunk
// c+1 overlaps the loss kernel of chunk c.
//
//   copy stream     H2D chunk 0 | H2D chunk 1 | H2D chunk 2 | ...
//   compute stream  select, compact | loss chunk 0 | loss chunk 1 | ...
//
// Step order and arithmetic are exactly those of the device-pointer entry points, which this file
// only calls: pods_select -> pods_compact -> grpo_seq_weights -> grpo_loss_chunk per chunk ->
// grpo_loss_finalize.

#include <new>

#include "pods_common.cuh"

struct pods_host_step {
    int64_t G, src_ld, T_cap, chunk_rows;
    int32_t n, m, V;
    int64_t M, R;                       // kept rollouts, all rollouts
    int device;
    cudaStream_t compute, copy;
    cudaEvent_t loaded[2], released[2];
    // device buffers
    float* rewards;
    int32_t *lengths, *src_tokens, *idx, *k, *tokens;
    float *src_old, *src_ref, *adv, *old_logp, *ref_logp, *logp, *loss;
    int64_t* cu_seqlens;
    double *seq_weight, *loss_acc;
    uint32_t* status;
    uint16_t* stage[2];                 // [chunk_rows, V] bf16 each
    uint16_t* dlogits;                  // [T_cap, V] bf16
    void* workspace;
    size_t workspace_bytes;
};

namespace {

template <typename T>
bool dev_alloc(T** p, size_t count) {
    *p = nullptr;
    return cudaMalloc(reinterpret_cast<void**>(p), (count ? count : 1) * sizeof(T)) == cudaSuccess;
}

void release(pods_host_step* h) {
    if (h == nullptr) return;
    void* bufs[] = {h->rewards, h->lengths, h->src_tokens, h->idx, h->k, h->tokens, h->src_old, h->src_ref, h->adv,
                    h->old_logp, h->ref_logp, h->logp, h->loss, h->cu_seqlens, h->seq_weight, h->loss_acc, h->status,
                    h->stage[0], h->stage[1], h->dlogits, h->workspace};
    for (void* b : bufs)
        if (b != nullptr) cudaFree(b);
    for (int i = 0; i < 2; ++i) {
        if (h->loaded[i]) cudaEventDestroy(h->loaded[i]);
        if (h->released[i]) cudaEventDestroy(h->released[i]);
    }
    if (h->compute) cudaStreamDestroy(h->compute);
    if (h->copy) cudaStreamDestroy(h->copy);
    delete h;
}

}  // namespace

extern "C" int pods_host_step_create(int64_t G, int32_t n, int32_t m, int64_t src_ld, int64_t T_cap, int32_t V,
                                     int64_t chunk_rows, pods_host_step** out) {
    if (out == nullptr) return PODS_ERR_INVALID_ARG;
    *out = nullptr;
    if (G < 1 || n < 1 || m < 1 || m > n || src_ld < 1 || T_cap < 1 || V < 1 || chunk_rows < 1) return PODS_ERR_INVALID_ARG;
    if (n > PODS_MAX_N || V % 8 != 0) return PODS_ERR_UNSUPPORTED;      // staged rows are packed: 16-byte aligned only if V % 8 == 0
    pods_host_step* h = new (std::nothrow) pods_host_step();
    if (h == nullptr) return PODS_ERR_CUDA;
    h->G = G; h->n = n; h->m = m; h->src_ld = src_ld; h->T_cap = T_cap; h->V = V;
    h->chunk_rows = chunk_rows < T_cap ? chunk_rows : T_cap;
    h->M = G * (int64_t)m;
    h->R = G * (int64_t)n;
    bool ok = cudaGetDevice(&h->device) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&h->compute, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&h->copy, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i) {
        ok = ok && cudaEventCreateWithFlags(&h->loaded[i], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&h->released[i], cudaEventDisableTiming) == cudaSuccess;
    }
    h->workspace_bytes = grpo_loss_chunk_workspace_bytes(h->chunk_rows);
    ok = ok && dev_alloc(&h->rewards, (size_t)h->R) && dev_alloc(&h->lengths, (size_t)h->R) &&
         dev_alloc(&h->src_tokens, (size_t)(h->R * src_ld)) && dev_alloc(&h->src_old, (size_t)(h->R * src_ld)) &&
         dev_alloc(&h->src_ref, (size_t)(h->R * src_ld)) && dev_alloc(&h->idx, (size_t)h->M) &&
         dev_alloc(&h->k, (size_t)G) && dev_alloc(&h->adv, (size_t)h->M) && dev_alloc(&h->tokens, (size_t)T_cap) &&
         dev_alloc(&h->old_logp, (size_t)T_cap) && dev_alloc(&h->ref_logp, (size_t)T_cap) &&
         dev_alloc(&h->logp, (size_t)T_cap) && dev_alloc(&h->loss, 1) && dev_alloc(&h->cu_seqlens, (size_t)h->M + 1) &&
         dev_alloc(&h->seq_weight, (size_t)h->M) && dev_alloc(&h->loss_acc, 1) && dev_alloc(&h->status, 1) &&
         dev_alloc(&h->stage[0], (size_t)(h->chunk_rows * V)) && dev_alloc(&h->stage[1], (size_t)(h->chunk_rows * V)) &&
         dev_alloc(&h->dlogits, (size_t)(T_cap * V)) &&
         cudaMalloc(&h->workspace, h->workspace_bytes) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        release(h);
        return PODS_ERR_CUDA;
    }
    *out = h;
    return PODS_OK;
}

extern "C" int pods_host_step_destroy(pods_host_step* h) {
    if (h == nullptr) return PODS_OK;
    cudaStreamSynchronize(h->compute);
    cudaStreamSynchronize(h->copy);
    release(h);
    return PODS_OK;
}

extern "C" void* pods_host_step_dlogits(pods_host_step* h) { return h ? h->dlogits : nullptr; }

extern "C" int pods_host_step_run(pods_host_step* h, const float* rewards, const int32_t* lengths,
                                  const int32_t* src_tokens, const float* src_old, const float* src_ref,
                                  const void* logits, int64_t T_logits, float eps, float beta, int32_t rule,
                                  uint64_t seed, uint32_t flags, float* loss_out, float* logp_out, int32_t* idx_out,
                                  float* adv_out, int64_t* T_out, uint32_t* status_out) {
    if (h == nullptr || rewards == nullptr || lengths == nullptr || src_tokens == nullptr || src_old == nullptr ||
        logits == nullptr || loss_out == nullptr)
        return PODS_ERR_INVALID_ARG;
    if (src_ref == nullptr && beta != 0.0f) return PODS_ERR_INVALID_ARG;
    if (T_logits < 0 || T_logits > h->T_cap) return PODS_ERR_INVALID_ARG;
    const cudaStream_t cs = h->compute;
    const size_t rollouts = (size_t)h->R, padded = (size_t)(h->R * h->src_ld);

    // ---- small inputs up, selection and compaction ----------------------------------------------
    PODS_RETURN_IF_CUDA_ERROR(cudaMemsetAsync(h->status, 0, sizeof(uint32_t), cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaMemsetAsync(h->loss_acc, 0, sizeof(double), cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(h->rewards, rewards, rollouts * sizeof(float), cudaMemcpyHostToDevice, cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(h->lengths, lengths, rollouts * sizeof(int32_t), cudaMemcpyHostToDevice, cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(h->src_tokens, src_tokens, padded * sizeof(int32_t), cudaMemcpyHostToDevice, cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(h->src_old, src_old, padded * sizeof(float), cudaMemcpyHostToDevice, cs));
    if (src_ref != nullptr)
        PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(h->src_ref, src_ref, padded * sizeof(float), cudaMemcpyHostToDevice, cs));
    int rc = pods_select(h->rewards, h->G, h->n, h->m, rule, seed, flags, h->idx, h->adv, h->k, h->status, cs);
    if (rc != PODS_OK) return rc;
    const float* src_streams[2] = {h->src_old, h->src_ref};
    float* dst_streams[2] = {h->old_logp, h->ref_logp};
    rc = pods_compact(h->idx, h->G, h->n, h->m, h->lengths, h->src_tokens, h->src_ld, src_streams,
                      src_ref != nullptr ? 2 : 1, h->cu_seqlens, h->tokens, dst_streams, h->T_cap, h->status, cs);
    if (rc != PODS_OK) return rc;
    int64_t T = 0;
    PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(&T, h->cu_seqlens + h->M, sizeof(int64_t), cudaMemcpyDeviceToHost, cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaStreamSynchronize(cs));
    if (T_out != nullptr) *T_out = T;
    if (T != T_logits) return PODS_ERR_INVALID_ARG;      // the caller's logits are not those of the kept rollouts
    rc = grpo_seq_weights(nullptr, h->cu_seqlens, h->M, h->seq_weight, cs);
    if (rc != PODS_OK) return rc;

    // ---- logits up in chunks through two staging buffers, the loss kernel behind them --------------
    const uint16_t* lg = static_cast<const uint16_t*>(logits);
    int64_t c = 0;
    for (int64_t r0 = 0; r0 < T; r0 += h->chunk_rows, ++c) {
        const int b = (int)(c & 1);
        const int64_t rows = T - r0 < h->chunk_rows ? T - r0 : h->chunk_rows;
        if (c >= 2) PODS_RETURN_IF_CUDA_ERROR(cudaStreamWaitEvent(h->copy, h->released[b], 0));
        PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(h->stage[b], lg + r0 * h->V, (size_t)(rows * h->V) * sizeof(uint16_t),
                                                  cudaMemcpyHostToDevice, h->copy));
        PODS_RETURN_IF_CUDA_ERROR(cudaEventRecord(h->loaded[b], h->copy));
        PODS_RETURN_IF_CUDA_ERROR(cudaStreamWaitEvent(cs, h->loaded[b], 0));
        rc = grpo_loss_chunk(h->stage[b], h->V, h->tokens + r0, h->old_logp + r0,
                             src_ref != nullptr ? h->ref_logp + r0 : nullptr, h->adv, h->seq_weight, h->cu_seqlens,
                             h->M, r0, nullptr, rows, h->V, eps, beta, 1.0f, h->loss_acc, h->logp + r0,
                             h->dlogits + r0 * h->V, h->V, h->workspace, h->workspace_bytes, h->status, cs);
        if (rc != PODS_OK) return rc;
        PODS_RETURN_IF_CUDA_ERROR(cudaEventRecord(h->released[b], cs));
    }
    rc = grpo_loss_finalize(h->loss_acc, h->loss, cs);
    if (rc != PODS_OK) return rc;

    // ---- results down ---------------------------------------------------------------------------
    PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(loss_out, h->loss, sizeof(float), cudaMemcpyDeviceToHost, cs));
    if (logp_out != nullptr && T > 0)
        PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(logp_out, h->logp, (size_t)T * sizeof(float), cudaMemcpyDeviceToHost, cs));
    if (idx_out != nullptr)
        PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(idx_out, h->idx, (size_t)h->M * sizeof(int32_t), cudaMemcpyDeviceToHost, cs));
    if (adv_out != nullptr)
        PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(adv_out, h->adv, (size_t)h->M * sizeof(float), cudaMemcpyDeviceToHost, cs));
    if (status_out != nullptr)
        PODS_RETURN_IF_CUDA_ERROR(cudaMemcpyAsync(status_out, h->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaStreamSynchronize(cs));
    PODS_RETURN_IF_CUDA_ERROR(cudaStreamSynchronize(h->copy));
    return PODS_OK;
}

// grpo_logp_from_hidden: log pi_theta(o_t | p, o_<t) (the policy term of L_GRPO, Section 3.1, and L_PODS,
// Section 3.2) straight from the last hidden states, for the passes that need no gradient (the frozen
// sampling policy's old_logp, the reference policy's ref_logp): logits = hidden W^T are formed tile by tile
// on the tensor cores and reduced to the row's softmax statistics on the spot, so the [T,V] logits never
// reach HBM.
//
// Kernel 1, lm_head_stats_kernel (persistent, one CTA per SM, six warps):
//   warp 0   producer: TMA tile loads (cp.async.bulk.tensor, 128-byte swizzle, no multicast) of a 128 x 64
//            block of hidden and a 256 x 64 block of W per stage into a ring of four stages;
//   warp 1   one thread issues tcgen05.mma (M = 128, N = 256, K = 16, bf16 in, fp32 accumulate) from shared
//            memory into one of two 256-column accumulators in tensor memory; tcgen05.commit releases the
//            stage, and after the last k-block hands the accumulator to the epilogue;
//   warps 2-5  epilogue: thread r of the four warps owns row r of the tile (a TMEM lane): it reads its 256
//            logits with tcgen05.ld, 32 columns at a time, and folds them into a running (maximum, sum of
//            exponentials) pair in base 2; no thread ever needs another thread's values.
//   The vocabulary is cut into parts of a few tiles; a work item is (part, block of 128 rows), items are
//   dealt out part-major so that the CTAs running at the same time read the same rows of W (from L2).
//   At the end of an item the 128 pairs go to the workspace.  While the epilogue reduces one accumulator the
//   tensor core fills the other.
// Kernel 2, lm_head_merge_kernel: one warp per row merges the parts' pairs into the log-sum-exp, takes the
//   target's logit as the dot product hidden[t] . W[token] (fp32) and writes logp (and the lse).
//
// Every wait on an mbarrier is bounded; a wait that runs out raises PODS_STATUS_TIMEOUT, and the roles carry
// on to the end of their loops (arriving wherever they owe an arrival) so that the CTA ends and frees its
// tensor memory.

#include "lm_head_common.cuh"

using namespace pods_lm;

namespace {

struct StatsArgs {
    int64_t T;
    int32_t V, d;
    int32_t n_row_blocks;        // ceil(T / 128)
    int32_t n_col_tiles;         // ceil(V / 256)
    int32_t tiles_per_part;
    int32_t n_parts;
    int64_t n_items;             // n_parts * n_row_blocks, part-major
    float2* partial;             // [n_parts][n_row_blocks * 128]: (maximum of x log2e, sum of 2^(x log2e - maximum))
    uint32_t* status;
};

__global__ void __launch_bounds__(kThreads, 1)
lm_head_stats_kernel(const __grid_constant__ CUtensorMap map_hidden, const __grid_constant__ CUtensorMap map_w,
                     const StatsArgs a) {
    extern __shared__ unsigned char smem_raw[];
    // the swizzled tiles want 1024-byte aligned stages
    unsigned char* const tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Barriers& bar = *reinterpret_cast<Barriers*>(tiles + (size_t)kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_blocks = (a.d + BK - 1) / BK;

    const uint32_t tmem_base = pipeline_setup(bar, warp);
    bool timed_out = false;

    if (warp == 0) {
        // =============================== producer ===============================
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int64_t loads = 0;
            for (int64_t item = blockIdx.x; item < a.n_items; item += gridDim.x) {
                const int part = (int)(item / a.n_row_blocks), rb = (int)(item % a.n_row_blocks);
                const int t0 = part * a.tiles_per_part, t1 = min(a.n_col_tiles, t0 + a.tiles_per_part);
                for (int ct = t0; ct < t1; ++ct) {
                    for (int kb = 0; kb < k_blocks; ++kb) {
                        if (!mbar_wait(&bar.empty[stage], phase ^ 1u, timed_out)) timed_out = true;
                        unsigned char* sa = tiles + (size_t)stage * kStageBytes;
                        mbar_expect_tx(&bar.full[stage], kStageBytes);
                        tma_load_tile(sa, &map_hidden, kb * BK, rb * BM, &bar.full[stage]);
                        tma_load_tile(sa + kStageBytesA, &map_w, kb * BK, ct * BN, &bar.full[stage]);
                        ++loads;
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (!drain_loads(bar, loads)) timed_out = true;
        }
        __syncwarp();
    } else if (warp == 1) {
        // =============================== tensor-core issuer ===============================
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            for (int64_t item = blockIdx.x; item < a.n_items; item += gridDim.x) {
                const int part = (int)(item / a.n_row_blocks);
                const int t0 = part * a.tiles_per_part, t1 = min(a.n_col_tiles, t0 + a.tiles_per_part);
                for (int ct = t0; ct < t1; ++ct) {
                    if (!mbar_wait(&bar.acc_empty[acc], acc_phase ^ 1u, timed_out)) timed_out = true;
                    tcgen05_fence_after();
                    const uint32_t tmem_acc = tmem_base + (uint32_t)(acc * BN);
                    for (int kb = 0; kb < k_blocks; ++kb) {
                        if (!mbar_wait(&bar.full[stage], phase, timed_out)) timed_out = true;
                        tcgen05_fence_after();
                        const uint32_t sa = smem_u32(tiles + (size_t)stage * kStageBytes);
                        const uint64_t da = smem_desc_k_major(sa), db = smem_desc_k_major(sa + kStageBytesA);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k)      // 16 features = 32 bytes further along the rows
                            umma(tmem_acc, da + (uint64_t)(k * UMMA_K * 2 >> 4), db + (uint64_t)(k * UMMA_K * 2 >> 4),
                                 instr_desc(false, false), (kb | k) != 0 ? 1u : 0u);
                        umma_commit(&bar.empty[stage]);
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    umma_commit(&bar.acc_full[acc]);
                    if (++acc == kAccumulators) { acc = 0; acc_phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else {
        // =============================== epilogue: one row per thread ===============================
        const int quarter = warp & 3;                           // the TMEM lanes a warp may read: 32 (warp % 4) ..
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int64_t item = blockIdx.x; item < a.n_items; item += gridDim.x) {
            const int part = (int)(item / a.n_row_blocks), rb = (int)(item % a.n_row_blocks);
            const int t0 = part * a.tiles_per_part, t1 = min(a.n_col_tiles, t0 + a.tiles_per_part);
            float m_run = -INFINITY, s_run = 0.0f;              // maximum of y = x log2e so far; sum of 2^(y - m_run)
            for (int ct = t0; ct < t1; ++ct) {
                if (!mbar_wait(&bar.acc_full[acc], acc_phase, timed_out)) timed_out = true;
                tcgen05_fence_after();
                const int valid_cols = min(BN, a.V - ct * BN);  // columns past the vocabulary hold 0 W 's products
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    float v[32];
                    tmem_load_32(tmem_base + lane_addr + (uint32_t)(acc * BN + c0), v);
                    if (c0 + 32 > valid_cols) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = (c0 + i < valid_cols) ? v[i] : -INFINITY;
                    }
                    float cm = v[0];
#pragma unroll
                    for (int i = 1; i < 32; ++i) cm = fmaxf(cm, v[i]);
                    const float m_new = fmaxf(m_run, cm * kLog2e);
                    if (m_new != -INFINITY) {
                        float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            s0 += ex2(fmaf(v[i], kLog2e, -m_new));
                            s1 += ex2(fmaf(v[i + 1], kLog2e, -m_new));
                            s2 += ex2(fmaf(v[i + 2], kLog2e, -m_new));
                            s3 += ex2(fmaf(v[i + 3], kLog2e, -m_new));
                        }
                        s_run = s_run * ex2(m_run - m_new) + ((s0 + s1) + (s2 + s3));
                        m_run = m_new;
                    }
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar.acc_empty[acc]);
                if (++acc == kAccumulators) { acc = 0; acc_phase ^= 1u; }
            }
            const size_t slot = (size_t)part * ((size_t)a.n_row_blocks * BM) + (size_t)rb * BM + row_in_tile;
            if (PODS_INDEX_OK(slot, (size_t)a.n_parts * a.n_row_blocks * BM, a.status)) a.partial[slot] = make_float2(m_run, s_run);
        }
    }
    if (timed_out && lane == 0) pods_raise(a.status, PODS_STATUS_TIMEOUT);
    pipeline_teardown(tmem_base, warp);
}

// One warp per row: the parts' (maximum, sum) pairs -> log-sum-exp; the target's logit; logp.
__global__ void __launch_bounds__(256)
lm_head_merge_kernel(const uint16_t* __restrict__ hidden, int64_t ldh, const uint16_t* __restrict__ W, int64_t ldw,
                     const int32_t* __restrict__ tokens, int64_t T, int32_t V, int32_t d, const float2* __restrict__ partial,
                     int32_t n_parts, int64_t rows_padded, float* __restrict__ logp, float* __restrict__ lse_out,
                     uint32_t* status) {
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    int tok = tokens[t];
    if (tok < 0 || tok >= V) { tok = 0; if (lane == 0) pods_raise(status, PODS_STATUS_TOKEN_RANGE); }
    double lse;
    float x_tok;
    merge_row(hidden, ldh, W, ldw, t, tok, d, partial, n_parts, rows_padded, lane, &lse, &x_tok);
    if (lane == 0) {
        logp[t] = (float)((double)x_tok - lse);
        if (lse_out != nullptr) lse_out[t] = (float)lse;
    }
}

}  // namespace

int pods_lm::launch_lm_head_stats(const void* hidden, int64_t ldh, const void* W, int64_t ldw, int64_t T, int32_t V,
                                  int32_t d, const Plan& plan, float2* partial, uint32_t* status, cudaStream_t s) {
    CUtensorMap map_h, map_w;
    int rc = make_map(&map_h, hidden, T, d, ldh, BM);
    if (rc != PODS_OK) return rc;
    rc = make_map(&map_w, W, V, d, ldw, BN);
    if (rc != PODS_OK) return rc;
    StatsArgs a;
    a.T = T;
    a.V = V;
    a.d = d;
    a.n_row_blocks = plan.n_row_blocks;
    a.n_col_tiles = plan.n_col_tiles;
    a.tiles_per_part = plan.tiles_per_part;
    a.n_parts = plan.n_parts;
    a.n_items = (int64_t)plan.n_parts * plan.n_row_blocks;
    a.partial = partial;
    a.status = status;
    PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(lm_head_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    lm_head_stats_kernel<<<plan.grid, kThreads, kSmemBytes, s>>>(map_h, map_w, a);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

extern "C" size_t grpo_logp_from_hidden_workspace_bytes(int64_t T, int32_t V, int32_t d) {
    (void)d;
    if (T <= 0 || V <= 0) return 0;
    // one (maximum, sum) pair per row and part of the vocabulary; the parts follow from the current device's SM count
    const Plan plan = make_plan(T, V, pods_sm_count());
    return align_up((size_t)plan.n_parts * (size_t)plan.n_row_blocks * BM * sizeof(float2), 256);
}

extern "C" int grpo_logp_from_hidden(const void* hidden, int64_t ldh, const void* W, int64_t ldw,
                                     const int32_t* tokens, int64_t T, int32_t V, int32_t d, float* logp,
                                     float* lse, void* workspace, size_t workspace_bytes, uint32_t* status,
                                     void* stream) {
    if (T < 0 || V < 1 || d < 8 || d % 8 != 0 || ldh < d || ldw < d || ldh % 8 != 0 || ldw % 8 != 0)
        return PODS_ERR_INVALID_ARG;
    if (T == 0) return PODS_OK;
    if (hidden == nullptr || W == nullptr || tokens == nullptr || logp == nullptr) return PODS_ERR_INVALID_ARG;
    if (!pods_aligned(hidden, 16) || !pods_aligned(W, 16) || !pods_aligned(logp, 4)) return PODS_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < grpo_logp_from_hidden_workspace_bytes(T, V, d) ||
        !pods_aligned(workspace, 16))
        return PODS_ERR_WORKSPACE;

    const Plan plan = make_plan(T, V, pods_sm_count());
    float2* partial = static_cast<float2*>(workspace);
    cudaStream_t s = pods_stream(stream);
    const int rc = launch_lm_head_stats(hidden, ldh, W, ldw, T, V, d, plan, partial, status, s);
    if (rc != PODS_OK) return rc;
    const int warps_per_block = 8;
    lm_head_merge_kernel<<<(unsigned)((T + warps_per_block - 1) / warps_per_block), warps_per_block * 32, 0, s>>>(
        static_cast<const uint16_t*>(hidden), ldh, static_cast<const uint16_t*>(W), ldw, tokens, T, V, d, partial,
        plan.n_parts, (int64_t)plan.n_row_blocks * BM, logp, lse, status);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

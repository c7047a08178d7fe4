// grpo_loss_from_hidden: L_PODS (Section 3.2) and its gradient when the logits are the LM-head projection
// hidden W^T, with the [T,V] logits and their gradient never stored in full: the gradient goes straight on to
// d loss / d hidden and d loss / d W.
//
// Per call (T rows of one chunk):
//   1. statistics pass (lm_head_logp.cu): logits tile by tile on the tensor cores -> per-row log-sum-exp;
//   2. lm_head_row_terms_kernel: log-prob, the token's loss term and its gradient factor g_t (fp64 scalars);
//   then, for one panel of the vocabulary after the other (a panel is as many 256-column tiles as keep the
//   panel's gradient block within a byte limit, 512 MB unless changed):
//   3. lm_head_dlogits_kernel: the panel's logits AGAIN on the tensor cores (same pipeline as pass 1), and in the
//      epilogue dlogits = g_t ([v == token] - 2^(x log2e - lse log2e)) rounded to bf16 into the panel buffer
//      [rows, panel columns] - the only place a piece of the [T,V] gradient ever exists;
//   4. lm_head_grad_gemm_pair_kernel<false>: dhidden[T,d] (+)= panel[T, cols] . W[cols, d]
//   5. lm_head_grad_gemm_pair_kernel<true>:  dW[cols, d] += panel^T[cols, T] . hidden[T, d]
//      both with tcgen05.mma reading the operands whose contraction index is NOT contiguous in memory (W and hidden
//      by rows of d, the panel by rows of vocabulary entries for step 5) as MN-major shared-memory tiles, so
//      no transposed copy of anything is made.
// Roles, barriers and bounded waits are those of the statistics kernel: a TMA producer warp, one thread issuing
// the MMAs into one of two 256-column accumulators in tensor memory, four epilogue warps (one tile row per
// thread; eight warps, half a row per thread, where the epilogue forms the gradient).  Kernels 3-5 run as PAIRS of
// CTAs (cta_group::2): a pair shares one 256 x 256 tile, each CTA loading its rows of A and half of B, which cuts the
// bytes a CTA takes from L2 per contraction block from 48 KB to 32 KB and deepens the ring from four to six stages.
// All loads are plain (never multicast) TMA loads of this GPU's own memory into the loading CTA's own shared memory.

#include "grpo_loss_common.cuh"
#include "lm_head_common.cuh"

using namespace pods_lm;

namespace {

// Upper limit of the gradient panel (rows x panel columns, bf16); pods_set_loss_from_hidden_panel_bytes moves it.
size_t g_panel_bytes = (size_t)512 << 20;

// What the gradient epilogue needs of a row: 16 bytes.
struct __align__(16) RowGrad {
    float g;             // grad_scale mask_t w_i dloss/dlogp
    float lse2;          // log-sum-exp of the row times log2(e)
    int token;           // in [0, V)
    float g_token;       // g (1 - p_token), formed in fp64: the target's own gradient entry
};

// ------------------------------------------------------------------------------------------------------
// Step 2: one warp per row.  Rows beyond T (padding of the last 128-row block) get a zero record.
// ------------------------------------------------------------------------------------------------------
struct TermsArgs {
    const uint16_t* hidden;
    int64_t ldh;
    const uint16_t* W;
    int64_t ldw;
    const float2* partial;
    int32_t n_parts;
    int64_t rows_padded;
    pods_loss::RowArgs row;      // tokens, old/ref log-probs, advantages, weights, mask, T, V, eps, beta, grad_scale, logp
    int32_t d;
    RowGrad* grad;               // [rows_padded]
};

__global__ void __launch_bounds__(256)
lm_head_row_terms_kernel(const TermsArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= a.rows_padded) return;
    if (t >= a.row.T) {
        if (lane == 0) a.grad[t] = RowGrad{0.0f, 0.0f, 0, 0.0f};
        return;
    }
    int tok = a.row.tokens[t];
    if (tok < 0 || tok >= a.row.V) { tok = 0; if (lane == 0) pods_raise(a.row.status, PODS_STATUS_TOKEN_RANGE); }
    double lse;
    float x_tok;
    merge_row(a.hidden, a.ldh, a.W, a.ldw, t, tok, a.d, a.partial, a.n_parts, a.rows_padded, lane, &lse, &x_tok);
    if (lane == 0) {
        const double logp = (double)x_tok - lse;
        const pods_loss::RowInputs in = pods_loss::load_row_inputs(a.row, t);
        const pods_loss::TokenTerms tt = pods_loss::token_terms(logp, in, a.row.eps, a.row.beta, a.row.grad_scale);
        a.row.logp[t] = (float)logp;
        a.row.row_loss[t] = tt.weighted_loss;
        RowGrad r;
        r.g = (float)tt.g;
        r.lse2 = (float)(lse * 1.4426950408889634);
        r.token = tok;
        r.g_token = (float)(tt.g * -expm1(logp));
        a.grad[t] = r;
    }
}

// ------------------------------------------------------------------------------------------------------
// Step 3: the panel's logits again, turned into the gradient with respect to the logits on the way out.
// ------------------------------------------------------------------------------------------------------
struct DlogitsArgs {
    int32_t V, d;
    int32_t n_row_blocks;        // PAIRS of 128-row blocks (what tile_of counts)
    int32_t n_blocks128;         // 128-row blocks: the panel and `grad` have n_blocks128 * 128 rows
    int32_t tile0;               // first 256-column tile of the panel, counted over the whole vocabulary
    int32_t n_col_tiles;         // tiles of this panel
    int32_t group_rows;          // row blocks per group of the tile order (see tile_of)
    int64_t n_items;             // tiles of the panel: column tiles x row blocks
    const RowGrad* grad;         // [n_blocks128 * 128]
    int64_t ldp;                 // row pitch of the panel (bf16 [n_blocks128 * 128, ldp]), >= n_col_tiles * 256
    uint32_t* status;
};

// Order of the panel's tiles: groups of `group_rows` blocks of rows; inside a group one column tile after the other,
// and for each the group's row blocks.  The CTAs that run at the same time (consecutive items) then share a few
// column tiles of W and the group's row blocks of hidden - 32 MB at 64 row blocks per group and d = 2048 - instead of
// sweeping all of hidden (67 MB at 16384 rows, more than one L2 partition holds) for every column tile, and the
// panel's rows of W cross HBM once per group (2 to 4 times per panel; 8 times with groups of 16 row blocks).
__device__ __forceinline__ void tile_of(const DlogitsArgs& a, int64_t item, int* ct, int* rb) {
    const int64_t per_group = (int64_t)a.group_rows * a.n_col_tiles;
    const int n_groups = (a.n_row_blocks + a.group_rows - 1) / a.group_rows;
    int g = (int)(item / per_group);
    if (g > n_groups - 1) g = n_groups - 1;
    const int64_t rem = item - (int64_t)g * per_group;
    const int rows_here = min(a.group_rows, a.n_row_blocks - g * a.group_rows);
    *ct = (int)(rem / rows_here);
    *rb = g * a.group_rows + (int)(rem % rows_here);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Eight epilogue warps here (two per quarter of the TMEM lanes, each taking half of the tile's columns): with four,
// a warp alone on its scheduler spent about 15 us per tile on the dependent chain load - exponentials - round - store,
// more than the 12 us the tensor core needs for the tile.
constexpr int kDlogitsThreads = 64 + 8 * 32;
// The gradient leaves through shared memory: a warp stages 32 rows x 64 columns (whole 128-byte lines) and one thread
// sends them off as one bulk tensor store.  Stored straight from registers (16 bytes per lane and instruction, every
// lane another line) the same data cost 1.5 ms of 7.7 per 16384 rows.
constexpr uint32_t kStagingBytesPerWarp = 32 * 128;
constexpr size_t kDlogitsSmemBytes = 1024 + (size_t)kPairStages * kPairStageBytes + 8 * kStagingBytesPerWarp + 256;

// CTA pairs (see lm_head_common.cuh): an item is a 256 x 256 tile of logits, CTA r of the pair holds rows 128 r ..
// of it and loads columns 128 r .. of W's tile; n_row_blocks, group_rows and tile_of count PAIRS of 128-row blocks.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kDlogitsThreads, 1)
lm_head_dlogits_kernel(const __grid_constant__ CUtensorMap map_hidden, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_panel, const DlogitsArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* const tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* const staging = tiles + (size_t)kPairStages * kPairStageBytes;    // 1024-byte aligned, 4 KB per warp
    PairBarriers& bar = *reinterpret_cast<PairBarriers*>(staging + 8 * kStagingBytesPerWarp);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_blocks = (a.d + BK - 1) / BK;
    const uint32_t rank = cluster_ctarank();
    const uint32_t tmem_base = pair_setup(bar, warp, 8);
    const int64_t first = blockIdx.x >> 1, stride = gridDim.x >> 1;
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int64_t loads = 0;
            for (int64_t item = first; item < a.n_items; item += stride) {
                int ct, rb;
                tile_of(a, item, &ct, &rb);
                {
                    for (int kb = 0; kb < k_blocks; ++kb) {
                        if (!mbar_wait(&bar.empty[stage], phase ^ 1u, timed_out)) timed_out = true;
                        unsigned char* sa = tiles + (size_t)stage * kPairStageBytes;
                        if (rank == 0) mbar_expect_tx(&bar.full[stage], 2 * kPairStageBytes);
                        tma_load_tile_pair(sa, &map_hidden, kb * BK, (2 * rb + (int)rank) * BM, &bar.full[stage]);
                        tma_load_tile_pair(sa + kPairStageBytesA, &map_w, kb * BK,
                                           (a.tile0 + ct) * BN + (int)rank * (BN / 2), &bar.full[stage]);
                        ++loads;
                        if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (rank == 0 && !drain_loads_pair(bar, loads)) timed_out = true;
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            for (int64_t item = first; item < a.n_items; item += stride) {
                {
                    if (!mbar_wait_cluster(&bar.acc_empty[acc], acc_phase ^ 1u, timed_out)) timed_out = true;
                    tcgen05_fence_after();
                    const uint32_t tmem_acc = tmem_base + (uint32_t)(acc * BN);
                    for (int kb = 0; kb < k_blocks; ++kb) {
                        if (!mbar_wait(&bar.full[stage], phase, timed_out)) timed_out = true;
                        tcgen05_fence_after();
                        const uint32_t sa = smem_u32(tiles + (size_t)stage * kPairStageBytes);
                        const uint64_t da = smem_desc_k_major(sa), db = smem_desc_k_major(sa + kPairStageBytesA);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k)
                            umma_pair(tmem_acc, da + (uint64_t)(k * UMMA_K * 2 >> 4), db + (uint64_t)(k * UMMA_K * 2 >> 4),
                                      instr_desc_pair(false, false), (kb | k) != 0 ? 1u : 0u);
                        umma_commit_pair(&bar.empty[stage]);
                        if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                    }
                    umma_commit_pair(&bar.acc_full[acc]);
                    if (++acc == kAccumulators) { acc = 0; acc_phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else {
        // epilogue: warps 2-9; a warp reads the TMEM lanes of its quarter (warp % 4) and one half of the columns
        const int quarter = warp & 3;
        const int col_begin = ((warp - 2) >> 2) * (BN / 2);
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        unsigned char* const stage_warp = staging + (size_t)(warp - 2) * kStagingBytesPerWarp;   // 32 lines of 128 bytes
        unsigned char* const stage_line = stage_warp + lane * 128;
        const uint64_t stream_policy = l2_policy_evict_first();      // the panel is written once and read much later
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int64_t item = first; item < a.n_items; item += stride) {
            int ct, rb;
            tile_of(a, item, &ct, &rb);
            const int block = 2 * rb + (int)rank;                         // this CTA's 128-row block
            const bool block_ok = block < a.n_blocks128;                  // an odd count leaves the last pair's second half empty
            const int64_t row = (int64_t)block * BM + row_in_tile;
            const RowGrad rg = block_ok ? a.grad[PODS_CLAMPED(row, (int64_t)a.n_blocks128 * BM, a.status)]
                                        : RowGrad{0.0f, 0.0f, 0, 0.0f};
            const float neg_g = -rg.g;
            {
                if (!mbar_wait(&bar.acc_full[acc], acc_phase, timed_out)) timed_out = true;
                tcgen05_fence_after();
                const int col0 = (a.tile0 + ct) * BN;                     // vocabulary entry of the tile's first column
                const int valid_cols = min(BN, a.V - col0);              // beyond the vocabulary the gradient is 0
                const int tok_col = rg.token - col0;                     // the target's column in this tile, if inside
#pragma unroll 1
                for (int c0 = col_begin; c0 < col_begin + BN / 2; c0 += 64) {
                    // 64 columns = one 128-byte line of the panel per row; the warp's 32 lines are staged in shared
                    // memory (16-byte pieces swizzled as the store's tensor map expects) and leave as one bulk store
                    uint4 q[8];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int c = c0 + 32 * h;
                        float v[32];
                        tmem_load_32(tmem_base + lane_addr + (uint32_t)(acc * BN + c), v);
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = neg_g * ex2(fmaf(v[i], kLog2e, -rg.lse2));
                        if (c + 32 > valid_cols) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = (c + i < valid_cols) ? v[i] : 0.0f;
                        }
                        if ((unsigned)(tok_col - c) < 32u) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = (tok_col - c == i) ? rg.g_token : v[i];
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            q[4 * h + j] = make_uint4(pack_bf16x2(v[8 * j], v[8 * j + 1]), pack_bf16x2(v[8 * j + 2], v[8 * j + 3]),
                                                      pack_bf16x2(v[8 * j + 4], v[8 * j + 5]), pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
                    }
                    // the previous store must have finished reading the staging lines before they are overwritten
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4*>(stage_line + ((j ^ (lane & 7)) << 4)) = q[j];
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && block_ok && PODS_INDEX_OK((int64_t)ct * BN + c0 + 63, a.ldp, a.status)) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%1, %2}], [%3], %4;"
                                     ::"l"(reinterpret_cast<uint64_t>(&map_panel)), "r"(ct * BN + c0),
                                       "r"(block * BM + quarter * 32), "r"(smem_u32(stage_warp)), "l"(stream_policy) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_leader(&bar.acc_empty[acc]);
                if (++acc == kAccumulators) { acc = 0; acc_phase ^= 1u; }
            }
        }
    }
    // a warp's bulk stores must be complete before its shared memory goes away
    if (warp >= 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (timed_out && lane == 0) pods_raise(a.status, PODS_STATUS_TIMEOUT);
    pair_teardown(tmem_base, warp);
}

// ------------------------------------------------------------------------------------------------------
// Steps 4 and 5: C[m, n] (+)= sum_k A[m, k] B[k, n] with C fp32 row-major, B stored by rows of n (MN-major) and
// A stored either by rows of k (A_MN = false: the panel as it is) or by rows of m (A_MN = true: the panel
// transposed, read in place).
// ------------------------------------------------------------------------------------------------------
struct GemmArgs {
    int32_t m_tiles, n_tiles, k_blocks;
    int32_t b_k0;                // first contraction row of B inside its matrix
    int64_t m_valid, n_valid;    // rows and columns of C that exist
    float* C;
    int64_t ldc;
    int32_t accumulate;          // 0: C = product, 1: C += product
    uint32_t* status;
};

// By CTA pairs (cluster of two, tcgen05 cta_group::2): a pair owns a 256 x 256 tile of C.  CTA r of the pair loads
// rows m0 + 128 r .. of A and columns n0 + 128 r .. of B, the leader issues M = 256 MMAs that read both CTAs' shared
// memory and fill both CTAs' tensor memory, and each CTA's epilogue adds its own 128 rows into C.
template <bool A_MN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
lm_head_grad_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                              const GemmArgs g) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* const tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    PairBarriers& bar = *reinterpret_cast<PairBarriers*>(tiles + (size_t)kPairStages * kPairStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t tmem_base = pair_setup(bar, warp, 4);
    const int m_pairs = (g.m_tiles + 1) / 2;
    const int64_t n_tiles_total = (int64_t)m_pairs * g.n_tiles;
    const int64_t first = blockIdx.x >> 1, stride = gridDim.x >> 1;
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int64_t loads = 0;
            for (int64_t tile = first; tile < n_tiles_total; tile += stride) {
                const int m0 = (int)(tile / g.n_tiles) * 2 * BM + (int)rank * BM;
                const int n0 = (int)(tile % g.n_tiles) * BN + (int)rank * (BN / 2);
                for (int kb = 0; kb < g.k_blocks; ++kb) {
                    if (!mbar_wait(&bar.empty[stage], phase ^ 1u, timed_out)) timed_out = true;
                    unsigned char* sa = tiles + (size_t)stage * kPairStageBytes;
                    if (rank == 0) mbar_expect_tx(&bar.full[stage], 2 * kPairStageBytes);
                    if (A_MN) {
#pragma unroll
                        for (int i = 0; i < BM / 64; ++i)
                            tma_load_tile_pair(sa + i * kBoxBytes, &map_a, m0 + 64 * i, kb * BK, &bar.full[stage]);
                    } else {
                        tma_load_tile_pair(sa, &map_a, kb * BK, m0, &bar.full[stage]);
                    }
#pragma unroll
                    for (int i = 0; i < BN / 2 / 64; ++i)
                        tma_load_tile_pair(sa + kPairStageBytesA + i * kBoxBytes, &map_b, n0 + 64 * i, g.b_k0 + kb * BK, &bar.full[stage]);
                    ++loads;
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (rank == 0 && !drain_loads_pair(bar, loads)) timed_out = true;
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            constexpr uint32_t idesc = instr_desc_pair(A_MN, true);
            constexpr uint64_t a_step = A_MN ? (uint64_t)(UMMA_K * 128 >> 4) : (uint64_t)(UMMA_K * 2 >> 4);
            constexpr uint64_t b_step = (uint64_t)(UMMA_K * 128 >> 4);
            for (int64_t tile = first; tile < n_tiles_total; tile += stride) {
                if (!mbar_wait_cluster(&bar.acc_empty[acc], acc_phase ^ 1u, timed_out)) timed_out = true;
                tcgen05_fence_after();
                const uint32_t tmem_acc = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < g.k_blocks; ++kb) {
                    if (!mbar_wait(&bar.full[stage], phase, timed_out)) timed_out = true;
                    tcgen05_fence_after();
                    const uint32_t sa = smem_u32(tiles + (size_t)stage * kPairStageBytes);
                    const uint64_t da = A_MN ? smem_desc_mn_major(sa) : smem_desc_k_major(sa);
                    const uint64_t db = smem_desc_mn_major(sa + kPairStageBytesA);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_pair(tmem_acc, da + a_step * k, db + b_step * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_commit_pair(&bar.empty[stage]);
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                }
                umma_commit_pair(&bar.acc_full[acc]);
                if (++acc == kAccumulators) { acc = 0; acc_phase ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int64_t tile = first; tile < n_tiles_total; tile += stride) {
            const int64_t row = (int64_t)(tile / g.n_tiles) * 2 * BM + (int64_t)rank * BM + row_in_tile;
            const int n0 = (int)(tile % g.n_tiles) * BN;
            const bool row_ok = row < g.m_valid;
            float* const c_row = g.C + (row_ok ? row : 0) * g.ldc;
            if (!mbar_wait(&bar.acc_full[acc], acc_phase, timed_out)) timed_out = true;
            tcgen05_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                float v[32];
                tmem_load_32(tmem_base + lane_addr + (uint32_t)(acc * BN + c0), v);
                if (row_ok) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int col = n0 + c0 + 4 * q;
                        if (col + 3 < g.n_valid) {
                            float4* p = reinterpret_cast<float4*>(c_row + col);
                            float4 o = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                            if (g.accumulate) {
                                const float4 old = *p;
                                o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                            }
                            *p = o;
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(&bar.acc_empty[acc]);
            if (++acc == kAccumulators) { acc = 0; acc_phase ^= 1u; }
        }
    }
    if (timed_out && lane == 0) pods_raise(g.status, PODS_STATUS_TIMEOUT);
    pair_teardown(tmem_base, warp);
}

// How a call is cut up: the statistics plan, the panels of the vocabulary and the workspace regions.
struct Layout {
    Plan stats;                  // statistics pass over the whole vocabulary
    int64_t rows_padded;         // T rounded up to whole 128-row blocks
    int total_tiles;             // 256-column tiles of the vocabulary
    int tiles_per_panel, n_panels;
    int64_t ldp;                 // panel row pitch in elements = tiles_per_panel * 256 + 64
    size_t off_row_loss, off_grad, off_panel, bytes;
};

// Time of one panel of c column tiles in units of one 128 x 256 x 64 block of tensor-core work per CTA: every kernel
// runs its 256 x 256 pair tiles in waves over the SM pairs, so what counts is (waves) x (contraction blocks per tile)
// for the three of them.
int64_t panel_cost(int64_t c, int64_t row_blocks, int64_t d, int sms) {
    const int64_t pairs = sms / 2 > 0 ? sms / 2 : 1, row_pairs = (row_blocks + 1) / 2;
    const int64_t n_d = (d + BN - 1) / BN;
    const int64_t dlogits = (c * row_pairs + pairs - 1) / pairs * ((d + BK - 1) / BK);
    const int64_t dhidden = (row_pairs * n_d + pairs - 1) / pairs * (c * BN / BK);
    const int64_t dw = (c * n_d + pairs - 1) / pairs * (row_blocks * BM / BK);
    return dlogits + dhidden + dw + 150;             // + three launches' ramp-up and tail
}

Layout make_layout(int64_t T, int32_t V, int32_t d, int sms) {
    Layout l;
    l.stats = make_plan(T, V, sms);
    l.rows_padded = (int64_t)l.stats.n_row_blocks * BM;
    l.total_tiles = l.stats.n_col_tiles;
    int64_t max_tiles = (int64_t)(g_panel_bytes / ((size_t)l.rows_padded * BN * 2));
    if (max_tiles < 1) max_tiles = 1;
    if (max_tiles > l.total_tiles) max_tiles = l.total_tiles;
    // tiles per panel: the count within the memory limit with the least wave-quantisation loss over the whole call
    int64_t best = -1;
    l.tiles_per_panel = (int)max_tiles;
    for (int64_t c = max_tiles; c >= 1 && c >= max_tiles / 2; --c) {
        const int64_t full = l.total_tiles / c, rest = l.total_tiles % c;
        const int64_t cost = full * panel_cost(c, l.stats.n_row_blocks, d, sms) +
                             (rest ? panel_cost(rest, l.stats.n_row_blocks, d, sms) : 0);
        if (best < 0 || cost < best) { best = cost; l.tiles_per_panel = (int)c; }
    }
    l.n_panels = (l.total_tiles + l.tiles_per_panel - 1) / l.tiles_per_panel;
    l.ldp = (int64_t)l.tiles_per_panel * BN + 64;       // + one 128-byte line: rows of the panel must not be a power of two apart
    size_t off = align_up((size_t)l.stats.n_parts * (size_t)l.rows_padded * sizeof(float2), 256);
    l.off_row_loss = off;
    off += align_up((size_t)T * sizeof(double), 256);
    l.off_grad = off;
    off += align_up((size_t)l.rows_padded * sizeof(RowGrad), 256);
    l.off_panel = off;
    off += align_up((size_t)l.rows_padded * (size_t)l.ldp * 2, 256);
    l.bytes = off;
    return l;
}

template <bool A_MN>
int launch_gemm(const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmArgs& g, int sms, cudaStream_t s) {
    if ((int64_t)g.m_tiles * g.n_tiles <= 0 || g.k_blocks <= 0) return PODS_OK;
    // an even grid: one pair of CTAs per 256 x 256 tile at a time
    const int64_t pair_tiles = (int64_t)((g.m_tiles + 1) / 2) * g.n_tiles;
    const int64_t pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
    PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(lm_head_grad_gemm_pair_kernel<A_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemBytes));
    lm_head_grad_gemm_pair_kernel<A_MN><<<(int)(2 * pairs), kThreads, kPairSmemBytes, s>>>(map_a, map_b, g);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

}  // namespace

extern "C" size_t pods_set_loss_from_hidden_panel_bytes(size_t bytes) {
    const size_t before = g_panel_bytes;
    g_panel_bytes = bytes < (size_t)65536 ? (size_t)65536 : bytes;
    return before;
}

extern "C" size_t grpo_loss_from_hidden_workspace_bytes(int64_t T, int32_t V, int32_t d) {
    if (T <= 0 || V <= 0 || d <= 0) return 0;
    return make_layout(T, V, d, pods_sm_count()).bytes;
}

extern "C" int grpo_loss_from_hidden(const void* hidden, int64_t ldh, const void* W, int64_t ldw, const int32_t* tokens,
                                     const float* old_logp, const float* ref_logp, const float* adv,
                                     const double* seq_weight, const int64_t* cu_seqlens, int64_t M, int64_t row0,
                                     const uint8_t* mask, int64_t T, int32_t V, int32_t d, float eps, float beta,
                                     float grad_scale, double* loss_acc, float* logp, float* dhidden, int64_t lddh,
                                     float* dW, int64_t lddw, void* workspace, size_t workspace_bytes,
                                     uint32_t* status, void* stream) {
    if (T < 0 || V < 1 || M < 1 || row0 < 0 || d < 8 || d % 8 != 0 || ldh < d || ldw < d || ldh % 8 != 0 ||
        ldw % 8 != 0 || lddh < d || lddw < d || lddh % 4 != 0 || lddw % 4 != 0)
        return PODS_ERR_INVALID_ARG;
    if (!(eps >= 0.0f) || !(beta == beta)) return PODS_ERR_INVALID_ARG;
    if (T == 0) return PODS_OK;
    if (hidden == nullptr || W == nullptr || tokens == nullptr || old_logp == nullptr || adv == nullptr ||
        seq_weight == nullptr || cu_seqlens == nullptr || loss_acc == nullptr || logp == nullptr ||
        dhidden == nullptr || dW == nullptr)
        return PODS_ERR_INVALID_ARG;
    if (ref_logp == nullptr && beta != 0.0f) return PODS_ERR_INVALID_ARG;
    if (!pods_aligned(hidden, 16) || !pods_aligned(W, 16) || !pods_aligned(dhidden, 16) || !pods_aligned(dW, 16) ||
        !pods_aligned(loss_acc, 8) || !pods_aligned(logp, 4))
        return PODS_ERR_INVALID_ARG;
    const int sms = pods_sm_count();
    const Layout l = make_layout(T, V, d, sms);
    if (workspace == nullptr || workspace_bytes < l.bytes || !pods_aligned(workspace, 256)) return PODS_ERR_WORKSPACE;

    unsigned char* ws = static_cast<unsigned char*>(workspace);
    float2* partial = reinterpret_cast<float2*>(ws);
    double* row_loss = reinterpret_cast<double*>(ws + l.off_row_loss);
    RowGrad* grad = reinterpret_cast<RowGrad*>(ws + l.off_grad);
    uint16_t* panel = reinterpret_cast<uint16_t*>(ws + l.off_panel);
    cudaStream_t s = pods_stream(stream);

    // 1. statistics of every row over the whole vocabulary
    int rc = launch_lm_head_stats(hidden, ldh, W, ldw, T, V, d, l.stats, partial, status, s);
    if (rc != PODS_OK) return rc;

    // 2. log-probs, loss terms, gradient factors
    TermsArgs ta;
    ta.hidden = static_cast<const uint16_t*>(hidden);
    ta.ldh = ldh;
    ta.W = static_cast<const uint16_t*>(W);
    ta.ldw = ldw;
    ta.partial = partial;
    ta.n_parts = l.stats.n_parts;
    ta.rows_padded = l.rows_padded;
    ta.d = d;
    ta.grad = grad;
    pods_loss::RowArgs& a = ta.row;
    a.logits = nullptr;
    a.ldl = 0;
    a.tokens = tokens;
    a.old_logp = old_logp;
    a.ref_logp = ref_logp;
    a.adv = adv;
    a.seq_weight = seq_weight;
    a.cu_seqlens = cu_seqlens;
    a.M = M;
    a.row0 = row0;
    a.mask = mask;
    a.T = T;
    a.V = V;
    a.eps = eps;
    a.beta = beta;
    a.grad_scale = grad_scale;
    a.logp = logp;
    a.dlogits = nullptr;
    a.ldd = 0;
    a.row_loss = row_loss;
    a.prep = nullptr;
    a.status = status;
    a.vec_ok = 0;
    a.precise = 0;
    const int warps_per_block = 8;
    lm_head_row_terms_kernel<<<(unsigned)((l.rows_padded + warps_per_block - 1) / warps_per_block), warps_per_block * 32, 0, s>>>(ta);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    rc = pods_loss::launch_loss_reduce(row_loss, T, loss_acc, s);
    if (rc != PODS_OK) return rc;

    // 3-5. panel by panel
    CUtensorMap map_h_rows, map_w_rows;          // hidden / W tiles by rows of d: K-major operands of the logits
    CUtensorMap map_w_box, map_h_box;            // the same matrices in 64 x 64 boxes: MN-major B operands
    CUtensorMap map_panel_rows, map_panel_box;   // the panel as K-major A (dhidden) and as MN-major A (dW)
    CUtensorMap map_panel_store;                 // the panel in 32 x 64 boxes: what an epilogue warp stores at a time
    if ((rc = make_map(&map_h_rows, hidden, T, d, ldh, BM)) != PODS_OK) return rc;
    if ((rc = make_map(&map_w_rows, W, V, d, ldw, BN / 2)) != PODS_OK) return rc;
    if ((rc = make_map(&map_w_box, W, V, d, ldw, 64)) != PODS_OK) return rc;
    if ((rc = make_map(&map_h_box, hidden, T, d, ldh, 64)) != PODS_OK) return rc;
    if ((rc = make_map(&map_panel_rows, panel, l.rows_padded, (int64_t)l.tiles_per_panel * BN, l.ldp, BM)) != PODS_OK) return rc;
    if ((rc = make_map(&map_panel_box, panel, l.rows_padded, (int64_t)l.tiles_per_panel * BN, l.ldp, 64)) != PODS_OK) return rc;
    if ((rc = make_map(&map_panel_store, panel, l.rows_padded, (int64_t)l.tiles_per_panel * BN, l.ldp, 32)) != PODS_OK) return rc;
    PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(lm_head_dlogits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDlogitsSmemBytes));

    for (int p = 0; p < l.n_panels; ++p) {
        const int tile0 = p * l.tiles_per_panel;
        const int n_tiles = (l.total_tiles - tile0 < l.tiles_per_panel) ? l.total_tiles - tile0 : l.tiles_per_panel;
        if (n_tiles <= 0) break;
        const int64_t cols = (int64_t)n_tiles * BN;
        const Plan pp = make_plan(T, cols, sms);

        DlogitsArgs da;
        da.V = V;
        da.d = d;
        da.n_row_blocks = (pp.n_row_blocks + 1) / 2;
        da.n_blocks128 = pp.n_row_blocks;
        da.tile0 = tile0;
        da.n_col_tiles = n_tiles;
        da.group_rows = da.n_row_blocks < 32 ? da.n_row_blocks : 32;    // 32 pairs = 64 blocks of 128 rows
        da.n_items = (int64_t)n_tiles * da.n_row_blocks;
        da.grad = grad;
        da.ldp = l.ldp;
        da.status = status;
        lm_head_dlogits_kernel<<<(int)(2 * (da.n_items < sms / 2 ? da.n_items : sms / 2)), kDlogitsThreads, kDlogitsSmemBytes, s>>>(map_h_rows, map_w_rows, map_panel_store, da);
        PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());

        GemmArgs gh;                             // dhidden[T, d] (+)= panel[T, cols] . W[tile0 * 256 + (0 .. cols), d]
        gh.m_tiles = pp.n_row_blocks;
        gh.n_tiles = (d + BN - 1) / BN;
        gh.k_blocks = (int)(cols / BK);
        gh.b_k0 = tile0 * BN;
        gh.m_valid = T;
        gh.n_valid = d;
        gh.C = dhidden;
        gh.ldc = lddh;
        gh.accumulate = p > 0 ? 1 : 0;
        gh.status = status;
        if ((rc = launch_gemm<false>(map_panel_rows, map_w_box, gh, sms, s)) != PODS_OK) return rc;

        GemmArgs gw;                             // dW[tile0 * 256 + (0 .. cols), d] += panel^T . hidden
        gw.m_tiles = (int)(cols / BM);
        gw.n_tiles = (d + BN - 1) / BN;
        gw.k_blocks = (int)(l.rows_padded / BK);
        gw.b_k0 = 0;
        gw.m_valid = (int64_t)V - (int64_t)tile0 * BN < cols ? (int64_t)V - (int64_t)tile0 * BN : cols;
        gw.n_valid = d;
        gw.C = dW + (int64_t)tile0 * BN * lddw;
        gw.ldc = lddw;
        gw.accumulate = 1;
        gw.status = status;
        if ((rc = launch_gemm<true>(map_panel_box, map_h_box, gw, sms, s)) != PODS_OK) return rc;
    }
    return PODS_OK;
}

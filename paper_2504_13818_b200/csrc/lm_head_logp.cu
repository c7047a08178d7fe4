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

#include <cuda.h>
#include <math.h>

#include "pods_common.cuh"

namespace {

constexpr int BM = 128;                 // rows of a tile: the TMEM lanes
constexpr int BN = 256;                 // vocabulary entries of a tile: one MMA's N
constexpr int BK = 64;                  // hidden features per stage: 128 bytes of bf16, the swizzle span
constexpr int UMMA_K = 16;              // features per tcgen05.mma of kind::f16
constexpr int kStages = 4;
constexpr int kAccumulators = 2;        // 2 x 256 fp32 columns = the 512 columns of tensor memory
constexpr int kThreads = 192;
constexpr uint32_t kStageBytesA = BM * BK * 2, kStageBytesB = BN * BK * 2;
constexpr uint32_t kStageBytes = kStageBytesA + kStageBytesB;
constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + 256 /*barriers*/;
constexpr uint32_t kWaitLimit = 1u << 22;   // polls (each may suspend up to ~1 us) before a wait gives up
constexpr float kLog2e = 1.4426950408889634f;

struct Barriers {
    unsigned long long full[kStages];          // TMA -> MMA: the stage's two blocks have landed
    unsigned long long empty[kStages];         // MMA -> TMA: the stage has been consumed
    unsigned long long acc_full[kAccumulators];    // MMA -> epilogue: the tile's accumulator is complete
    unsigned long long acc_empty[kAccumulators];   // epilogue -> MMA: the accumulator has been read
    uint32_t tmem_base;
    uint32_t pad;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 1000;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the barrier's phase did not complete within kWaitLimit polls (or `hurry` is set:
// after a first time-out nothing is waited for any more).
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, bool hurry) {
    const uint32_t limit = hurry ? 1u : kWaitLimit;
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// One 2-D tile of a row-major bf16 matrix into shared memory; completion is counted on `bar`.
// x = first feature (a multiple of 64: 128-byte aligned), y = first row.  This CTA's own shared memory only.
__device__ __forceinline__ void tma_load_tile(void* dst, const CUtensorMap* map, int x, int y, void* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

// Shared-memory operand descriptor of tcgen05.mma for a K-major bf16 block stored as rows of 128 bytes with the
// 128-byte swizzle (what the TMA load above writes): start address / 16, leading byte offset 1 (not used by
// swizzled K-major layouts), stride between groups of eight rows 1024 bytes, descriptor version 1, swizzle mode 2.
__device__ __forceinline__ uint64_t smem_operand_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor of kind::f16: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1), both K-major
// (bits 15, 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void umma(uint32_t tmem_acc, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_acc), "l"(a_desc), "l"(b_desc), "r"(kInstrDesc), "r"(accumulate) : "memory");
}
// Arrives on `bar` once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(void* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane (the warp reads its 32 lanes at once).
__device__ __forceinline__ void tmem_load_32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

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

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar.full[s], 1); mbar_init(&bar.empty[s], 1); }
        for (int b = 0; b < kAccumulators; ++b) { mbar_init(&bar.acc_full[b], 1); mbar_init(&bar.acc_empty[b], 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {       // the warp that allocates tensor memory also frees it
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bar.tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = bar.tmem_base;
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
            // every load has to have landed before the CTA may end (at once when nothing went wrong)
            for (int s = 0; s < kStages; ++s) {
                const int64_t uses = loads > s ? (loads - s + kStages - 1) / kStages : 0;
                if (uses > 0 && !mbar_wait(&bar.full[s], (uint32_t)((uses - 1) & 1), false)) timed_out = true;
            }
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
                        const uint64_t da = smem_operand_desc(sa), db = smem_operand_desc(sa + kStageBytesA);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k)      // 16 features = 32 bytes further along the rows
                            umma(tmem_acc, da + (uint64_t)(k * UMMA_K * 2 >> 4), db + (uint64_t)(k * UMMA_K * 2 >> 4),
                                 (kb | k) != 0 ? 1u : 0u);
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
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
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
    // the target's logit: hidden[t] . W[tok], eight features per 128-bit load
    const uint4* h4 = reinterpret_cast<const uint4*>(hidden + t * ldh);
    const uint4* w4 = reinterpret_cast<const uint4*>(W + (int64_t)tok * ldw);
    float dot = 0.0f;
    for (int j = lane; j < d / 8; j += 32) {
        const uint4 hv = h4[j], wv = w4[j];
        const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w}, ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            dot = fmaf(__uint_as_float(hw[q] << 16), __uint_as_float(ww[q] << 16), dot);
            dot = fmaf(__uint_as_float(hw[q] & 0xffff0000u), __uint_as_float(ww[q] & 0xffff0000u), dot);
        }
    }
    // the parts: lane p takes parts p, p + 32, ...
    float m = -INFINITY, s = 0.0f;
    for (int p = lane; p < n_parts; p += 32) {
        const float2 ms = partial[(size_t)p * rows_padded + t];
        const float m_new = fmaxf(m, ms.x);
        if (m_new != -INFINITY) {
            s = s * exp2f(m - m_new) + ms.y * exp2f(ms.x - m_new);
            m = m_new;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        dot += __shfl_xor_sync(PODS_FULL_MASK, dot, o);
        const float mo = __shfl_xor_sync(PODS_FULL_MASK, m, o), so = __shfl_xor_sync(PODS_FULL_MASK, s, o);
        const float m_new = fmaxf(m, mo);
        if (m_new != -INFINITY) {
            s = s * exp2f(m - m_new) + so * exp2f(mo - m_new);
            m = m_new;
        }
    }
    if (lane == 0) {
        const double lse = ((double)m + log2((double)s)) * 0.6931471805599453;
        logp[t] = (float)((double)dot - lse);
        if (lse_out != nullptr) lse_out[t] = (float)lse;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link the driver).
EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = nullptr;
    if (fn != nullptr) return fn;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
        return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
    return fn;
}

// Row-major bf16 matrix [rows, cols] with row pitch ld elements; tiles of box_rows x 64, 128-byte swizzle,
// elements outside the matrix read as zero.
int make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_rows) {
    EncodeTiledFn encode = tensor_map_encoder();
    if (encode == nullptr) return PODS_ERR_CUDA;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    const CUresult rc = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? PODS_OK : PODS_ERR_CUDA;
}

struct Plan {
    int n_row_blocks, n_col_tiles, tiles_per_part, n_parts, grid;
};

// Parts of the vocabulary: the tile count per part that minimises (waves of items over the SMs) x (tiles per
// item), the smaller count among equals: small parts keep the CTAs' rows of W together in L2.
Plan make_plan(int64_t T, int32_t V, int sms) {
    Plan p;
    p.n_row_blocks = (int)((T + BM - 1) / BM);
    p.n_col_tiles = (V + BN - 1) / BN;
    int64_t best_cost = -1;
    p.tiles_per_part = p.n_col_tiles;
    for (int tpp = 1; tpp <= p.n_col_tiles && tpp <= 64; ++tpp) {
        const int parts = (p.n_col_tiles + tpp - 1) / tpp;
        const int64_t items = (int64_t)parts * p.n_row_blocks;
        const int64_t waves = (items + sms - 1) / sms;
        const int64_t cost = waves * tpp * 64 + parts;          // a little for the items' fixed cost
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; p.tiles_per_part = tpp; }
    }
    p.n_parts = (p.n_col_tiles + p.tiles_per_part - 1) / p.tiles_per_part;
    const int64_t items = (int64_t)p.n_parts * p.n_row_blocks;
    p.grid = (int)(items < sms ? items : sms);
    return p;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

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
    a.partial = static_cast<float2*>(workspace);
    a.status = status;

    cudaStream_t s = pods_stream(stream);
    PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(lm_head_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    lm_head_stats_kernel<<<plan.grid, kThreads, kSmemBytes, s>>>(map_h, map_w, a);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    const int warps_per_block = 8;
    lm_head_merge_kernel<<<(unsigned)((T + warps_per_block - 1) / warps_per_block), warps_per_block * 32, 0, s>>>(
        static_cast<const uint16_t*>(hidden), ldh, static_cast<const uint16_t*>(W), ldw, tokens, T, V, d, a.partial,
        plan.n_parts, (int64_t)plan.n_row_blocks * BM, logp, lse, status);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

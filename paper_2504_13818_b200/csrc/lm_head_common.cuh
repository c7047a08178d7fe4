// Pieces shared by the kernels that form the LM-head projection hidden W^T (or its transposes) on the tensor
// cores: tile sizes, mbarrier / TMA / tcgen05 wrappers, operand descriptors, tensor-map construction.
// Everything here addresses this CTA's own shared memory and this GPU's own global memory; no load is multicast.
#pragma once

#include <cuda.h>
#include <math.h>

#include "pods_common.cuh"

namespace pods_lm {

constexpr int BM = 128;                 // rows of a tile: the TMEM lanes
constexpr int BN = 256;                 // columns of a tile: one MMA's N
constexpr int BK = 64;                  // contraction entries per stage: 128 bytes of bf16, the swizzle span
constexpr int UMMA_K = 16;              // contraction entries per tcgen05.mma of kind::f16
constexpr int kStages = 4;
constexpr int kAccumulators = 2;        // 2 x 256 fp32 columns = the 512 columns of tensor memory
constexpr int kThreads = 192;
constexpr uint32_t kStageBytesA = BM * BK * 2, kStageBytesB = BN * BK * 2;
constexpr uint32_t kStageBytes = kStageBytesA + kStageBytesB;
constexpr uint32_t kBoxBytes = 64 * BK * 2;     // one 64 x 64 box of a matrix whose tile dimension is contiguous
constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + 256 /*barriers*/;
constexpr uint32_t kWaitLimit = 1u << 22;   // polls (each may suspend up to ~1 us) before a wait gives up
constexpr float kLog2e = 1.4426950408889634f;

struct Barriers {
    unsigned long long full[kStages];          // TMA -> MMA: the stage's blocks have landed
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

// One 2-D box of a row-major bf16 matrix into shared memory; completion is counted on `bar`.
// x = first element along the rows (a multiple of 64: 128-byte aligned), y = first row.
__device__ __forceinline__ void tma_load_tile(void* dst, const CUtensorMap* map, int x, int y, void* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

// L2 policy for data that is written once and read much later (the gradient panel's stores): first in line for
// eviction.  NOT for loads that several CTAs share: with this hint on the panel's loads the sharers' later requests
// missed and the panel crossed HBM three to four times.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// Shared-memory operand descriptors of tcgen05.mma for bf16 blocks stored as rows of 128 bytes with the
// 128-byte swizzle (what the TMA loads above write).  Common fields: start address / 16 in bits 0-13,
// descriptor version 1 (bit 46), swizzle mode 2 = 128 bytes (bits 61-63).
//
// K-major (each 128-byte row holds 64 consecutive contraction entries of one tile row): the leading byte
// offset is not used by swizzled K-major layouts (1); groups of eight rows are 1024 bytes apart.  A step of 16
// contraction entries moves the start address 32 bytes along the rows.
__device__ __forceinline__ uint64_t smem_desc_k_major(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// MN-major (each 128-byte row holds 64 consecutive tile rows - or columns, for B - at ONE contraction entry; a box
// is 64 such rows, i.e. 64 contraction entries): groups of eight contraction entries are 1024 bytes apart (the
// stride byte offset), the next 64 tile rows are one box further (the leading byte offset).  A step of 16
// contraction entries moves the start address 16 rows = 2048 bytes.
__device__ __forceinline__ uint64_t smem_desc_mn_major(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | ((uint64_t)(kBoxBytes >> 4) << 16) |
           ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1), bit 15 / 16 set
// when A / B is MN-major, N / 8 in bits 17-22, M / 16 in bits 24-28.
__host__ __device__ constexpr uint32_t instr_desc(bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t tmem_acc, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                     uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_acc), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on `bar` once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(void* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc_all(uint32_t* slot) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free_all(uint32_t tmem_base) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

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

// Barriers initialised, tensor memory allocated by warp 1 (which also frees it), everything visible to the CTA.
// `epilogue_warps` warps arrive (one lane each) when an accumulator has been read.
__device__ __forceinline__ uint32_t pipeline_setup(Barriers& bar, int warp, uint32_t epilogue_warps = 4) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar.full[s], 1); mbar_init(&bar.empty[s], 1); }
        for (int b = 0; b < kAccumulators; ++b) { mbar_init(&bar.acc_full[b], 1); mbar_init(&bar.acc_empty[b], epilogue_warps); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_all(&bar.tmem_base);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    return bar.tmem_base;
}
__device__ __forceinline__ void pipeline_teardown(uint32_t tmem_base, int warp) {
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        tmem_free_all(tmem_base);
    }
}
// After the producer's last load: every load has to have landed before the CTA may end.
__device__ __forceinline__ bool drain_loads(Barriers& bar, int64_t loads) {
    bool ok = true;
    for (int s = 0; s < kStages; ++s) {
        const int64_t uses = loads > s ? (loads - s + kStages - 1) / kStages : 0;
        if (uses > 0 && !mbar_wait(&bar.full[s], (uint32_t)((uses - 1) & 1), false)) ok = false;
    }
    return ok;
}

// ---------------------------------------------------------------------------------------------------------
// CTA pairs (a cluster of two CTAs on the two SMs of a TPC, tcgen05 cta_group::2): the pair computes one
// 256 x 256 tile; each CTA loads its own 128 rows of A and HALF of B (128 of the 256 columns), the leader (cluster
// rank 0) issues the MMAs for both, each CTA's tensor memory receives its own 128 rows of the accumulator.  Per
// contraction block a CTA then takes 32 KB from L2 instead of 48 KB, and the ring holds six stages instead of four.
// Barriers live at the same shared-memory offsets in both CTAs.  No load is multicast: every CTA issues its own loads
// into its own shared memory; only the completion is counted on the LEADER's barrier.
// ---------------------------------------------------------------------------------------------------------
constexpr int kPairStages = 6;
constexpr uint32_t kPairStageBytesA = BM * BK * 2, kPairStageBytesB = (BN / 2) * BK * 2;
constexpr uint32_t kPairStageBytes = kPairStageBytesA + kPairStageBytesB;          // per CTA
constexpr size_t kPairSmemBytes = 1024 + (size_t)kPairStages * kPairStageBytes + 256;

struct PairBarriers {
    unsigned long long full[kPairStages];      // leader's: both CTAs' loads of the stage have landed
    unsigned long long empty[kPairStages];     // each CTA's own: the stage has been consumed (signalled in both CTAs)
    unsigned long long acc_full[kAccumulators];    // each CTA's own: the accumulator is complete (signalled in both)
    unsigned long long acc_empty[kAccumulators];   // leader's: the epilogue warps of BOTH CTAs have read it
    uint32_t tmem_base;
    uint32_t pad;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The shared::cluster address of the same shared-memory location in the pair's leader (cluster rank 0).
__device__ __forceinline__ uint32_t leader_addr(const void* p) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(r) : "r"(smem_u32(p)));
    return r;
}
__device__ __forceinline__ void mbar_arrive_leader(const void* bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(leader_addr(bar)) : "memory");
}
// Bounded wait on one of this CTA's barriers whose arrivals come from BOTH CTAs of the pair: acquire at cluster scope.
__device__ __forceinline__ bool mbar_wait_cluster(void* bar, uint32_t parity, bool hurry) {
    const uint32_t limit = hurry ? 1u : kWaitLimit;
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, 1000;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (ok != 0) return true;
    }
    return false;
}
// A box into THIS CTA's shared memory; the bytes are counted on the LEADER's barrier at the same offset.
__device__ __forceinline__ void tma_load_tile_pair(void* dst, const CUtensorMap* map, int x, int y, const void* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(leader_addr(bar)) : "memory");
}
// Instruction descriptor of the pair's MMA: M = 256 (128 rows in each CTA), N = 256.
__host__ __device__ constexpr uint32_t instr_desc_pair(bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
}
__device__ __forceinline__ void umma_pair(uint32_t tmem_acc, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_acc), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the barrier at this offset in BOTH CTAs of the pair once every MMA issued so far has completed.
__device__ __forceinline__ void umma_commit_pair(void* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
// Both CTAs of the pair call these with the same warp (warp 1).
__device__ __forceinline__ void tmem_alloc_all_pair(uint32_t* slot) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free_all_pair(uint32_t tmem_base) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}
// Barriers initialised (both CTAs initialise their own copies), tensor memory allocated, and the whole PAIR in step:
// no CTA may signal its partner's barriers before they exist.
__device__ __forceinline__ uint32_t pair_setup(PairBarriers& bar, int warp, uint32_t epilogue_warps_per_cta) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) { mbar_init(&bar.full[s], 1); mbar_init(&bar.empty[s], 1); }
        for (int b = 0; b < kAccumulators; ++b) {
            mbar_init(&bar.acc_full[b], 1);
            mbar_init(&bar.acc_empty[b], 2 * epilogue_warps_per_cta);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_all_pair(&bar.tmem_base);
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    tcgen05_fence_after();
    return bar.tmem_base;
}
// Neither CTA may leave (its shared memory and barriers are the partner's too) before both are done.
__device__ __forceinline__ void pair_teardown(uint32_t tmem_base, int warp) {
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tcgen05_fence_after();
        tmem_free_all_pair(tmem_base);
    }
}
// The last use of each stage's full barrier (leader only): every load of BOTH CTAs has landed.
__device__ __forceinline__ bool drain_loads_pair(PairBarriers& bar, int64_t loads) {
    bool ok = true;
    for (int s = 0; s < kPairStages; ++s) {
        const int64_t uses = loads > s ? (loads - s + kPairStages - 1) / kPairStages : 0;
        if (uses > 0 && !mbar_wait(&bar.full[s], (uint32_t)((uses - 1) & 1), false)) ok = false;
    }
    return ok;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link the driver).
static inline EncodeTiledFn tensor_map_encoder() {
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

// Row-major bf16 matrix [rows, cols] with row pitch ld elements; boxes of box_rows x 64, 128-byte swizzle,
// elements outside the matrix read as zero.
static inline int make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_rows) {
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

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Parts of a range of column tiles: the tile count per part that minimises (waves of items over the SMs) x
// (tiles per item), the smaller count among equals: small parts keep the CTAs' rows of W together in L2.
struct Plan {
    int n_row_blocks, n_col_tiles, tiles_per_part, n_parts, grid;
};
static inline Plan make_plan(int64_t T, int64_t cols, int sms) {
    Plan p;
    p.n_row_blocks = (int)((T + BM - 1) / BM);
    p.n_col_tiles = (int)((cols + BN - 1) / BN);
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

// Log-sum-exp of a row from the (maximum of x log2e, sum of 2^(x log2e - maximum)) pairs its parts left, and
// the target's logit as the fp32 dot product hidden[t] . W[tok]; one warp per row, every lane gets the results.
__device__ __forceinline__ void merge_row(const uint16_t* __restrict__ hidden, int64_t ldh,
                                          const uint16_t* __restrict__ W, int64_t ldw, int64_t t, int tok, int32_t d,
                                          const float2* __restrict__ partial, int32_t n_parts, int64_t rows_padded,
                                          int lane, double* lse, float* x_tok) {
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
    *lse = ((double)m + log2((double)s)) * 0.6931471805599453;
    *x_tok = dot;
}

// lm_head_logp.cu: the statistics pass (tcgen05) that leaves one (maximum, sum) pair per row and part in
// `partial` ([plan.n_parts][plan.n_row_blocks * 128]), with plan = make_plan(T, V, SM count).
int launch_lm_head_stats(const void* hidden, int64_t ldh, const void* W, int64_t ldw, int64_t T, int32_t V, int32_t d,
                         const Plan& plan, float2* partial, uint32_t* status, cudaStream_t stream);

}  // namespace pods_lm

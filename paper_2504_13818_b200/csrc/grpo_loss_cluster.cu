// grpo_loss, cluster-resident rows: the fast path of the GRPO-PODS loss + gradient kernel.
//
// A thread-block cluster of CL CTAs owns one row of bf16 logits at a time; CTA r keeps the r-th
// segment of the row in its shared memory from the moment it is loaded until its gradient has been
// stored, so HBM sees exactly one read and one write per element and every other access is to
// shared memory.  Several clusters are resident per SM group, each in a different phase, so that
// the DRAM-bound load, the MUFU-bound sum and the store overlap.  Per row and CTA:
//
//   load    one thread issues bulk asynchronous copies global -> shared (8 KB pieces counted on one
//           mbarrier, never multicast) as soon as the previous row's store has finished reading the
//           buffer; another thread fetches the row's scalar inputs meanwhile;
//   max     packed bf16x2 maxima of the segment; block arg-max (m_r and its first position);
//   sum     e = 2^(x log2e - ref_r), ref_r = fl(m_r log2e), once per element: summed in fp32 per
//           thread / fp64 across threads with that one instance of m_r left out (this keeps Z - 1
//           accurate when one logit dominates), and bf16(e) written back in place;
//   share   (m_r, position, sum_r) published in shared memory; ONE cluster barrier; warp 0 of
//           every CTA reads the CL triples through distributed shared memory, combines them into
//           the row maximum M and Z - 1, and evaluates the fp64 scalar terms with its lanes in
//           parallel (redundantly per CTA: no second barrier);
//   grad    in place: bf16(coef_r * e) by a packed bf16 fused multiply-add with coef_r split into
//           two bf16 terms (coef_r folds in 2^(ref_r - M log2e)); the target entry is then
//           overwritten with g (1 - p);
//   store   one bulk asynchronous copy shared -> global of the whole segment.
//
// The wait on the load's mbarrier is bounded: after kSpinLimit failed polls the CTA raises
// PODS_STATUS_TIMEOUT and carries on with whatever is in the buffer, still taking part in every
// barrier, so neither it nor its cluster peers can hang.

#include "grpo_loss_common.cuh"

using namespace pods_loss;

namespace {

constexpr int kClBlock = 256;                 // threads per CTA
constexpr int kChunkVecs = 512;               // 16-byte vectors per bulk copy (8 KB)
constexpr int kCtrlBytes = 1024;              // barriers, exchange slots and row scalars ahead of the buffer
constexpr uint32_t kSpinLimit = 1u << 22;     // polls of one mbarrier before giving up

struct ClusterCtrl {
    unsigned long long full;                  // mbarrier of the row's load
    unsigned long long xkey[2];               // this CTA's arg-max key, read by the peers (slot = row parity:
    double xsum[2];                           // this CTA's partial sum      a slow peer may still be reading the
                                              //                             previous row's pair)
    unsigned long long red_k[kClBlock / 32];
    double red_d[kClBlock / 32];
    RowInputs in;                             // scalar inputs of the current row
    float x_tok;
    int token;
    float coef, target;
    int write_mode;
};
static_assert(sizeof(ClusterCtrl) <= kCtrlBytes, "control block too large");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; returns false if the barrier did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Global -> this CTA's shared memory, completion counted on an mbarrier.  No multicast.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, void* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The same barrier for warps that neither published nor will read anything remote: no fences.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_only() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ unsigned long long ld_peer_u64(const void* local, uint32_t rank) {
    uint32_t ra;
    unsigned long long v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(smem_u32(local)), "r"(rank));
    asm volatile("ld.shared::cluster.u64 %0, [%1];" : "=l"(v) : "r"(ra) : "memory");
    return v;
}

// e = 2^(x log2e - ref) for the eight values of a vector: returns their sum, leaves bf16(e) in q.
__device__ __forceinline__ float exp_vec_inplace(uint4& q, float ref) {
    const float e0 = ex2_approx(fmaf(bf16_lo(q.x), kLog2e, -ref)), e1 = ex2_approx(fmaf(bf16_hi(q.x), kLog2e, -ref));
    const float e2 = ex2_approx(fmaf(bf16_lo(q.y), kLog2e, -ref)), e3 = ex2_approx(fmaf(bf16_hi(q.y), kLog2e, -ref));
    const float e4 = ex2_approx(fmaf(bf16_lo(q.z), kLog2e, -ref)), e5 = ex2_approx(fmaf(bf16_hi(q.z), kLog2e, -ref));
    const float e6 = ex2_approx(fmaf(bf16_lo(q.w), kLog2e, -ref)), e7 = ex2_approx(fmaf(bf16_hi(q.w), kLog2e, -ref));
    q.x = pack_bf16x2(e0, e1);
    q.y = pack_bf16x2(e2, e3);
    q.z = pack_bf16x2(e4, e5);
    q.w = pack_bf16x2(e6, e7);
    return ((e0 + e1) + (e2 + e3)) + ((e4 + e5) + (e6 + e7));
}

// Sum over the vector's values of 2^(x log2e - ref), the first one equal to mx left out.
__device__ __noinline__ float exp_sum_excluding(uint4 q, float ref, float mx) {
    const float v[8] = {bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y),
                        bf16_lo(q.z), bf16_hi(q.z), bf16_lo(q.w), bf16_hi(q.w)};
    float s = 0.0f;
    bool skipped = false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const bool skip = !skipped && v[i] == mx;
        skipped |= skip;
        s += skip ? 0.0f : ex2_approx(fmaf(v[i], kLog2e, -ref));
    }
    return s;
}

// bf16(e * (c_hi + c_lo)) for two packed bf16 e: the small term first, then one fused rounding.
__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t e, uint32_t c_hi, uint32_t c_lo) {
    uint32_t t, o;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(t) : "r"(e), "r"(c_lo));
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(o) : "r"(e), "r"(c_hi), "r"(t));
    return o;
}

template <int CL>
__global__ void __launch_bounds__(kClBlock)
grpo_loss_cluster_kernel(const RowArgs a, const int seg_vecs) {
    extern __shared__ __align__(128) unsigned char smem[];
    ClusterCtrl& c = *reinterpret_cast<ClusterCtrl*>(smem);
    uint4* buf = reinterpret_cast<uint4*>(smem + kCtrlBytes);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_rank();
    const int64_t cluster_id = blockIdx.x / CL, n_clusters = gridDim.x / CL;
    const int nvec = a.V / 8;
    const int seg0 = (int)rank * seg_vecs;                                   // first vector of my segment
    const int cnt = max(0, min(seg_vecs, nvec - seg0));                      // vectors in my segment

    if (tid == 0) {
        mbar_init(&c.full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    uint32_t parity = 0;
    bool timed_out = false;
    for (int64_t t = cluster_id; t < a.T; t += n_clusters, parity ^= 1u) {
        const uint16_t* row = a.logits + t * a.ldl;
        uint16_t* drow = a.dlogits + t * a.ldd;

        // ---- load ------------------------------------------------------------------------------
        if (tid == 0) {
            bulk_wait_read();                      // the previous row's store has finished reading buf
            mbar_expect_tx(&c.full, (uint32_t)cnt * 16u);
            for (int v0 = 0; v0 < cnt; v0 += kChunkVecs)
                bulk_load(buf + v0, reinterpret_cast<const uint4*>(row) + seg0 + v0,
                          (uint32_t)min(kChunkVecs, cnt - v0) * 16u, &c.full);
        } else if (tid == 32) {
            int tok = a.tokens[t];
            if (tok < 0 || tok >= a.V) { tok = 0; if (rank == 0) pods_raise(a.status, PODS_STATUS_TOKEN_RANGE); }
            c.token = tok;
            c.x_tok = __uint_as_float((uint32_t)row[tok] << 16);   // before any peer stores this row in place
            c.in = load_row_inputs(a, t);
        }
        // after one timeout the CTA stops waiting for good: it fails fast instead of stalling per row
        if (!mbar_wait(&c.full, parity, timed_out ? 1u : kSpinLimit)) timed_out = true;

        // ---- max of my segment -------------------------------------------------------------------
        float m_t = -INFINITY;
        int pos_t = 0x7fffffff;
#pragma unroll 4
        for (int j = tid; j < cnt; j += kClBlock) {
            const float vm = vec_max(buf[j]);
            const bool up = vm > m_t;
            m_t = up ? vm : m_t;
            pos_t = up ? j : pos_t;
        }
        unsigned long long key = argmax_key(m_t, pos_t);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const unsigned long long o = __shfl_xor_sync(PODS_FULL_MASK, key, d);
            key = o > key ? o : key;
        }
        if (lane == 0) c.red_k[warp] = key;
        __syncthreads();
        unsigned long long seg_key = c.red_k[0];
#pragma unroll
        for (int w = 1; w < kClBlock / 32; ++w) seg_key = c.red_k[w] > seg_key ? c.red_k[w] : seg_key;
        const float m_r = argmax_key_value(seg_key);
        const int excl = argmax_key_pos(seg_key);                              // local vector of the left-out instance
        const float ref_r = m_r * kLog2e;

        // ---- sum, bf16(e) written back in place --------------------------------------------------
        float s_t = 0.0f;
        if (excl < cnt && (excl % kClBlock) == tid) s_t = exp_sum_excluding(buf[excl], ref_r, m_r);
#pragma unroll 2
        for (int j = tid; j < cnt; j += kClBlock) {
            uint4 q = buf[j];
            const float sum = exp_vec_inplace(q, ref_r);
            s_t += (j == excl) ? 0.0f : sum;
            buf[j] = q;
        }
        double sd = (double)s_t;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) sd += __shfl_xor_sync(PODS_FULL_MASK, sd, d);
        if (lane == 0) c.red_d[warp] = sd;
        __syncthreads();

        // ---- share: one cluster barrier, then the scalar terms on warp 0 -----------------------
        if (warp == 0) {
            if (lane == 0) {
                double s = 0.0;
#pragma unroll
                for (int w = 0; w < kClBlock / 32; ++w) s += c.red_d[w];
                c.xkey[parity] = seg_key;
                c.xsum[parity] = s;
            }
            __syncwarp();
            cluster_sync();                                                    // release my pair, acquire the peers'
            // lane r < CL holds the pair of rank r
            unsigned long long k_r = 0ull;
            double s_r = 0.0;
            if (lane < CL) {
                k_r = ld_peer_u64(&c.xkey[parity], lane);
                s_r = __longlong_as_double((long long)ld_peer_u64(&c.xsum[parity], lane));
            }
            // the row maximum; among equal maxima the lowest rank's instance is the one left out
            const float mr = argmax_key_value(k_r);
            unsigned long long best = lane < CL ? (k_r & 0xffffffff00000000ull) | (uint32_t)(0xffu - lane) : 0ull;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                const unsigned long long o = __shfl_xor_sync(PODS_FULL_MASK, best, d);
                best = o > best ? o : best;
            }
            const float mx = argmax_key_value(best);
            const int owner = 0xff - (int)(best & 0xffu);
            // sum_r is relative to ref_r: bring it to the row maximum; every segment but the owner's
            // gets back the instance of its own maximum that it left out
            double scale_r = 0.0, contrib = 0.0;
            if (lane < CL && mr != -INFINITY) {
                scale_r = exp((double)(mr - mx));
                const double true_r = s_r * ref_correction(mr, mr * kLog2e);
                contrib = (lane == owner) ? true_r : (true_r + 1.0) * scale_r;
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) contrib += __shfl_xor_sync(PODS_FULL_MASK, contrib, d);
            const double zp = contrib;                                         // Z - 1
            const double my_scale = __shfl_sync(PODS_FULL_MASK, scale_r, (int)rank);
            // scalar terms: the transcendental calls on three lanes at once
            const RowInputs in = c.in;
            const float x_tok = c.x_tok;
            const double logp = ((double)x_tok - (double)mx) - log1p(zp);
            double part = 0.0;
            if (lane == 0) part = exp(logp - in.old_logp);                     // rho
            else if (lane == 1) part = in.has_ref ? exp(in.ref_logp - logp) : 1.0;    // e^d
            else if (lane == 2) part = (x_tok == mx) ? zp / (1.0 + zp) : -expm1(logp);   // 1 - p
            const double rho = __shfl_sync(PODS_FULL_MASK, part, 0);
            const double ed = __shfl_sync(PODS_FULL_MASK, part, 1);
            const double one_minus_p = __shfl_sync(PODS_FULL_MASK, part, 2);
            if (lane == 0) {
                const double eps = (double)a.eps, beta = (double)a.beta;
                const double clipped = rho < 1.0 - eps ? 1.0 - eps : (rho > 1.0 + eps ? 1.0 + eps : rho);
                const double s1 = rho * in.adv, s2 = clipped * in.adv;
                double loss = -(s1 < s2 ? s1 : s2);
                double dl = (s1 <= s2) ? -in.adv * rho : 0.0;
                if (in.has_ref) {
                    const double d = in.ref_logp - logp;
                    loss += beta * (ed - d - 1.0);
                    dl += beta * (1.0 - ed);
                }
                const double g = (in.w != 0.0) ? (double)a.grad_scale * in.w * dl : 0.0;
                if (rank == 0) {
                    a.logp[t] = (float)logp;
                    a.row_loss[t] = (in.w != 0.0) ? in.w * loss : 0.0;   // a masked row adds nothing, whatever its inputs
                }
                // e^(x - M) = e_stored * 2^(ref_r - m_r log2e) * e^(m_r - M)
                c.coef = (float)(-g / (1.0 + zp) * ref_correction(m_r, ref_r) * my_scale);
                c.target = (float)(g * one_minus_p);
                c.write_mode = (g != 0.0) ? 1 : 0;
            }
        } else {
            cluster_arrive_relaxed();
        }
        __syncthreads();
        if (warp != 0) cluster_wait_only();        // completes at once: warp 0 is already past it

        // ---- grad, in place ------------------------------------------------------------------------
        if (c.write_mode == 0) {
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            for (int j = tid; j < cnt; j += kClBlock) buf[j] = z;
        } else {
            const float coef = c.coef;
            const uint16_t hi16 = to_bf16_bits(coef);
            const uint16_t lo16 = to_bf16_bits(coef - __uint_as_float((uint32_t)hi16 << 16));
            const uint32_t c_hi = (uint32_t)hi16 * 0x10001u, c_lo = (uint32_t)lo16 * 0x10001u;
#pragma unroll 4
            for (int j = tid; j < cnt; j += kClBlock) {
                uint4 q = buf[j];
                q.x = scale_bf16x2(q.x, c_hi, c_lo);
                q.y = scale_bf16x2(q.y, c_hi, c_lo);
                q.z = scale_bf16x2(q.z, c_hi, c_lo);
                q.w = scale_bf16x2(q.w, c_hi, c_lo);
                buf[j] = q;
            }
            const int tok_vec = (c.token >> 3) - seg0;                         // the target entry, if it is mine:
            if (tok_vec >= 0 && tok_vec < cnt && (tok_vec % kClBlock) == tid)  // rewritten by the thread that wrote it
                reinterpret_cast<uint16_t*>(buf)[tok_vec * 8 + (c.token & 7)] = to_bf16_bits(c.target);
        }
        fence_proxy_async();                       // my shared-memory writes, before the bulk copy reads them
        __syncthreads();

        // ---- store ---------------------------------------------------------------------------------
        if (tid == 0 && cnt > 0)
            bulk_store(reinterpret_cast<uint4*>(drow) + seg0, buf, (uint32_t)cnt * 16u);
    }
    if (tid == 0) bulk_wait_all();
    if (timed_out && lane == 0) pods_raise(a.status, PODS_STATUS_TIMEOUT);
    cluster_sync();                                // no CTA leaves while a peer may still read its exchange slots
}

template <int CL>
int launch_cluster(const RowArgs& a, cudaStream_t stream, bool* launched) {
    *launched = false;
    const int nvec = a.V / 8;
    int seg_vecs = (nvec + CL - 1) / CL;
    const size_t smem = (size_t)kCtrlBytes + (size_t)seg_vecs * 16;
    if (smem > 227 * 1024 || (size_t)seg_vecs * 16 >= (1u << 20)) return PODS_OK;     // does not fit: caller falls back
    auto kernel = grpo_loss_cluster_kernel<CL>;
    PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(CL, 1, 1);
    cfg.blockDim = dim3(kClBlock, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int max_clusters = 0;
    PODS_RETURN_IF_CUDA_ERROR(cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg));
    if (max_clusters < 1) return PODS_OK;
    const int64_t n_clusters = a.T < max_clusters ? a.T : max_clusters;
    cfg.gridDim = dim3((unsigned)(n_clusters * CL), 1, 1);
    PODS_RETURN_IF_CUDA_ERROR(cudaLaunchKernelEx(&cfg, kernel, a, seg_vecs));
    *launched = true;
    return PODS_OK;
}

}  // namespace

namespace pods_loss {

// Runs the chunk on the cluster path if the row shape allows it (16-byte aligned rows, V a multiple
// of 8 and large enough to be worth a cluster, segments that fit in shared memory).
int launch_grpo_loss_cluster(const RowArgs& a, cudaStream_t stream, bool* launched) {
    *launched = false;
    if (!a.vec_ok || a.V % 8 != 0 || a.V < 16384) return PODS_OK;
    return launch_cluster<8>(a, stream, launched);
}

}  // namespace pods_loss

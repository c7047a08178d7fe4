// grpo_loss, cluster-resident rows: the fast path of the GRPO-PODS loss + gradient kernel
// (L_PODS of Section 3.2 and its derivative with respect to the bf16 logits).
//
// A thread-block cluster of CL CTAs owns one row of logits at a time; CTA r keeps the r-th segment
// of the row in its shared memory from the moment it is loaded until its gradient has been stored,
// so HBM sees exactly one read and one write per element and every other access is to shared
// memory.  A CTA is eight consumer warps, one producer warp and one exchange warp that meet only
// through mbarriers, over a ring of NS segment buffers; no warp ever waits at a CTA-wide barrier.
// CL is chosen per launch: the smallest of 1 .. 10, 12, 16 whose padded stage (whole blocks of 32
// vectors per consumer warp) leaves room for the ring with two CTAs per SM (1 for a 16 K vocabulary,
// 8 for 128 K, 9 for 152 K, 16 from 222 K up): small clusters have fewer partners to wait for and leave
// fewer CTA slots of the GPU empty (cluster placement fills 296 slots with clusters of 1 or 2, 264 with
// 8, 270 with 9, 224 with 16).  Sizes above 8 are non-portable cluster sizes, which the launch asks for
// explicitly.
//
//   producer  one thread: bulk asynchronous copies global -> shared of the row's segment (8 KB
//             pieces counted on the stage's `full` barrier, one destination CTA each); as soon as the
//             consumers report a stage `done` it loads the row NS ahead into it.
//   consumer  warp w owns a fixed slice of the segment and is independent of the other warps:
//       front(i)  the slice is read from shared memory ONCE into registers (IT vectors per lane);
//                 max    packed bf16x2 maxima, warp arg-max -> m_w and the vector that holds its
//                        first instance;
//                 sum    e = 2^(x log2e - ref_w), ref_w = fl(m_w log2e), once per element, summed
//                        in fp32 with that ONE instance of m_w left out (this keeps Z - 1 accurate
//                        when one logit dominates), bf16(e) written back to shared memory in place;
//                        (m_w, sum_w) is handed to the exchange warp;
//       back(i-1) grad   bf16(coef_w * e) by packed bf16 multiply-adds with coef_w split into two
//                        bf16 terms (coef_w folds in 2^(ref_w - M log2e)), stored straight to global
//                        memory with 128-bit stores, the target entry then overwritten
//                        with g (1 - p) by the lane that stored its vector; the warp then arrives
//                        on the stage's `done` barrier.
//             front(i) runs before back(i-1), so the exchange of row i-1 has a whole sweep to finish.
//             Shared memory sees 8 bytes of traffic per element (2 in, 2 read, 2 written, 2 read).
//             A stage is written through both proxies (bulk copies in, bf16(e) by ordinary stores), so a
//             consumer fences the two before it reports the stage done.
//   exchange  for every row: writes the CTA's eight (m_w, sum_w) pairs into the slots it owns in
//             every peer's shared memory, each as ONE 64-bit word that carries the row's tag, so
//             that no fence or barrier crosses the cluster: a reader polls its 8 CL slots until all
//             show the tag.  It then combines the pairs into the row maximum M and Z - 1, evaluates
//             the fp64 scalar terms of the objective (three exponentials in one call on three
//             lanes, no logarithm), publishes the eight coef_w, and only then (nobody waits for it)
//             takes the logarithm for logp and the loss.
//
// Every wait is bounded: after kSpinLimit failed polls the waiter raises PODS_STATUS_TIMEOUT, stops
// waiting for good and carries on with whatever is in the buffers, still arriving on every barrier
// it owes, so neither it nor its cluster peers can hang; before the CTA returns the producer waits
// (again with a limit) for any copy still in flight.
//
// The per-row scalar inputs (token, its logit, old/ref log-prob, mask and rollout weight, advantage)
// are gathered beforehand by a small kernel into one 32-byte record per row, so that the exchange
// warp fetches them with two independent loads, one row ahead.

#include "grpo_loss_common.cuh"

using namespace pods_loss;

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kProducerWarp = kConsumerWarps;       // warp 8
constexpr int kExchangeWarp = kConsumerWarps + 1;   // warp 9
constexpr int kThreads = kConsumers + 64;
constexpr int kMaxStages = 3;
constexpr int kPieceVecs = 512;               // 16-byte vectors per bulk load (8 KB)
// (m_w, sum_w) slots per row parity: 64 serve clusters of up to 8 CTAs, 128 the larger ones (up to 16, which
// the launch has to ask for as a non-portable cluster size)
__host__ __device__ constexpr int slot_count(int cl) { return cl <= 8 ? 64 : 128; }
// barriers, row scalars and exchange slots ahead of the buffers
__host__ __device__ constexpr int ctrl_bytes(int cl) { return cl <= 8 ? 1408 : 2432; }
constexpr uint32_t kSpinLimit = 1u << 24;     // polls of one barrier or slot before giving up
constexpr uint32_t kSuspendNs = 1000;         // upper bound on the time one poll may suspend the thread: a wait
                                              // that never completes ends after at most 2^24 us = 17 s

struct Pair {
    uint32_t key;                             // ordered bf16 slice maximum in the upper half
    float sum;                                // sum of 2^(x log2e - ref_w) over the slice, one maximum left out
};

struct RowPublish {                           // what back(i) needs, per row parity
    float coef[kConsumerWarps];
    float target;
    int write_mode;
    int token;
    int pad;
};

template <int SLOTS>
struct Ctrl {
    unsigned long long full[kMaxStages];      // producer -> consumers: the stage's segment has landed
    unsigned long long done[kMaxStages];      // consumers -> producer: the stage has been read for the last time
    unsigned long long sumdone[2];            // consumers -> exchange: the CTA's pairs of the row are in `part`
    unsigned long long ready[2];              // exchange -> consumers: `pub` of the row is valid
    Pair part[2][kConsumerWarps];
    RowPublish pub[2];
    unsigned long long xslot[2][SLOTS];       // slot [parity][8 rank + warp] is written by CTA `rank` of the cluster:
                                              // (sum_w bits) << 32 | (ordered bf16 m_w) << 16 | tag of the row
};
static_assert(sizeof(Ctrl<slot_count(8)>) <= ctrl_bytes(8) && sizeof(Ctrl<slot_count(16)>) <= ctrl_bytes(16),
              "control block too large");

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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendNs) : "memory");
    return ok != 0;
}
// Bounded waits; return false if the barrier did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Global -> this CTA's shared memory, completion counted on an mbarrier; one destination CTA.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, void* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t peer_address(const void* local, uint32_t rank) {
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(smem_u32(local)), "r"(rank));
    return ra;
}
// One 64-bit store into a slot of a peer's shared memory.  The word carries its own row tag, so the
// reader needs no barrier and the writer no fence: the reader polls the slot until the tag is the
// row's (an aligned 64-bit store is seen whole or not at all).
__device__ __forceinline__ void push_word(uint32_t peer_slot, unsigned long long v) {
    asm volatile("st.relaxed.cluster.shared::cluster.b64 [%0], %1;" ::"r"(peer_slot), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long poll_word(const unsigned long long* slot) {
    unsigned long long v;
    asm volatile("ld.relaxed.cluster.shared::cta.b64 %0, [%1];" : "=l"(v) : "r"(smem_u32(slot)) : "memory");
    return v;
}

// One record per row with everything the objective needs besides the logits.
__global__ void __launch_bounds__(256)
grpo_row_prep_kernel(const RowArgs a, RowPrep* __restrict__ prep) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= a.T) return;
    int tok = a.tokens[t];
    if (tok < 0 || tok >= a.V) { tok = 0; pods_raise(a.status, PODS_STATUS_TOKEN_RANGE); }
    const RowInputs in = load_row_inputs(a, t);
    RowPrep r;
    r.w = in.w;
    r.adv = (float)in.adv;
    r.x_tok = __uint_as_float((uint32_t)a.logits[t * a.ldl + tok] << 16);
    r.old_logp = (float)in.old_logp;
    r.ref_logp = (float)in.ref_logp;
    r.token = tok;
    r.pad = 0;
    prep[t] = r;
}

template <int CL, int IT>
__global__ void __launch_bounds__(kThreads, 2)
grpo_loss_cluster_kernel(const RowArgs a, const int seg_vecs, const int n_stages) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kSlots = slot_count(CL);
    Ctrl<kSlots>& c = *reinterpret_cast<Ctrl<kSlots>*>(smem);
    uint4* const bufs = reinterpret_cast<uint4*>(smem + ctrl_bytes(CL));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_rank();
    const int64_t cluster_id = blockIdx.x / CL, n_clusters = gridDim.x / CL;
    const int nvec = a.V / 8;
    const int seg0 = (int)rank * seg_vecs;                                   // first vector of my segment
    const int cnt = max(0, min(seg_vecs, nvec - seg0));                      // vectors in my segment
    const int stage_vecs = 32 * IT * kConsumerWarps;                         // a stage: IT whole blocks of 32 vectors per warp
    const int64_t n_rows = cluster_id < a.T ? (a.T - cluster_id + n_clusters - 1) / n_clusters : 0;
    const bool has_ref = a.ref_logp != nullptr && a.beta != 0.0f;

    if (tid < 2 * kSlots) (&c.xslot[0][0])[tid] = 0ull;            // tag 0 is no row's tag
    // beyond the segment every stage holds -inf for good, so the sweeps load whole blocks without a bounds
    // test: the copies and the write-back of the exponentials never reach there
    for (int st = 0; st < n_stages; ++st)
        for (int j = cnt + tid; j < stage_vecs; j += kThreads)
            bufs[(size_t)st * stage_vecs + j] = make_uint4(kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair);
    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(&c.full[s], 1);                  // the copy issuer, with the byte count
            mbar_init(&c.done[s], kConsumerWarps);
        }
        for (int p = 0; p < 2; ++p) {
            mbar_init(&c.sumdone[p], kConsumerWarps);
            mbar_init(&c.ready[p], kConsumerWarps);    // the eight lanes that publish a coefficient each
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    cluster_sync();                                    // every slot of the cluster is cleared before anyone writes to it

    bool timed_out = false;

    if (warp == kProducerWarp) {
        // =================================== producer (one thread) ===================================
        if (lane == 0) {
            // issue(i, s): the loads of row i into stage s
            auto issue = [&](int64_t i, int s) {
                const int64_t t = cluster_id + i * n_clusters;
                const uint4* src = reinterpret_cast<const uint4*>(a.logits + t * a.ldl) + seg0;
                if (cnt > 0) {
                    mbar_expect_tx(&c.full[s], (uint32_t)cnt * 16u);
                    uint4* dst = bufs + (size_t)s * stage_vecs;
                    for (int v0 = 0; v0 < cnt; v0 += kPieceVecs)
                        bulk_load(dst + v0, src + v0, (uint32_t)min(kPieceVecs, cnt - v0) * 16u, &c.full[s]);
                } else {
                    mbar_arrive(&c.full[s]);
                }
            };
            const int64_t ahead = n_rows < n_stages ? n_rows : n_stages;
            for (int64_t i = 0; i < ahead; ++i) issue(i, (int)i);
            int s = 0;
            uint32_t parity = 0;
            for (int64_t i = 0; i + n_stages < n_rows; ++i) {
                if (!mbar_wait(&c.done[s], parity, timed_out ? 1u : kSpinLimit)) timed_out = true;
                issue(i + n_stages, s);
                if (++s == n_stages) { s = 0; parity ^= 1u; }
            }
            // a consumer may have given up on a load that is still in flight: every load has to have landed
            // before the CTA ends (the waits return at once when nothing went wrong)
            for (int st = 0; st < n_stages; ++st) {
                const int64_t uses = n_rows > st ? (n_rows - st + n_stages - 1) / n_stages : 0;
                if (uses > 0 && !mbar_wait(&c.full[st], (uint32_t)((uses - 1) & 1), kSpinLimit)) timed_out = true;
            }
        }
        __syncwarp();
    } else if (warp == kExchangeWarp) {
        // =================================== exchange warp ===================================
        const int n_slots = CL * kConsumerWarps;
        const uint4* prep4 = reinterpret_cast<const uint4*>(a.prep);
        // the row's scalar inputs, fetched one row ahead (every lane reads the same two vectors)
        uint4 nx0 = make_uint4(0u, 0u, 0u, 0u), nx1 = nx0;
        if (n_rows > 0) { nx0 = prep4[2 * cluster_id]; nx1 = prep4[2 * cluster_id + 1]; }
        for (int64_t i = 0; i < n_rows; ++i) {
            const uint32_t xp = (uint32_t)(i & 1), xparity = (uint32_t)((i >> 1) & 1);
            const int64_t t = cluster_id + i * n_clusters;
            RowPrep in;
            in.w = __hiloint2double((int)nx0.y, (int)nx0.x);
            in.adv = __uint_as_float(nx0.z);
            in.x_tok = __uint_as_float(nx0.w);
            in.old_logp = __uint_as_float(nx1.x);
            in.ref_logp = __uint_as_float(nx1.y);
            in.token = (int)nx1.z;
            if (i + 1 < n_rows) { nx0 = prep4[2 * (t + n_clusters)]; nx1 = prep4[2 * (t + n_clusters) + 1]; }
            if (!mbar_wait(&c.sumdone[xp], xparity, timed_out ? 1u : kSpinLimit)) timed_out = true;
            // lane l pushes pair (l % 8) of this CTA to peers l / 8, l / 8 + 4, l / 8 + 8, ...
            const unsigned long long tag = (unsigned long long)((i + 1) & 0xffff);
            {
                const int w = lane & 7;
                const Pair mine = c.part[xp][w];
                const unsigned long long word = ((unsigned long long)__float_as_uint(mine.sum) << 32) |
                                                (unsigned long long)(mine.key & 0xffff0000u) | tag;
                for (uint32_t peer = (uint32_t)lane >> 3; peer < (uint32_t)CL; peer += 4)
                    push_word(peer_address(&c.xslot[xp][rank * kConsumerWarps + w], peer), word);
            }
            // lane l collects slots l, l + 32, ...: polls until all carry the row's tag
            constexpr int NW = (CL * kConsumerWarps + 31) / 32;
            unsigned long long word[NW];
            {
                const uint32_t limit = timed_out ? 1u : kSpinLimit;
                uint32_t it = 0;
                for (;;) {
                    bool ok = true;
#pragma unroll
                    for (int q = 0; q < NW; ++q) {
                        word[q] = tag;
                        if (lane + 32 * q < n_slots) word[q] = poll_word(&c.xslot[xp][lane + 32 * q]);
                        ok = ok && (word[q] & 0xffffull) == tag;
                    }
                    if (__all_sync(PODS_FULL_MASK, ok)) break;
                    if (++it >= limit) { timed_out = true; break; }
                }
            }
            // the row maximum; among equal maxima the lowest slot's instance is the one left out of the sums
            uint32_t cand = 0u;
#pragma unroll
            for (int q = 0; q < NW; ++q)
                if (lane + 32 * q < n_slots)
                    cand = max(cand, ((uint32_t)word[q] & 0xffff0000u) | (uint32_t)(0xffff - lane - 32 * q));
            const uint32_t best = __reduce_max_sync(PODS_FULL_MASK, cand);
            const float mx = from_ordered16(best >> 16);
            const int owner_slot = 0xffff - (int)(best & 0xffffu);
            // the exponentials of the scalar terms need only the maximum: three lanes, three calls at once
            const double xr = (double)in.x_tok - (double)mx;                   // <= 0
            // lane 0: rho Z, lane 1: e^d / Z, lane 2: p Z (one call, a different argument per lane)
            const double part = exp(lane == 0 ? xr - (double)in.old_logp : (lane == 1 ? (double)in.ref_logp - xr : xr));
            // sum_w is relative to ref_w: bring it to the row maximum; every slice but the owner's gets back
            // the instance of its own maximum that it left out
            float m_q[NW], scale_q[NW];
            double contrib = 0.0;
#pragma unroll
            for (int q = 0; q < NW; ++q) {
                m_q[q] = from_ordered16((uint32_t)word[q] >> 16);
                scale_q[q] = 0.0f;
                if (lane + 32 * q < n_slots && m_q[q] != -INFINITY) {
                    scale_q[q] = ex2_approx((m_q[q] - mx) * kLog2e);
                    const double tr = (double)__uint_as_float((uint32_t)(word[q] >> 32)) * ref_correction(m_q[q], m_q[q] * kLog2e);
                    contrib += (lane + 32 * q == owner_slot) ? tr : (tr + 1.0) * (double)scale_q[q];
                }
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) contrib += __shfl_xor_sync(PODS_FULL_MASK, contrib, d);
            const double zp = contrib;                                         // Z - 1
            const double Z = 1.0 + zp;
            const double inv_z = 1.0 / Z;
            // the factors of this CTA's own slices: slot rank * 8 + w sits in word (slot / 32) of lane (slot % 32)
            const int my_slot = (int)rank * kConsumerWarps + (lane & 7);
            float my_scale = 0.0f, my_m = 0.0f;
#pragma unroll
            for (int q = 0; q < NW; ++q) {
                const float sc = __shfl_sync(PODS_FULL_MASK, scale_q[q], my_slot & 31);
                const float mm = __shfl_sync(PODS_FULL_MASK, m_q[q], my_slot & 31);
                if ((my_slot >> 5) == q) { my_scale = sc; my_m = mm; }
            }
            const double adv = (double)in.adv;
            const double rho = __shfl_sync(PODS_FULL_MASK, part, 0) * inv_z;
            const double ed = has_ref ? __shfl_sync(PODS_FULL_MASK, part, 1) * Z : 1.0;
            const double pz = __shfl_sync(PODS_FULL_MASK, part, 2);
            // 1 - p: exact route when the target holds the maximum (p may be close to 1), plain otherwise (p < 1/2)
            const double one_minus_p = (in.x_tok == mx) ? zp * inv_z : 1.0 - pz * inv_z;
            const double eps = (double)a.eps, beta = (double)a.beta;
            const double clipped = rho < 1.0 - eps ? 1.0 - eps : (rho > 1.0 + eps ? 1.0 + eps : rho);
            const double t1 = rho * adv, t2 = clipped * adv;
            double dl = (t1 <= t2) ? -adv * rho : 0.0;
            if (has_ref) dl += beta * (1.0 - ed);
            const double g = (in.w != 0.0) ? (double)a.grad_scale * in.w * dl : 0.0;
            if (lane < kConsumerWarps) {
                // e^(x - M) = e_stored * 2^(ref_w - m_w log2e) * e^(m_w - M)
                c.pub[xp].coef[lane] = my_m == -INFINITY ? 0.0f     // a slice of -inf only: its e are all 0
                                       : (float)(-g * inv_z * ref_correction(my_m, my_m * kLog2e) * (double)my_scale);
                if (lane == 0) {
                    c.pub[xp].target = (float)(g * one_minus_p);
                    c.pub[xp].write_mode = (g != 0.0) ? 1 : 0;
                    c.pub[xp].token = in.token;
                }
                mbar_arrive(&c.ready[xp]);
            }
            // ---- nobody waits for these: the log-prob and the row's loss term --------------------------
            if (rank == 0 && lane == 0) {
                const double logp = xr - log1p(zp);
                double loss = -(t1 < t2 ? t1 : t2);
                if (has_ref) {
                    const double d = (double)in.ref_logp - logp;
                    loss += beta * (ed - d - 1.0);
                }
                a.logp[t] = (float)logp;
                a.row_loss[t] = (in.w != 0.0) ? in.w * loss : 0.0;   // a masked row adds nothing, whatever its inputs
            }
            __syncwarp();
        }
    } else {
        // =================================== consumer warps ===================================
        // my slice of the stage: IT blocks of 32 vectors, of which those below hi belong to the segment
        const int lo = warp * 32 * IT, hi = max(lo, min(cnt, lo + 32 * IT));

        // back(i): the gradient of row i over my slice, once the exchange warp has published its factors
        auto back = [&](int64_t i, int s) {
            const uint32_t xp = (uint32_t)(i & 1);
            const uint4* const buf = bufs + (size_t)s * stage_vecs;
            const int64_t t = cluster_id + i * n_clusters;
            uint4* const out = reinterpret_cast<uint4*>(a.dlogits + t * a.ldd) + seg0;
            if (!mbar_wait(&c.ready[xp], (uint32_t)((i >> 1) & 1), timed_out ? 1u : kSpinLimit)) timed_out = true;
            if (c.pub[xp].write_mode == 0) {
                const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int k = 0; k < IT; ++k) {
                    const int j = lo + lane + 32 * k;
                    if (j < hi) __stcs(out + j, z);
                }
            } else {
                const float coef = c.pub[xp].coef[warp];
                const uint16_t hi16 = to_bf16_bits(coef);
                const uint16_t lo16 = to_bf16_bits(coef - __uint_as_float((uint32_t)hi16 << 16));
                const uint32_t c_hi = (uint32_t)hi16 * 0x10001u, c_lo = (uint32_t)lo16 * 0x10001u;
                const int token = c.pub[xp].token;
                const int tok_vec = (token >> 3) - seg0;                        // the vector with the target entry, if it is mine
                const uint16_t target_bits = to_bf16_bits(c.pub[xp].target);
                uint4 q[IT];
#pragma unroll
                for (int k = 0; k < IT; ++k) {
                    const int j = lo + lane + 32 * k;
                    q[k] = buf[j];
                }
#pragma unroll
                for (int k = 0; k < IT; ++k) {
                    const int j = lo + lane + 32 * k;
                    scale_vec(q[k], c_hi, c_lo);
                    if (j < hi && PODS_INDEX_OK(seg0 + j, nvec, a.status) && PODS_INDEX_OK(t, a.T, a.status)) out[j] = q[k];
                }
                // the target entry, if it is in my slice: rewritten by the lane that stored its vector
                if (tok_vec >= lo && tok_vec < hi && ((tok_vec - lo) & 31) == lane)
                    reinterpret_cast<uint16_t*>(out)[(int64_t)tok_vec * 8 + (token & 7)] = target_bits;
            }
            // The stage holds bf16(e) written by these lanes with ordinary stores; the producer refills it with
            // bulk copies, which go through the asynchronous proxy: order the two before handing it back.
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();                              // every lane has its values: the stage may be loaded again
            if (lane == 0) mbar_arrive(&c.done[s]);
        };

        int s = 0, s_prev = 0;
        uint32_t parity = 0;
        for (int64_t i = 0; i < n_rows; ++i) {
            const uint32_t xp = (uint32_t)(i & 1);
            uint4* const buf = bufs + (size_t)s * stage_vecs;

            if (!mbar_wait(&c.full[s], parity, timed_out ? 1u : kSpinLimit)) timed_out = true;

            // ---- my slice into registers; its maximum ------------------------------------------
            uint4 q[IT];
#pragma unroll
            for (int k = 0; k < IT; ++k) {
                const int j = lo + lane + 32 * k;
                q[k] = buf[j];                                      // -inf beyond the segment
            }
            uint32_t pm[4] = {kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair};
#pragma unroll
            for (int k = 0; k < IT; ++k) max_vec(pm, q[k]);
            const uint32_t pmax = max_bf16x2(max_bf16x2(pm[0], pm[1]), max_bf16x2(pm[2], pm[3]));
            const float m_t = fmaxf(bf16_lo(pmax), bf16_hi(pmax)) + 0.0f;             // -0 -> +0
            const uint32_t key_w = __reduce_max_sync(PODS_FULL_MASK, (ordered16(m_t) << 16) | (uint32_t)(31 - lane));
            const float m_w = from_ordered16(key_w >> 16);
            const int owner = 31 - (int)(key_w & 0xffffu);               // lowest lane that holds an instance of m_w
            const float ref_w = m_w == -INFINITY ? 0.0f : m_w * kLog2e;     // a slice of -inf only: every e is 0, not NaN
            // which of the owner's vectors holds it: the first k with that maximum (-1 on every other lane)
            int excl = -1;
            {
                // lane k looks at the owner's k-th vector (still unmodified in shared memory)
                const int j = lo + owner + 32 * lane;
                const bool hit = lane < IT && j < hi && vec_max(buf[j]) == m_w;
                const uint32_t hits = __ballot_sync(PODS_FULL_MASK, hit);
                if (lane == owner && hits != 0u) excl = __ffs(hits) - 1;
            }

            // ---- sum, bf16(e) written back in place ----------------------------------------------
            float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
            for (int k = 0; k < IT; ++k) {
                const int j = lo + lane + 32 * k;
                const float part = (k == excl) ? exp_sum_excluding(q[k], ref_w, m_w) : 0.0f;
                const float sum = exp_vec_inplace(q[k], ref_w);
                if (k & 1) s1 += (k == excl) ? part : sum; else s0 += (k == excl) ? part : sum;
                if (j < hi && PODS_INDEX_OK(j, stage_vecs, a.status)) buf[j] = q[k];
            }
            float sw = s0 + s1;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) sw += __shfl_xor_sync(PODS_FULL_MASK, sw, d);
            if (lane == 0) {
                Pair mine;
                mine.key = key_w & 0xffff0000u;
                mine.sum = sw;
                c.part[xp][warp] = mine;
                mbar_arrive(&c.sumdone[xp]);
            }

            if (i > 0) back(i - 1, s_prev);
            s_prev = s;
            if (++s == n_stages) { s = 0; parity ^= 1u; }
        }
        if (n_rows > 0) back(n_rows - 1, s_prev);
    }
    if (timed_out && lane == 0) pods_raise(a.status, PODS_STATUS_TIMEOUT);
    cluster_sync();                                    // no CTA leaves while a peer may still write its exchange slots
}

// One CTA, one mbarrier that nothing ever arrives on: the wait must give up after `polls` polls and
// report it, and the kernel must end normally.
__global__ void bounded_wait_selftest_kernel(uint32_t polls, uint32_t* status) {
    __shared__ unsigned long long never;
    if (threadIdx.x == 0) mbar_init(&never, 1);
    __syncthreads();
    if (!mbar_wait(&never, 0u, polls) && threadIdx.x == 0) pods_raise(status, PODS_STATUS_TIMEOUT);
}

constexpr size_t kHalfSmBytes = 233472 / 2 - 1024;      // what a CTA may hold for two of them to share an SM

struct ClusterPlan {
    int seg_vecs;        // vectors of a row per CTA
    int it;              // vectors per lane of a consumer warp's slice: the kernel's IT
    int n_stages;
    size_t smem;
};

// Segments, slice depth and ring for a row of nvec vectors over `cl` CTAs.  A stage holds 32 * it vectors
// per consumer warp (4 KB * it).  Three stages (one row being loaded, one in front(), one waiting for
// back()) if two CTAs then still share an SM, else two stages with two CTAs per SM, which beat three
// stages with one CTA per SM by 3 % (measured, V = 155648 .. 196608).  false: does not fit that way.
bool plan_cluster(int nvec, int cl, int min_it, int max_it, ClusterPlan* p) {
    p->seg_vecs = ((nvec + cl - 1) / cl + 7) & ~7;                               // segments start on 128-byte lines of the row
    const int block = 32 * kConsumerWarps;
    p->it = (p->seg_vecs + block - 1) / block;
    if (p->it < min_it) p->it = min_it;
    if (p->it > max_it) return false;
    const size_t stage_bytes = (size_t)p->it * block * 16;
    for (int stages = kMaxStages; stages >= 2; --stages) {
        p->n_stages = stages;
        p->smem = (size_t)ctrl_bytes(cl) + (size_t)stages * stage_bytes;
        if (p->smem <= kHalfSmBytes) return true;
    }
    return false;
}

template <int CL, int IT>
int launch_cluster_it(const RowArgs& a, const ClusterPlan& plan, cudaStream_t stream, bool* launched) {
    auto kernel = grpo_loss_cluster_kernel<CL, IT>;
    PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem));
    if (CL > 8) PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(CL, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int max_clusters = 0;
    PODS_RETURN_IF_CUDA_ERROR(cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg));
    if (max_clusters < 1) return PODS_OK;
    const int64_t n_clusters = a.T < max_clusters ? a.T : max_clusters;
    cfg.gridDim = dim3((unsigned)(n_clusters * CL), 1, 1);
    grpo_row_prep_kernel<<<(unsigned)((a.T + 255) / 256), 256, 0, stream>>>(a, a.prep);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    PODS_RETURN_IF_CUDA_ERROR(cudaLaunchKernelEx(&cfg, kernel, a, plan.seg_vecs, plan.n_stages));
    *launched = true;
    return PODS_OK;
}

// Slice depths each cluster size is instantiated for.  With the full ring and two CTAs per SM a stage holds
// at most 9 blocks per warp (3 x 36 KB + control <= 113 KB), i.e. segments of up to 2304 vectors.  A size
// is only chosen when the size before it does not fit, so its segments are at least that share of 2304
// vectors and its depths start at kMinIt; the largest size goes on to depth 12 on a ring of two stages.
template <int CL> constexpr int kMinIt = CL == 1 ? 1 : CL == 2 ? 5 : (CL == 3 || CL == 4 || CL == 16) ? 7 : CL <= 8 ? 8 : CL == 12 ? 8 : 9;
template <int CL> constexpr int kMaxIt = CL == 16 ? 12 : 9;

template <int CL, int IT>
int launch_cluster_from(const RowArgs& a, const ClusterPlan& plan, cudaStream_t stream, bool* launched) {
    if (plan.it == IT) return launch_cluster_it<CL, IT>(a, plan, stream, launched);
    if constexpr (IT < kMaxIt<CL>) return launch_cluster_from<CL, IT + 1>(a, plan, stream, launched);
    return PODS_OK;
}

// Launches on clusters of CL if the row fits: with the full ring, or (any_ring) with the ring of two as well.
template <int CL>
bool try_cluster(const RowArgs& a, bool any_ring, cudaStream_t stream, bool* launched, int* rc) {
    ClusterPlan plan;
    if (!plan_cluster(a.V / 8, CL, kMinIt<CL>, kMaxIt<CL>, &plan)) return false;
    if (plan.n_stages < kMaxStages && !any_ring) return false;
    *rc = launch_cluster_from<CL, kMinIt<CL>>(a, plan, stream, launched);
    return true;
}

}  // namespace

extern "C" int pods_selftest_bounded_wait(uint32_t polls, uint32_t* status, void* stream) {
    if (status == nullptr || polls == 0 || polls > (1u << 20)) return PODS_ERR_INVALID_ARG;
    bounded_wait_selftest_kernel<<<1, 64, 0, pods_stream(stream)>>>(polls, status);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

// Rows shorter than this go to the row-tile or the general row kernel: per row the cluster path pays a
// fixed price (a pipeline stage and an exchange per row), which very short rows do not repay.  Measured on
// B200 with the cluster size chosen below: 4.4 TB/s at V = 8192 (the row kernel: 3.8), 5.7-6.0 from 12288 on;
// 2.8 at V = 4096, where the row-tile kernel does 3.6.
static int32_t g_cluster_min_vocab = 8192;

extern "C" int32_t pods_set_loss_cluster_min_vocab(int32_t min_vocab) {
    const int32_t v = min_vocab < 2048 ? 2048 : min_vocab;
    return __atomic_exchange_n(&g_cluster_min_vocab, v, __ATOMIC_RELAXED);
}

namespace pods_loss {

// Runs the chunk on the cluster path if the row shape allows it (16-byte aligned rows, V a multiple
// of 8 and large enough to be worth a cluster, segments that fit in shared memory).
int launch_grpo_loss_cluster(const RowArgs& a, cudaStream_t stream, bool* launched) {
    *launched = false;
    if (!a.vec_ok || a.V % 8 != 0 || a.V < __atomic_load_n(&g_cluster_min_vocab, __ATOMIC_RELAXED)) return PODS_OK;
    // as few CTAs per row as leave room for the full ring with two CTAs per SM: fewer partners to exchange
    // with, and small clusters fill the GPU better than large ones (resident CTAs of the 296 slots of a B200,
    // from cudaOccupancyMaxActiveClusters: sizes 1, 2: 296; 3: 279; 4: 284; 5: 280; 6: 270; 7: 259; 8: 264;
    // 9: 270; 10: 260; 11: 231; 12: 252; 13: 221; 14: 196; 15: 210; 16: 224 - hence no 11 and no 13 to 15)
    int rc = PODS_OK;
    if (try_cluster<1>(a, false, stream, launched, &rc) || try_cluster<2>(a, false, stream, launched, &rc) ||
        try_cluster<3>(a, false, stream, launched, &rc) || try_cluster<4>(a, false, stream, launched, &rc) ||
        try_cluster<5>(a, false, stream, launched, &rc) || try_cluster<6>(a, false, stream, launched, &rc) ||
        try_cluster<7>(a, false, stream, launched, &rc) || try_cluster<8>(a, false, stream, launched, &rc) ||
        try_cluster<9>(a, false, stream, launched, &rc) || try_cluster<10>(a, false, stream, launched, &rc) ||
        try_cluster<12>(a, false, stream, launched, &rc) || try_cluster<16>(a, true, stream, launched, &rc))
        return rc;
    return PODS_OK;                                       // rows too long for the register-held slices
}

}  // namespace pods_loss

// pods_select: the down-sampling rule D(o, r; m) -> S (Definition 3.1) for G prompt groups per
// launch, and the advantages of the kept subset (Section 3.2).
//
// Two kernels.  The max-variance and max-reward rules (Algorithm 2; the m highest) run on
// pods_select_fast_kernel, described above its definition: a network sort of bare 32-bit keys, the
// running sums and split scores of Theorem 1's proof in registers, and the kept set read off two
// thresholds.  The random and percentile rules need every element's sorted position and run on
// pods_select_kernel:
//
// One group is handled by LANES consecutive lanes of a warp (8, 16 or 32), each lane holding E
// elements in registers (LANES * E >= n, padded with +infinity keys).  Steps, per group:
//   1. load the rewards (coalesced), build a 64-bit key (order-preserving reward bits or the
//      rollout's Philox word : index) so that one unsigned compare gives the stable order of argsort;
//   2. bitonic sort: strides below E are compare-exchanges between registers of a lane, larger
//      strides exchange with another lane by shuffle;
//   3. fp64 sums of the centred rewards over the kept subset (and the full group);
//   4. kept elements are marked in a bitmap indexed by original index, then written out in
//      ascending original index with a ballot compaction, together with their advantages.

#include <math.h>

#include "pods_common.cuh"

namespace {

constexpr int kSelectWarps = 4;                 // warps per CTA
constexpr int kSelectThreads = kSelectWarps * 32;

// Philox4x32-10 (Salmon et al., SC'11): 10 rounds of two 32x32->64 multiplies and key bumps.
__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                      uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

// fp32 -> uint32 whose unsigned order is the order of the floats; -0 is folded into +0 and every
// NaN becomes the largest key below the padding sentinel.
__device__ __forceinline__ uint32_t ordered_bits(float r) {
    uint32_t u = __float_as_uint(r);
    if ((u << 1) == 0u) u = 0u;                              // -0 -> +0
    if ((u & 0x7fffffffu) > 0x7f800000u) u = 0x7fffffffu;    // any NaN -> one positive NaN
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float from_ordered_bits(uint32_t o) {
    const uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    return __uint_as_float(u);
}

// Shared memory of one group: prefix sums at sorted positions 0..m and suffix sums at positions
// n-m..n of the centred rewards and their squares (fp64), a copy of the rewards (random rule only),
// and two bitmaps (kept original indices, kept sorted positions).
struct SelectSmemLayout {
    int slot_bytes;
    int rbuf_off, sel_off, pos_off;
};

__host__ __device__ inline SelectSmemLayout select_layout(int npad, int m) {
    SelectSmemLayout L;
    const int words = npad >= 32 ? npad / 32 : 1;
    L.rbuf_off = 4 * (m + 1) * 8;
    L.sel_off = L.rbuf_off + npad * 4;
    L.pos_off = L.sel_off + words * 4;
    L.slot_bytes = (L.pos_off + words * 4 + 7) & ~7;
    return L;
}

template <int LANES, int E>
__global__ void __launch_bounds__(kSelectThreads)
pods_select_kernel(const float* __restrict__ rewards, int64_t G, int n, int m, int rule, uint64_t seed,
                   uint32_t flags, int32_t* __restrict__ idx_out, float* __restrict__ adv_out,
                   int32_t* __restrict__ k_out, uint32_t* status) {
    constexpr int NPAD = LANES * E;
    constexpr int GPW = 32 / LANES;                 // groups per warp
    constexpr int WORDS = NPAD >= 32 ? NPAD / 32 : 1;
    constexpr uint32_t GROUP_MASK = LANES == 32 ? 0xffffffffu : ((1u << LANES) - 1u);

    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    const SelectSmemLayout lay = select_layout(NPAD, m);
    unsigned char* slot = smem_raw + (size_t)(warp * GPW + sub) * lay.slot_bytes;
    double* PL1 = reinterpret_cast<double*>(slot);      // sum of the j lowest,  j = 0..m
    double* PL2 = PL1 + (m + 1);
    double* SU1 = PL2 + (m + 1);                        // sum of the m-j highest, j = 0..m
    double* SU2 = SU1 + (m + 1);
    float* rbuf = reinterpret_cast<float*>(slot + lay.rbuf_off);
    uint32_t* sel = reinterpret_cast<uint32_t*>(slot + lay.sel_off);
    uint32_t* possel = reinterpret_cast<uint32_t*>(slot + lay.pos_off);

    const int64_t stride = (int64_t)gridDim.x * kSelectWarps * GPW;
    for (int64_t base = ((int64_t)blockIdx.x * kSelectWarps + warp) * GPW; base < G; base += stride) {
        const int64_t g = base + sub;
        const bool valid = g < G;
        const float* r_g = rewards + (valid ? g : 0) * (int64_t)n;

        // ---- 1. load and key ------------------------------------------------------------------
        uint64_t key[E];
        bool nonfinite = false;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int i = e * LANES + sl;                    // original index (coalesced load)
            key[e] = 0xffffffffffffffffull;                  // padding sorts last
            if (i < n) {
                const float r = valid ? r_g[i] : 0.0f;
                nonfinite |= !(fabsf(r) <= 3.402823466e38f);
                uint32_t hi;
                if (rule == PODS_RULE_RANDOM) {
                    rbuf[i] = r;
                    hi = philox_first_word((uint32_t)i, 0u, (uint32_t)((uint64_t)g & 0xffffffffu),
                                           (uint32_t)((uint64_t)g >> 32), (uint32_t)(seed & 0xffffffffu),
                                           (uint32_t)(seed >> 32));
                } else {
                    hi = ordered_bits(r);
                }
                key[e] = ((uint64_t)hi << 32) | (uint32_t)i;
            }
        }
        if (nonfinite && valid) pods_raise(status, PODS_STATUS_NONFINITE_REWARD);

        // ---- 2. bitonic sort over positions p = sl * E + e ------------------------------------
#pragma unroll
        for (int k = 2; k <= NPAD; k <<= 1) {
#pragma unroll
            for (int j = k >> 1; j > 0; j >>= 1) {
                if (j >= E) {
                    const int lane_xor = j / E;
                    const bool lower = (sl & lane_xor) == 0;
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const bool up = ((sl * E + e) & k) == 0;
                        const uint64_t other = __shfl_xor_sync(PODS_FULL_MASK, key[e], lane_xor);
                        const uint64_t lo = key[e] < other ? key[e] : other;
                        const uint64_t hi = key[e] < other ? other : key[e];
                        key[e] = (lower == up) ? lo : hi;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        if ((e & j) == 0) {
                            const bool up = ((sl * E + e) & k) == 0;
                            const uint64_t a = key[e], b = key[e | j];
                            const uint64_t lo = a < b ? a : b;
                            const uint64_t hi = a < b ? b : a;
                            key[e] = up ? lo : hi;
                            key[e | j] = up ? hi : lo;
                        }
                    }
                }
            }
        }

        // ---- 3. centred rewards and fp64 prefix sums over the sorted order ------------------
        double x[E];
        double centre;
        if (rule == PODS_RULE_RANDOM) {
            __syncwarp();
            centre = (double)rbuf[0];
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const int p = sl * E + e;
                x[e] = p < n ? (double)rbuf[(uint32_t)key[e]] - centre : 0.0;
            }
        } else {
            const uint64_t first = __shfl_sync(PODS_FULL_MASK, key[0], sub * LANES);
            centre = (double)from_ordered_bits((uint32_t)(first >> 32));     // the group minimum
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const int p = sl * E + e;
                x[e] = p < n ? (double)from_ordered_bits((uint32_t)(key[e] >> 32)) - centre : 0.0;
            }
        }

        int kstar = -1;
        if (rule == PODS_RULE_MAXVAR && m < n) {
            double s1 = 0.0, s2 = 0.0;
#pragma unroll
            for (int e = 0; e < E; ++e) { s1 += x[e]; s2 += x[e] * x[e]; }
            double i1 = s1, i2 = s2;                         // inclusive scan over the lanes below
            double j1 = s1, j2 = s2;                         // inclusive scan over the lanes above
#pragma unroll
            for (int d = 1; d < LANES; d <<= 1) {
                const double t1 = __shfl_up_sync(PODS_FULL_MASK, i1, d, LANES);
                const double t2 = __shfl_up_sync(PODS_FULL_MASK, i2, d, LANES);
                const double u1 = __shfl_down_sync(PODS_FULL_MASK, j1, d, LANES);
                const double u2 = __shfl_down_sync(PODS_FULL_MASK, j2, d, LANES);
                if (sl >= d) { i1 += t1; i2 += t2; }
                if (sl + d < LANES) { j1 += u1; j2 += u2; }
            }
            // Both ends are summed directly (lowest upward, highest downward): no split score is a
            // difference of running totals, so equal splits score equal and nothing cancels.
            double a1 = i1 - s1, a2 = i2 - s2;               // sum over positions below this lane's first
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const int p = sl * E + e;
                if (p <= m) { PL1[p] = a1; PL2[p] = a2; }
                a1 += x[e];
                a2 += x[e] * x[e];
            }
            double b1 = j1 - s1, b2 = j2 - s2;               // sum over positions above this lane's last
            if (sl == LANES - 1 && n == NPAD) { SU1[m] = 0.0; SU2[m] = 0.0; }
#pragma unroll
            for (int e = E - 1; e >= 0; --e) {
                const int p = sl * E + e;
                b1 += x[e];
                b2 += x[e] * x[e];
                if (p >= n - m && p <= n) { SU1[p - (n - m)] = b1; SU2[p - (n - m)] = b2; }
            }
            __syncwarp();

            // ---- 4. score the splits: m^2 Var = m * sum x^2 - (sum x)^2 ----------------------
            double best = -INFINITY;
            int bestk = 0x7fffffff;
            for (int k = sl; k <= m; k += LANES) {
                const double q1 = PL1[m - k] + SU1[m - k];
                const double q2 = PL2[m - k] + SU2[m - k];
                // separately rounded products (no fused multiply-add): equal sums give equal scores
                const double score = __dsub_rn(__dmul_rn((double)m, q2), __dmul_rn(q1, q1));
                if (score > best || bestk == 0x7fffffff) { best = score; bestk = k; }
            }
#pragma unroll
            for (int d = LANES >> 1; d > 0; d >>= 1) {
                const double ob = __shfl_xor_sync(PODS_FULL_MASK, best, d);
                const int ok = __shfl_xor_sync(PODS_FULL_MASK, bestk, d);
                if (ok != 0x7fffffff && (bestk == 0x7fffffff || ob > best || (ob == best && ok < bestk))) {
                    best = ob;
                    bestk = ok;
                }
            }
            kstar = __shfl_sync(PODS_FULL_MASK, bestk, sub * LANES);   // one answer per group, even with NaN scores
            __syncwarp();
        } else if (rule == PODS_RULE_MAXVAR) {
            kstar = 0;                                       // m == n: every split is the whole group
        } else if (rule == PODS_RULE_MAXREWARD) {
            kstar = m;
        }

        // ---- 5. mark the kept elements ----------------------------------------------------------
        for (int w = sl; w < WORDS; w += LANES) { sel[w] = 0u; possel[w] = 0u; }
        __syncwarp();
        if (rule == PODS_RULE_PERCENTILE) {
            for (int j = sl; j < m; j += LANES) {
                const int pos = (int)(((2 * (int64_t)j + 1) * n) / (2 * (int64_t)m));
                atomicOr(&possel[pos >> 5], 1u << (pos & 31));
            }
            __syncwarp();
        }
        double s1 = 0.0, s2 = 0.0, f1 = 0.0, f2 = 0.0;      // sums over the kept subset / the full group
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int p = sl * E + e;
            bool keep;
            if (rule == PODS_RULE_PERCENTILE) keep = p < n && ((possel[p >> 5] >> (p & 31)) & 1u);
            else if (rule == PODS_RULE_RANDOM) keep = p < m;
            else keep = p < m - kstar || (p >= n - kstar && p < n);
            if (keep) {
                const uint32_t i = (uint32_t)key[e];
                atomicOr(&sel[i >> 5], 1u << (i & 31));
                s1 += x[e];
                s2 += x[e] * x[e];
            }
            f1 += x[e];
            f2 += x[e] * x[e];
        }
        if (flags & PODS_FLAG_ADV_BEFORE) { s1 = f1; s2 = f2; }
#pragma unroll
        for (int d = LANES >> 1; d > 0; d >>= 1) {
            s1 += __shfl_xor_sync(PODS_FULL_MASK, s1, d);
            s2 += __shfl_xor_sync(PODS_FULL_MASK, s2, d);
        }
        __syncwarp();

        // advantages: a = (x - S/c) / sigma with sigma^2 = (c Q - S^2) / (c d), d = c or c - 1
        const double cnt = (flags & PODS_FLAG_ADV_BEFORE) ? (double)n : (double)m;
        const double den = (flags & PODS_FLAG_STD_SAMPLE) ? cnt - 1.0 : cnt;
        const double J = __dsub_rn(__dmul_rn(cnt, s2), __dmul_rn(s1, s1));
        const double inv_sigma_c = (J > 0.0 && den > 0.0) ? sqrt(den / (cnt * J)) : 0.0;   // 1 / (c sigma)

        // ---- 6. emit in ascending original index ------------------------------------------------
        int written = 0;
        for (int i0 = 0; i0 < n; i0 += LANES) {
            const int i = i0 + sl;
            const bool bit = i < n && ((sel[i >> 5] >> (i & 31)) & 1u);
            const uint32_t ballot = __ballot_sync(PODS_FULL_MASK, bit);
            const uint32_t mine = (ballot >> (sub * LANES)) & GROUP_MASK;
            if (bit && valid) {
                const int off = written + __popc(mine & ((1u << sl) - 1u));
                const double xi = (double)r_g[i] - centre;
                idx_out[g * (int64_t)m + off] = i;
                adv_out[g * (int64_t)m + off] = (float)((xi * cnt - s1) * inv_sigma_c);
            }
            written += __popc(mine);
        }
        if (valid && sl == 0 && k_out != nullptr) k_out[g] = kstar;
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------------------------
// Fast path for the max-variance and max-reward rules: the sort carries 32-bit keys only.
// ---------------------------------------------------------------------------------------------
// Algorithm 2 needs the sorted VALUES (for the running sums and the scores of the m+1 splits), but
// which rollouts are kept follows from two thresholds: the kept set is every reward below v_lo (the
// value at sorted position m-k-1), the first few in index order of those equal to v_lo, every reward
// above v_hi (the value at sorted position n-k), and the last few in index order of those equal to
// v_hi - exactly the set the stable (reward, index) order picks.  So the network sorts bare 32-bit
// keys (one min and one max per compare-exchange, no payload), in the form whose first step of
// every merge level mirrors the block (position p against p ^ (k-1)) so that all steps put the
// minimum at the lower position and no direction has to be selected.
//
// A group is LANES lanes x E register elements.  Registers hold the keys only while they are being
// sorted; the group's keys in original order and in sorted order live in shared memory (rows of E
// words per lane, padded by four words so that 128-bit accesses of a quarter warp fall on distinct
// banks), which lets every later phase pick the distribution of work it needs:
//   sums     Algorithm 2 reads only the m lowest and the m highest sorted positions.  Those 2m values
//            are dealt out evenly, c = ceil(m / LANES) consecutive positions of each end per lane;
//            a lane sums its own, one scan over the group gives what lies below (lowest end) and
//            from it upward (highest end), and the lane then walks its c splits with both running
//            sums in registers: the split "j lowest + (m-j) highest" is scored by the lane that
//            holds sorted position j, no value goes through memory;
//   arg-max  three warp reductions on the order-preserving integer image of the fp64 score
//            (high word, low word, then the largest j, i.e. the smallest k, among equal scores);
//   classify every lane looks at its E rewards in original order and builds four bit masks
//            (below v_lo, equal to it, above v_hi, equal to it); one packed scan over the group
//            turns the counts into the number of ties to keep on either side and into each lane's
//            share of them;
//   emit     kept indices are staged in shared memory in ascending order, then the group's lanes
//            write indices and advantages side by side (consecutive lanes, consecutive addresses).

// reward -> uint32 whose unsigned order is the order of the floats: -0 is folded into +0 by the
// addition, the sign decides between flipping everything and setting the top bit.  NaNs are dealt
// with by the caller (they are rare): every NaN gets the key 0xfffffffe, padding 0xffffffff.
// all-ones for a set top bit, 0 otherwise, as the high half of u * 2 (signed): a multiply on the FMA pipe in place
// of a shift on the integer pipe, which the sort keeps busy (`two` holds an opaque 2)
__device__ __forceinline__ uint32_t top_bit_mask(uint32_t u, uint32_t two) {
    uint32_t r;
    asm("mul.hi.s32 %0, %1, %2;" : "=r"(r) : "r"(u), "r"(two));
    return r;
}
__device__ __forceinline__ uint32_t ordered_key(float r, uint32_t two) {
    const uint32_t u = __float_as_uint(r + 0.0f);
    return u ^ (top_bit_mask(u, two) | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t o, uint32_t two) {
    return __uint_as_float(o ^ (~top_bit_mask(o, two) | 0x80000000u));
}

constexpr uint32_t kKeyNaN = 0xfffffffeu;       // above +inf, below the padding
constexpr uint32_t kKeyPad = 0xffffffffu;
constexpr uint32_t kKeyNegInf = 0x007fffffu;    // ordered_key(-inf): nothing real sorts below it
constexpr uint32_t kKeyPosInf = 0xff800000u;    // ordered_key(+inf)

// order-preserving image of a double (NaNs land above or below everything, which is all they need)
__device__ __forceinline__ unsigned long long ordered_double(double v) {
    const long long b = __double_as_longlong(v);
    return (unsigned long long)b ^ ((unsigned long long)(b >> 63) | 0x8000000000000000ull);
}

// the lowest q set bits of mask (q <= popc(mask)); BITS is the width in use (16 or 32)
template <int BITS>
__device__ __forceinline__ uint32_t lowest_set_bits(uint32_t mask, int q) {
    // L = the largest prefix length whose population is still below q: the q-th set bit is bit L
    int L = 0;
#pragma unroll
    for (int step = BITS / 2; step > 0; step >>= 1) {
        const int t = L + step;
        if (__popc(mask & ((1u << t) - 1u)) < q) L = t;
    }
    const uint32_t upto = L >= 31 ? 0xffffffffu : ((2u << L) - 1u);
    return q > 0 ? (mask & upto) : 0u;
}

// ---- exact arg-max over the splits, for groups whose fp64 scores cannot decide --------------------------------
// A score m sum x^2 - (sum x)^2 of fp32 rewards needs up to ~75 bits; fp64 rounds it, and splits that tie exactly
// in real arithmetic (two kept values a < b: j of a and m-j of b score j (m-j) (b-a)^2, the same for j and m-j)
// come out a few ulps apart unless every sum happens to be exact (dyadic rewards).  When the fp64 scores leave a
// rival within 2^-40 of the best outside the best's own run of identical multisets, the group's scores are
// evaluated again here in double-double arithmetic (two fp64 words, ~106 bits: error-free products by fused
// multiply-add, sums by the branch-free two-sum), and scores closer than 2^-90 relative count as equal: exact for
// rewards whose magnitudes lie within ~2^11 of each other beyond their 24 bits, far below any rounding otherwise.
struct dd { double hi, lo; };
__device__ __forceinline__ dd two_sum(double a, double b) {
    const double s = __dadd_rn(a, b), bb = __dsub_rn(s, a);
    return {s, __dadd_rn(__dsub_rn(a, __dsub_rn(s, bb)), __dsub_rn(b, bb))};
}
__device__ __forceinline__ dd quick_two_sum(double a, double b) {          // |a| >= |b|
    const double s = __dadd_rn(a, b);
    return {s, __dsub_rn(b, __dsub_rn(s, a))};
}
__device__ __forceinline__ dd dd_add(dd x, dd y) {
    dd s = two_sum(x.hi, y.hi);
    const dd t = two_sum(x.lo, y.lo);
    s = quick_two_sum(s.hi, __dadd_rn(s.lo, t.hi));
    return quick_two_sum(s.hi, __dadd_rn(s.lo, t.lo));
}
__device__ __forceinline__ dd dd_sub(dd x, dd y) { return dd_add(x, {-y.hi, -y.lo}); }
__device__ __forceinline__ dd dd_add_d(dd x, double d) { return dd_add(x, {d, 0.0}); }
__device__ __forceinline__ dd dd_square_d(double a) {
    const double p = __dmul_rn(a, a);
    return {p, __fma_rn(a, a, -p)};
}
__device__ __forceinline__ dd dd_mul(dd x, dd y) {
    const double p = __dmul_rn(x.hi, y.hi);
    double e = __fma_rn(x.hi, y.hi, -p);
    e = __fma_rn(x.hi, y.lo, e);
    e = __fma_rn(x.lo, y.hi, e);
    return quick_two_sum(p, e);
}
__device__ __forceinline__ dd dd_mul_d(dd x, double d) {
    const double p = __dmul_rn(x.hi, d);
    return quick_two_sum(p, __fma_rn(x.lo, d, __fma_rn(x.hi, d, -p)));
}
__device__ __forceinline__ dd dd_shfl(dd v, int src) {
    return {__shfl_sync(PODS_FULL_MASK, v.hi, src), __shfl_sync(PODS_FULL_MASK, v.lo, src)};
}
// a >= b up to 2^-90 of the larger: the scores are non-negative up to rounding
__device__ __forceinline__ bool dd_not_below(dd a, dd b) {
    const dd d = dd_sub(a, b);
    const double diff = __dadd_rn(d.hi, d.lo);
    return diff >= -ldexp(fmax(fabs(a.hi), fabs(b.hi)), -90);
}

// Every lane of the warp calls this together.  Returns the exact jstar of the lane's group (the largest j among
// the splits of maximal score) and the sums of x and x^2 over that split's kept subset.
template <int LANES, int LOGE>
__device__ __noinline__ int exact_best_split(const uint32_t* sk, int n, int m, int c, int sub, int sl, uint32_t gmask,
                                             double centre, double* q1_out, double* q2_out) {
    auto at = [](int p) { return p + ((p >> LOGE) << 2); };
    const int j0 = sl * c, mine = max(0, min(c, m - j0)), hi0 = n - m;
    auto x_at = [&](int p) {
        const uint32_t o = sk[at(p)];
        return (double)__uint_as_float(o ^ (~(uint32_t)((int32_t)o >> 31) | 0x80000000u)) - centre;
    };
    dd sb1 = {0.0, 0.0}, sb2 = sb1, st1 = sb1, st2 = sb1;
    for (int i = 0; i < mine; ++i) {
        const double xb = x_at(j0 + i), xt = x_at(hi0 + j0 + i);
        sb1 = dd_add_d(sb1, xb); sb2 = dd_add(sb2, dd_square_d(xb));
        st1 = dd_add_d(st1, xt); st2 = dd_add(st2, dd_square_d(xt));
    }
    dd a1 = sb1, a2 = sb2, b1 = st1, b2 = st2;       // inclusive scans: the lanes below / from mine upward
#pragma unroll
    for (int d = 1; d < LANES; d <<= 1) {
        const int up = (sub * LANES) + max(sl - d, 0), down = (sub * LANES) + min(sl + d, LANES - 1);
        const dd t1 = dd_shfl(a1, up), t2 = dd_shfl(a2, up), u1 = dd_shfl(b1, down), u2 = dd_shfl(b2, down);
        if (sl >= d) { a1 = dd_add(a1, t1); a2 = dd_add(a2, t2); }
        if (sl + d < LANES) { b1 = dd_add(b1, u1); b2 = dd_add(b2, u2); }
    }
    a1 = dd_sub(a1, sb1); a2 = dd_sub(a2, sb2);
    dd best = {0.0, 0.0}, bq1 = best, bq2 = best;
    int bestj = -1;
    auto consider = [&](int j, dd q1, dd q2) {
        const dd score = dd_sub(dd_mul_d(q2, (double)m), dd_mul(q1, q1));
        if (bestj < 0 || dd_not_below(score, best)) {
            // keep the larger of the two as the reference, so that a chain of near-equal scores cannot drift
            if (bestj < 0 || !dd_not_below(best, score)) best = score;
            bestj = j; bq1 = q1; bq2 = q2;
        }
    };
    for (int i = 0; i < mine; ++i) {
        consider(j0 + i, dd_add(a1, b1), dd_add(a2, b2));
        const double xb = x_at(j0 + i), xt = x_at(hi0 + j0 + i);
        a1 = dd_add_d(a1, xb); a2 = dd_add(a2, dd_square_d(xb));
        b1 = dd_add_d(b1, -xt); b2 = dd_sub(b2, dd_square_d(xt));
    }
    if (sl == LANES - 1) consider(m, a1, a2);
    // the group's largest score (by its high word; words below that are inside the tolerance), then every lane
    // whose best is not below it competes with its j
    const unsigned long long ob = ordered_double(best.hi);
    const uint32_t hi = (uint32_t)(ob >> 32), lo = (uint32_t)ob;
    const uint32_t mh = __reduce_max_sync(gmask, bestj >= 0 ? hi : 0u);
    bool cand = bestj >= 0 && hi == mh;
    const uint32_t ml = __reduce_max_sync(gmask, cand ? lo : 0u);
    cand = cand && lo == ml;
    const uint32_t tops = __ballot_sync(PODS_FULL_MASK, cand) & gmask;
    const dd top = dd_shfl(best, tops ? __ffs(tops) - 1 : (sub * LANES));
    const bool in = bestj >= 0 && dd_not_below(best, top);
    const uint32_t mj = __reduce_max_sync(gmask, in ? (uint32_t)(bestj + 1) : 0u);
    const int jstar = mj > 0u ? (int)mj - 1 : m;
    const uint32_t owners = __ballot_sync(PODS_FULL_MASK, in && bestj == jstar) & gmask;
    const int owner = owners ? __ffs(owners) - 1 : (sub * LANES);
    *q1_out = __shfl_sync(PODS_FULL_MASK, bq1.hi, owner);
    *q2_out = __shfl_sync(PODS_FULL_MASK, bq2.hi, owner);
    return jstar;
}

// all-ones when k < v, from the high word of the 64-bit k - v (neg_v = 0 - v as 64 bits): one multiply-add
// on the FMA pipe instead of a compare and a select on the integer pipe, which the sort keeps busy.  `one` is a
// register holding 1 that the compiler cannot see through, so the multiply-add stays one.
__device__ __forceinline__ uint32_t below_mask(uint32_t k, unsigned long long neg_v, uint32_t one) {
    unsigned long long d;
    asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(d) : "r"(k), "r"(one), "l"(neg_v));
    return (uint32_t)(d >> 32);
}
// acc <- 2 acc + h with h = 0 or all-ones (-1): fed the elements from the last to the first, -acc ends up as the
// bit mask of the elements with h = -1 (bit e for element e).  Again a multiply-add (`two` holds an opaque 2).
__device__ __forceinline__ uint32_t push_mask_bit(uint32_t acc, uint32_t h, uint32_t two) {
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(acc), "r"(two), "r"(h));
    return r;
}

// A lane's standing among its own splits: the best score so far with its j and the sums over its kept subset, and
// the best score among its splits that keep another multiset than that best (`run` numbers the runs of identical
// multisets among the lane's splits): a rival the fp64 scores may fail to separate from the winner.
struct SplitBest {
    double best, q1, q2, runner_up;
    int j, run;
};

// m^2 Var = m * sum x^2 - (sum x)^2 of the split "j lowest + (m - j) highest" whose kept subset sums to q1, q2;
// separately rounded products, so that equal sums give equal scores.  The later of two equal scores leads.
template <bool EXACT>
__device__ __forceinline__ void consider_split(SplitBest& s, int jforce, int m, int j, int run, double q1, double q2) {
    const double score = __dsub_rn(__dmul_rn((double)m, q2), __dmul_rn(q1, q1));
    const bool take = jforce < 0 ? (s.j < 0 || score >= s.best) : (j == jforce);
    if (EXACT) {
        const bool other_run = s.j >= 0 && run != s.run;
        const double loser = take ? s.best : score;             // the one of the two that does not lead
        s.runner_up = other_run ? fmax(s.runner_up, loser) : s.runner_up;
    }
    s.best = take ? score : s.best;
    s.q1 = take ? q1 : s.q1;
    s.q2 = take ? q2 : s.q2;
    s.j = take ? j : s.j;
    s.run = take ? run : s.run;
}

// One scan over the group's LANES lanes: (b1, b2) -> the sums of the lanes below; (t1, t2) -> the sums from this
// lane upward.
template <int LANES>
__device__ __forceinline__ void scan_both_ends(int sl, double& b1, double& b2, double& t1, double& t2) {
    const double own1 = b1, own2 = b2;
#pragma unroll
    for (int d = 1; d < LANES; d <<= 1) {
        const double p1 = __shfl_up_sync(PODS_FULL_MASK, b1, d, LANES);
        const double p2 = __shfl_up_sync(PODS_FULL_MASK, b2, d, LANES);
        const double u1 = __shfl_down_sync(PODS_FULL_MASK, t1, d, LANES);
        const double u2 = __shfl_down_sync(PODS_FULL_MASK, t2, d, LANES);
        if (sl >= d) { b1 += p1; b2 += p2; }
        if (sl + d < LANES) { t1 += u1; t2 += u2; }
    }
    b1 -= own1; b2 -= own2;
}

template <int LANES, int E, bool EXACT>
__global__ void __launch_bounds__(kSelectThreads, E >= 32 ? 3 : 8)
pods_select_fast_kernel(const float* __restrict__ rewards, int64_t G, int n, int m, int rule, uint32_t flags,
                        int32_t* __restrict__ idx_out, float* __restrict__ adv_out, int32_t* __restrict__ k_out,
                        uint32_t* status) {
    constexpr int NPAD = LANES * E;
    constexpr int GPW = 32 / LANES;                 // groups per warp
    constexpr int LOGE = E == 4 ? 2 : E == 8 ? 3 : E == 16 ? 4 : 5;
    constexpr int ROWW = E + 4;                     // words of a lane's row in shared memory
    constexpr int GROUPW = LANES * ROWW;            // words of a group
    constexpr uint32_t GROUP_MASK = LANES == 32 ? 0xffffffffu : ((1u << LANES) - 1u);
    constexpr int MASK_BITS = E <= 16 ? 16 : 32;
    static_assert((1 << LOGE) == E, "E is 4, 8, 16 or 32");

    extern __shared__ __align__(16) uint32_t smem_words[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    uint32_t* const ok = smem_words + (size_t)((warp * GPW + sub) * 2) * GROUPW;   // keys in original order
    uint32_t* const sk = ok + GROUPW;                                               // keys in sorted order
    int32_t* const stage = reinterpret_cast<int32_t*>(sk);                         // kept indices (sk is dead by then)
    const uint32_t gmask = GROUP_MASK << (sub * LANES);
    auto at = [](int p) { return p + ((p >> LOGE) << 2); };                         // word of position p in a group
    const bool vec_rows = (n & 3) == 0 && (reinterpret_cast<uintptr_t>(rewards) & 15) == 0;
    const int c = (m + LANES - 1) / LANES;          // sorted positions of each end per lane
    const int nreal = max(0, min(E, n - sl * E));   // my elements that exist
    const uint32_t real_mask = nreal >= 32 ? 0xffffffffu : ((1u << nreal) - 1u);
    const float pad_value = __uint_as_float(0x7fffffffu);       // its key is kKeyPad
    uint32_t one, two;
    asm volatile("mov.u32 %0, 1;" : "=r"(one));
    asm volatile("mov.u32 %0, 2;" : "=r"(two));

    const int64_t stride = (int64_t)gridDim.x * kSelectWarps * GPW;
    for (int64_t base = ((int64_t)blockIdx.x * kSelectWarps + warp) * GPW; base < G; base += stride) {
        const int64_t g = base + sub;
        const bool valid = g < G;
        const float* r_g = rewards + (valid ? g : 0) * (int64_t)n;

        // ---- 1. load and key: lane sl holds original indices sl*E .. sl*E+E-1 -----------------------------
        uint32_t key[E];
        if (vec_rows) {
#pragma unroll
            for (int e = 0; e < E; e += 4) {
                const int i = sl * E + e;
                float4 v = make_float4(pad_value, pad_value, pad_value, pad_value);
                if (i < n) v = valid ? *reinterpret_cast<const float4*>(r_g + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                key[e] = ordered_key(v.x, two);
                key[e + 1] = ordered_key(v.y, two);
                key[e + 2] = ordered_key(v.z, two);
                key[e + 3] = ordered_key(v.w, two);
            }
        } else {
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const int i = sl * E + e;
                key[e] = ordered_key(i < n ? (valid ? r_g[i] : 0.0f) : pad_value, two);
            }
        }
#pragma unroll
        for (int e = 0; e < E; e += 4)
            *reinterpret_cast<uint4*>(ok + sl * ROWW + e) = make_uint4(key[e], key[e + 1], key[e + 2], key[e + 3]);

        // NaNs are not looked for on the way in: after the sort a NaN shows at one end of the order (beyond the
        // infinities); then, and only then, the group's keys are made canonical and sorted once more.
        uint32_t k_min, k_max;
        for (int pass = 0;; ++pass) {
            // ---- 2. bitonic sort of the keys over positions p = sl * E + e ------------------------------
#pragma unroll
            for (int k = 2; k <= NPAD; k <<= 1) {
                // mirror step: p against p ^ (k - 1)
                if (k <= E) {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const int f = e ^ (k - 1);
                        if (e < f) {
                            const uint32_t a = key[e], b = key[f];
                            key[e] = min(a, b);
                            key[f] = max(a, b);
                        }
                    }
                } else {
                    const int lane_xor = (k - 1) / E;                      // k / E - 1: all lane bits below k / E
                    const bool lower = (sl & (k / (2 * E))) == 0;
                    uint32_t other[E];
#pragma unroll
                    for (int e = 0; e < E; ++e) other[e] = __shfl_xor_sync(PODS_FULL_MASK, key[E - 1 - e], lane_xor);
#pragma unroll
                    for (int e = 0; e < E; ++e) key[e] = lower ? min(key[e], other[e]) : max(key[e], other[e]);
                }
                // the remaining steps of the level: p against p ^ j, minimum to the lower position
#pragma unroll
                for (int j = k >> 2; j > 0; j >>= 1) {
                    if (j >= E) {
                        const int lane_xor = j / E;
                        const bool lower = (sl & lane_xor) == 0;
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            const uint32_t other = __shfl_xor_sync(PODS_FULL_MASK, key[e], lane_xor);
                            key[e] = lower ? min(key[e], other) : max(key[e], other);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            if ((e & j) == 0) {
                                const uint32_t a = key[e], b = key[e | j];
                                key[e] = min(a, b);
                                key[e | j] = max(a, b);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < E; e += 4)
                *reinterpret_cast<uint4*>(sk + sl * ROWW + e) = make_uint4(key[e], key[e + 1], key[e + 2], key[e + 3]);
            __syncwarp();
            k_min = sk[0];
            k_max = sk[at(n - 1)];
            const bool stray_nan = k_min < kKeyNegInf || (k_max > kKeyPosInf && k_max != kKeyNaN);
            if (pass == 1 || !__any_sync(PODS_FULL_MASK, stray_nan)) break;
            // rare: every NaN, whatever its sign and payload, gets the one key above +inf; back to the sort
#pragma unroll
            for (int e = 0; e < E; ++e) {
                uint32_t kk = ok[sl * ROWW + e];
                if (e < nreal && (kk > kKeyPosInf || kk < kKeyNegInf)) kk = kKeyNaN;
                ok[sl * ROWW + e] = kk;
                key[e] = kk;
            }
            __syncwarp();
        }

        // ---- 3. fp64 running sums of the centred rewards over the two ends of the sorted order ------------
        const bool nonfinite = k_min <= kKeyNegInf || k_max >= kKeyPosInf;
        if (nonfinite && valid && sl == 0) pods_raise(status, PODS_STATUS_NONFINITE_REWARD);
        const double centre = (double)key_value(k_min, two);                      // the group minimum
        const int j0 = sl * c;                                               // my splits: j0 .. j0 + mine - 1
        const int mine = max(0, min(c, m - j0));
        const int hi0 = n - m;                        // sorted position j is the j-th lowest, hi0 + j the (m-j)-th highest
        // j = number of lowest rewards kept, k = m - j of the highest.  Algorithm 2 starts from k = 0 and replaces
        // only on a strictly larger variance: among equal scores the largest j wins.
        const int jforce = rule == PODS_RULE_MAXREWARD ? 0              // all from the top
                         : (nonfinite || m == n) ? m : -1;              // NaN scores: a scan with '>' stays at k = 0
        SplitBest sb = {0.0, 0.0, 0.0, -INFINITY, -1, -1};
        uint32_t differs = 0u;                        // bit i: splits j0+i and j0+i+1 keep different multisets
        if (c <= 4) {
            // the usual case (m <= 4 LANES): my values stay in registers between the two sweeps
            double xb[4], xt[4];
            double a1 = 0.0, a2 = 0.0, b1 = 0.0, b2 = 0.0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                xb[i] = 0.0; xt[i] = 0.0;
                if (i < mine) {
                    const uint32_t kb = sk[PODS_CLAMPED(at(j0 + i), GROUPW, status)];
                    const uint32_t kt = sk[PODS_CLAMPED(at(PODS_CLAMPED(hi0 + j0 + i, n, status)), GROUPW, status)];
                    differs |= (kb != kt ? 1u : 0u) << i;
                    xb[i] = (double)key_value(kb, two) - centre;
                    xt[i] = (double)key_value(kt, two) - centre;
                }
                a1 += xb[i]; a2 += xb[i] * xb[i];
                b1 += xt[i]; b2 += xt[i] * xt[i];
            }
            // a: the j lowest, summed upward; b: the m-j highest, i.e. what is left of the upper end
            scan_both_ends<LANES>(sl, a1, a2, b1, b2);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (i < mine) consider_split<EXACT>(sb, jforce, m, j0 + i, (EXACT ? __popc(differs & ((1u << i) - 1u)) : 0), a1 + b1, a2 + b2);
                a1 += xb[i]; a2 += xb[i] * xb[i];
                b1 -= xt[i]; b2 -= xt[i] * xt[i];
            }
            if (sl == LANES - 1) consider_split<EXACT>(sb, jforce, m, m, (EXACT ? __popc(differs) : 0), a1, a2);   // the m lowest, none of the highest
        } else {
            double a1 = 0.0, a2 = 0.0, b1 = 0.0, b2 = 0.0;
            for (int i = 0; i < mine; ++i) {
                const uint32_t kb = sk[at(j0 + i)], kt = sk[at(hi0 + j0 + i)];
                differs |= (kb != kt ? 1u : 0u) << i;
                const double xb = (double)key_value(kb, two) - centre;
                const double xt = (double)key_value(kt, two) - centre;
                a1 += xb; a2 += xb * xb;
                b1 += xt; b2 += xt * xt;
            }
            scan_both_ends<LANES>(sl, a1, a2, b1, b2);
            for (int i = 0; i < mine; ++i) {
                consider_split<EXACT>(sb, jforce, m, j0 + i, (EXACT ? __popc(differs & ((1u << i) - 1u)) : 0), a1 + b1, a2 + b2);
                const double xb = (double)key_value(sk[at(j0 + i)], two) - centre;
                const double xt = (double)key_value(sk[at(hi0 + j0 + i)], two) - centre;
                a1 += xb; a2 += xb * xb;
                b1 -= xt; b2 -= xt * xt;
            }
            if (sl == LANES - 1) consider_split<EXACT>(sb, jforce, m, m, (EXACT ? __popc(differs) : 0), a1, a2);
        }
        const double best = sb.best, runner_up = sb.runner_up;
        const int bestj = sb.j;
        double bq1 = sb.q1, bq2 = sb.q2;              // sums over the kept subset of my best split

        // ---- 4. arg-max over the group: largest score, then largest j --------------------------------------
        int jstar;
        {
            const unsigned long long ob = ordered_double(best);
            const uint32_t hi = (uint32_t)(ob >> 32), lo = (uint32_t)ob;
            const uint32_t mh = __reduce_max_sync(gmask, bestj >= 0 ? hi : 0u);
            bool cand = bestj >= 0 && hi == mh;
            const uint32_t ml = __reduce_max_sync(gmask, cand ? lo : 0u);
            cand = cand && lo == ml;
            const uint32_t mj = __reduce_max_sync(gmask, cand ? (uint32_t)(bestj + 1) : 0u);
            jstar = mj > 0u ? (int)mj - 1 : m;
            const uint32_t owners = __ballot_sync(PODS_FULL_MASK, cand && bestj == jstar) & gmask;
            const int owner = owners ? __ffs(owners) - 1 : lane;
            bq1 = __shfl_sync(PODS_FULL_MASK, bq1, owner);
            bq2 = __shfl_sync(PODS_FULL_MASK, bq2, owner);
            const double best_all = __shfl_sync(PODS_FULL_MASK, best, owner);
            // Split j+1 swaps the (m-j)-th highest reward for the (j+1)-th lowest; when the two are equal both
            // splits keep the same multiset of rewards and tie exactly, whatever rounding did to their fp64
            // scores.  Algorithm 2 keeps the smallest k, i.e. the largest j, of such a run: move up to its end.
            bool rival = false;
            if (jforce < 0) {
                // the run of splits around jstar that keep one and the same multiset
                auto run_of = [&](int j, int& lo, int& hi, bool want_lo) {
                    const int from = j - j0;                                  // my positions from here on lie ahead
                    const uint32_t below = from >= 32 ? 0xffffffffu : (from <= 0 ? 0u : (1u << from) - 1u);
                    const uint32_t ahead = differs & ~below, behind = differs & below;
                    const uint32_t stop = ahead != 0u ? (uint32_t)(j0 + __ffs(ahead) - 1) : (uint32_t)m;
                    hi = max(j, (int)__reduce_min_sync(gmask, stop));
                    if (want_lo) {
                        const uint32_t start = behind != 0u ? (uint32_t)(j0 + 32 - __clz(behind)) : 0u;
                        lo = (int)__reduce_max_sync(gmask, start);
                    }
                };
                int run_lo = 0, run_hi;
                run_of(jstar, run_lo, run_hi, EXACT);
                jstar = run_hi;
                if (EXACT) {
                    // a rival outside that run whose fp64 score is within 2^-40 of the best: fp64 cannot tell a tie
                    // from a win there, the exact evaluation has to.  My best if it lies outside the winner's run,
                    // and my runner-up (outside my best's run, hence outside the winner's whenever my best is inside)
                    const double near = best_all - fabs(best_all) * 9.094947017729282e-13;
                    rival = (bestj >= 0 && (bestj < run_lo || bestj > run_hi) && best >= near) || runner_up >= near;
                    if (c > 4) rival = true;           // long ends (m > 4 LANES): always settled exactly
                } else if (run_hi >= 1 && run_hi <= m - 1) {
                    // The one other tie that holds for any values: a kept subset of just two values a < b, j of a and
                    // m-j of b, scores j (m-j) (b-a)^2, the same as its mirror image (m-j of a, j of b).  fp64 rounds
                    // the two differently unless the sums are exact; when the mirror image of the run is a split
                    // too and lies above it, that one is the smaller k.
                    const uint32_t ka = sk[0], kb2 = sk[at(n - 1)];
                    const int jm = m - run_hi;                                 // as many of a as there were of b
                    const bool two_valued = ka != kb2 && sk[at(run_hi - 1)] == ka && (run_hi == m || sk[at(hi0 + run_hi)] == kb2);
                    const bool mirrored = jm > run_hi && sk[at(jm - 1)] == ka && (jm == m || sk[at(hi0 + jm)] == kb2);
                    if (two_valued && mirrored) {      // per group; the reductions below use the group's own mask
                        // the kept sums follow from the counts: x = 0 for a (the minimum), d = b - a for the others
                        const double d = (double)key_value(kb2, two) - centre, cntb = (double)run_hi;
                        run_of(jm, run_lo, run_hi, false);
                        jstar = run_hi;
                        bq1 = cntb * d;
                        bq2 = cntb * d * d;
                    }
                }
            }
            if (EXACT) {
                if (__any_sync(PODS_FULL_MASK, rival)) {   // every lane of the warp goes; only the groups concerned listen
                    double e1, e2;
                    const int jexact = exact_best_split<LANES, LOGE>(sk, n, m, c, sub, sl, gmask, centre, &e1, &e2);
                    if (__ballot_sync(PODS_FULL_MASK, rival) & gmask) { jstar = jexact; bq1 = e1; bq2 = e2; }
                }
            }
        }
        const int nlo = jstar, nhi = m - jstar;
        const int kstar = nhi;

        // sums over the whole group, for the "Before" normalisation only
        double s1 = bq1, s2 = bq2;
        if (flags & PODS_FLAG_ADV_BEFORE) {
            double f1 = 0.0, f2 = 0.0;
#pragma unroll 4
            for (int e = 0; e < E; ++e) {
                if (e < nreal) {
                    const double x = (double)key_value(sk[sl * ROWW + e], two) - centre;
                    f1 += x; f2 += x * x;
                }
            }
#pragma unroll
            for (int d = LANES >> 1; d > 0; d >>= 1) {
                f1 += __shfl_xor_sync(PODS_FULL_MASK, f1, d);
                f2 += __shfl_xor_sync(PODS_FULL_MASK, f2, d);
            }
            s1 = f1; s2 = f2;
        }

        // ---- 5. the two thresholds; my rewards in original order against them ---------------------------
        // keys of real rewards lie in [1, 0xfffffffe]: 0 and 0xffffffff match nothing when an end is empty
        const uint32_t v_lo = nlo > 0 ? sk[at(PODS_CLAMPED(nlo - 1, n, status))] : 0u;
        const uint32_t v_hi = nhi > 0 ? sk[at(PODS_CLAMPED(n - nhi, n, status))] : kKeyPad;
        // a run of equal rewards is cut when the sorted neighbour just outside a kept end has the end's value
        const bool cut = (nlo > 0 && nlo < n && sk[at(nlo)] == v_lo) || (nhi > 0 && nhi < n && sk[at(n - nhi - 1)] == v_hi);
        __syncwarp();                                    // sk has been read for the last time: it becomes `stage`
        uint32_t take = 0u;
        if (!__any_sync(PODS_FULL_MASK, cut)) {
            // no run is cut anywhere in the warp: everything up to v_lo and everything from v_hi on is kept
            const unsigned long long neg_le = 0ull - (unsigned long long)v_lo - 1ull, neg_hi = 0ull - (unsigned long long)v_hi;
            uint32_t a_le = 0u, a_lth = 0u;                     // minus the masks "up to v_lo" and "below v_hi"
#pragma unroll
            for (int e = E - 4; e >= 0; e -= 4) {
                const uint4 q = *reinterpret_cast<const uint4*>(ok + sl * ROWW + e);
                const uint32_t kk[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int t = 3; t >= 0; --t) {
                    a_le = push_mask_bit(a_le, below_mask(kk[t], neg_le, one), two);
                    a_lth = push_mask_bit(a_lth, below_mask(kk[t], neg_hi, one), two);
                }
            }
            take = ((0u - a_le) | ~(0u - a_lth)) & real_mask;
        } else {
            // four masks over my rewards: below v_lo, up to v_lo, below v_hi, up to v_hi (all on the FMA pipe)
            const unsigned long long neg_lo = 0ull - (unsigned long long)v_lo, neg_hi = 0ull - (unsigned long long)v_hi;
            uint32_t m_lt = 0u, m_le = 0u, m_lth = 0u, m_leh = 0u;
#pragma unroll
            for (int e = E - 4; e >= 0; e -= 4) {
                const uint4 q = *reinterpret_cast<const uint4*>(ok + sl * ROWW + e);
                const uint32_t kk[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int t = 3; t >= 0; --t) {
                    m_lt = push_mask_bit(m_lt, below_mask(kk[t], neg_lo, one), two);
                    m_le = push_mask_bit(m_le, below_mask(kk[t], neg_lo - 1ull, one), two);
                    m_lth = push_mask_bit(m_lth, below_mask(kk[t], neg_hi, one), two);
                    m_leh = push_mask_bit(m_leh, below_mask(kk[t], neg_hi - 1ull, one), two);
                }
            }
            m_lt = (0u - m_lt) & real_mask; m_le = 0u - m_le; m_lth = 0u - m_lth; m_leh = 0u - m_leh;
            const uint32_t m_el = m_le & ~m_lt & real_mask;              // equal to v_lo
            const uint32_t m_gt = ~m_leh & real_mask;                    // above v_hi
            const uint32_t m_eh = m_leh & ~m_lth & real_mask;            // equal to v_hi
            const int c_el = __popc(m_el), c_eh = __popc(m_eh);
            // four counts of up to 1024 in one word: below v_lo | above v_hi << 11 | equal v_lo << 22 | equal v_hi << 33
            const unsigned long long packed = (unsigned long long)__popc(m_lt) | ((unsigned long long)__popc(m_gt) << 11) |
                                              ((unsigned long long)c_el << 22) | ((unsigned long long)c_eh << 33);
            unsigned long long incl = packed;
#pragma unroll
            for (int d = 1; d < LANES; d <<= 1) {
                const unsigned long long t = __shfl_up_sync(PODS_FULL_MASK, incl, d, LANES);
                if (sl >= d) incl += t;
            }
            const unsigned long long total = __shfl_sync(PODS_FULL_MASK, incl, sub * LANES + LANES - 1);
            const unsigned long long before = incl - packed;
            const int need_lo = nlo - (int)(total & 2047);                        // rewards equal to v_lo to keep: the first by index
            const int need_hi = nhi - (int)((total >> 11) & 2047);                // rewards equal to v_hi to keep: the last by index
            const int skip_hi = (int)((total >> 33) & 2047) - need_hi;            // ... i.e. all but the first skip_hi of them
            const int q_lo = max(0, min(c_el, need_lo - (int)((before >> 22) & 2047)));   // of mine equal to v_lo: keep the first q_lo
            const int q_hi = max(0, min(c_eh, skip_hi - (int)((before >> 33) & 2047)));   // of mine equal to v_hi: drop the first q_hi
            uint32_t keep_lo = q_lo == c_el ? m_el : 0u, drop_hi = q_hi == c_eh ? m_eh : 0u;
            if (__any_sync(PODS_FULL_MASK, (q_lo != 0 && q_lo != c_el) || (q_hi != 0 && q_hi != c_eh))) {
                keep_lo = lowest_set_bits<MASK_BITS>(m_el, q_lo);                 // the cut falls inside some lane
                drop_hi = lowest_set_bits<MASK_BITS>(m_eh, q_hi);
            }
            take = m_lt | m_gt | keep_lo | (m_eh & ~drop_hi);
        }

        // ---- 6. kept indices in ascending order, then indices and advantages side by side -------------------
        const int my_takes = __popc(take);
        int off = my_takes;
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) {
            const int t = __shfl_up_sync(PODS_FULL_MASK, off, d, LANES);
            if (sl >= d) off += t;
        }
        off -= my_takes;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (((take >> e) & 1u) && PODS_INDEX_OK(off, m, status)) stage[off++] = sl * E + e;
        }
        __syncwarp();

        // advantages: a = (x - S/c) / sigma with sigma^2 = (c Q - S^2) / (c d), d = c or c - 1
        const double cnt = (flags & PODS_FLAG_ADV_BEFORE) ? (double)n : (double)m;
        const double den = (flags & PODS_FLAG_STD_SAMPLE) ? cnt - 1.0 : cnt;
        const double J = __dsub_rn(__dmul_rn(cnt, s2), __dmul_rn(s1, s1));
        const double inv_sigma_c = (J > 0.0 && den > 0.0) ? sqrt(den / (cnt * J)) : 0.0;   // 1 / (c sigma)
        if (valid) {
            int32_t* io = idx_out + g * (int64_t)m;
            float* ao = adv_out + g * (int64_t)m;
            for (int j = sl; j < m; j += LANES) {
                const int i = stage[j] & (NPAD - 1);
                const double xi = (double)key_value(ok[at(PODS_CLAMPED(i, n, status))], two) - centre;
                if (PODS_INDEX_OK(stage[j], n, status) && PODS_INDEX_OK(g * (int64_t)m + j, G * (int64_t)m, status)) {
                    io[j] = i;
                    ao[j] = (float)((xi * cnt - s1) * inv_sigma_c);
                }
            }
            if (sl == 0 && k_out != nullptr) k_out[g] = kstar;
        }
        __syncwarp();                                    // ok and stage are rewritten by the next group
    }
}

template <int LANES, int E>
int launch_select_fast(const float* rewards, int64_t G, int n, int m, int rule, uint32_t flags, int32_t* idx,
                       float* adv, int32_t* k_out, uint32_t* status, cudaStream_t stream) {
    constexpr int GPW = 32 / LANES;
    // per group: its keys in original and in sorted order, rows of E + 4 words per lane
    const size_t smem = (size_t)kSelectWarps * GPW * 2 * LANES * (E + 4) * sizeof(uint32_t);
    auto kernel = (flags & PODS_FLAG_EXACT_TIES) ? pods_select_fast_kernel<LANES, E, true> : pods_select_fast_kernel<LANES, E, false>;
    if (smem > 48 * 1024)
        PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t groups_per_cta = (int64_t)kSelectWarps * GPW;
    const int64_t needed = (G + groups_per_cta - 1) / groups_per_cta;
    const int64_t cap = (int64_t)pods_sm_count() * 16;
    const int grid = (int)(needed < cap ? needed : cap);
    kernel<<<grid, kSelectThreads, smem, stream>>>(rewards, G, n, m, rule, flags, idx, adv, k_out, status);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

template <int LANES, int E>
int launch_select(const float* rewards, int64_t G, int n, int m, int rule, uint64_t seed, uint32_t flags,
                  int32_t* idx, float* adv, int32_t* k_out, uint32_t* status, cudaStream_t stream) {
    constexpr int GPW = 32 / LANES;
    const SelectSmemLayout lay = select_layout(LANES * E, m);
    const size_t smem = (size_t)lay.slot_bytes * kSelectWarps * GPW;
    auto kernel = pods_select_kernel<LANES, E>;
    if (smem > 48 * 1024)
        PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t groups_per_cta = (int64_t)kSelectWarps * GPW;
    const int64_t needed = (G + groups_per_cta - 1) / groups_per_cta;
    const int64_t cap = (int64_t)pods_sm_count() * 16;
    const int grid = (int)(needed < cap ? needed : cap);
    kernel<<<grid, kSelectThreads, smem, stream>>>(rewards, G, n, m, rule, seed, flags, idx, adv, k_out, status);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

}  // namespace

extern "C" int pods_select(const float* rewards, int64_t G, int32_t n, int32_t m, int32_t rule, uint64_t seed,
                           uint32_t flags, int32_t* idx, float* adv, int32_t* k_out, uint32_t* status,
                           void* stream) {
    if (G < 0 || n < 1 || m < 1 || m > n) return PODS_ERR_INVALID_ARG;
    if (rule < PODS_RULE_MAXVAR || rule > PODS_RULE_PERCENTILE) return PODS_ERR_UNSUPPORTED;
    if (n > PODS_MAX_N) return PODS_ERR_UNSUPPORTED;
    if (G == 0) return PODS_OK;
    if (rewards == nullptr || idx == nullptr || adv == nullptr) return PODS_ERR_INVALID_ARG;
    if (!pods_aligned(rewards, 4) || !pods_aligned(idx, 4) || !pods_aligned(adv, 4)) return PODS_ERR_INVALID_ARG;
    cudaStream_t s = pods_stream(stream);
    if (rule == PODS_RULE_MAXVAR || rule == PODS_RULE_MAXREWARD) {
#define PODS_SELECT_FAST(LANES, E) \
    return launch_select_fast<LANES, E>(rewards, G, n, m, rule, flags, idx, adv, k_out, status, s)
        // as many elements per lane as registers allow (16): compare-exchanges between registers cost one
        // instruction per element, those between lanes a shuffle more, and the per-group scans get shorter
        if (n <= 8) PODS_SELECT_FAST(2, 4);
        if (n <= 16) PODS_SELECT_FAST(2, 8);
        if (n <= 32) PODS_SELECT_FAST(2, 16);
        if (n <= 64) PODS_SELECT_FAST(4, 16);
        if (n <= 128) PODS_SELECT_FAST(8, 16);
        if (n <= 256) PODS_SELECT_FAST(16, 16);
        if (n <= 512) PODS_SELECT_FAST(32, 16);
        PODS_SELECT_FAST(32, 32);
#undef PODS_SELECT_FAST
    }
#define PODS_SELECT_CASE(LANES, E) \
    return launch_select<LANES, E>(rewards, G, n, m, rule, seed, flags, idx, adv, k_out, status, s)
    if (n <= 8) PODS_SELECT_CASE(8, 1);
    if (n <= 16) PODS_SELECT_CASE(16, 1);
    if (n <= 32) PODS_SELECT_CASE(32, 1);
    if (n <= 64) PODS_SELECT_CASE(32, 2);
    if (n <= 128) PODS_SELECT_CASE(32, 4);
    if (n <= 256) PODS_SELECT_CASE(32, 8);
    if (n <= 512) PODS_SELECT_CASE(32, 16);
    PODS_SELECT_CASE(32, 32);
#undef PODS_SELECT_CASE
}

// Device helpers shared by the GRPO-PODS loss kernels: bf16 packing, the exponential, the row
// arguments and the scalar (per-row, fp64) part of the objective of Section 3.2.
#pragma once

#include <cuda_bf16.h>
#include <math.h>

#include "pods_common.cuh"

namespace pods_loss {

constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kNegInfPair = 0xff80ff80u;     // two bf16 -inf: neutral for max, adds 0 to a sum of 2^x

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint16_t to_bf16_bits(float v) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
}

// 2^(-lo) for lo = M*log2e - fl(M*log2e), |lo| < 2^-18: first-order expansion, fp64.
__device__ __forceinline__ double ref_correction(float mx, float mxc) {
    return 1.0 - (double)fmaf(mx, kLog2e, -mxc) * 0.6931471805599453;
}

__device__ __forceinline__ float vec_max(const uint4& q) {
    const uint32_t w = max_bf16x2(max_bf16x2(q.x, q.y), max_bf16x2(q.z, q.w));
    return fmaxf(bf16_lo(w), bf16_hi(w));
}

// Replace element e (0..7) of a packed vector of eight bf16 values.
__device__ __forceinline__ void patch_bf16(uint4& o, int e, uint16_t bits) {
    const uint32_t shift = (e & 1) ? 16u : 0u;
    const uint32_t keep = ~(0xffffu << shift), put = (uint32_t)bits << shift;
    const int w = e >> 1;
    o.x = w == 0 ? (o.x & keep) | put : o.x;
    o.y = w == 1 ? (o.y & keep) | put : o.y;
    o.z = w == 2 ? (o.z & keep) | put : o.z;
    o.w = w == 3 ? (o.w & keep) | put : o.w;
}

// Order-preserving key of (value, position): larger value first, then smaller position.
__device__ __forceinline__ unsigned long long argmax_key(float v, int pos) {
    uint32_t u = __float_as_uint(v + 0.0f);                        // -0 -> +0
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (uint32_t)(0x7fffffff - pos);
}
__device__ __forceinline__ float argmax_key_value(unsigned long long k) {
    const uint32_t o = (uint32_t)(k >> 32);
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}
__device__ __forceinline__ int argmax_key_pos(unsigned long long k) {
    return 0x7fffffff - (int)(uint32_t)(k & 0xffffffffu);
}

// ---- pieces of the register-held sweeps shared by the cluster-resident and the row-tile kernels ----

// bf16 value (as fp32, -0 already folded into +0) -> 16-bit key whose unsigned order is the order of the values.
__device__ __forceinline__ uint32_t ordered16(float v) {
    const uint32_t u = __float_as_uint(v) >> 16;
    return (u & 0x8000u) ? (~u & 0xffffu) : (u | 0x8000u);
}
__device__ __forceinline__ float from_ordered16(uint32_t o) {
    const uint32_t u = (o & 0x8000u) ? (o & 0x7fffu) : (~o & 0xffffu);
    return __uint_as_float(u << 16);
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
static __device__ __noinline__ float exp_sum_excluding(uint4 q, float ref, float mx) {
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
__device__ __forceinline__ void scale_vec(uint4& q, uint32_t c_hi, uint32_t c_lo) {
    q.x = scale_bf16x2(q.x, c_hi, c_lo);
    q.y = scale_bf16x2(q.y, c_hi, c_lo);
    q.z = scale_bf16x2(q.z, c_hi, c_lo);
    q.w = scale_bf16x2(q.w, c_hi, c_lo);
}

__device__ __forceinline__ void max_vec(uint32_t (&pm)[4], const uint4& q) {
    pm[0] = max_bf16x2(pm[0], q.x);
    pm[1] = max_bf16x2(pm[1], q.y);
    pm[2] = max_bf16x2(pm[2], q.z);
    pm[3] = max_bf16x2(pm[3], q.w);
}

// Everything the objective needs for one row besides the logits, gathered by the cluster path's
// preparation kernel: 32 bytes, read as two 16-byte vectors.
struct __align__(16) RowPrep {
    double w;            // mask_t / (M |o_i|)
    float adv, x_tok;    // advantage of the row's rollout; the target's logit
    float old_logp, ref_logp;
    int token;
    int pad;
};

struct RowArgs {
    const uint16_t* logits;
    int64_t ldl;
    const int32_t* tokens;
    const float* old_logp;
    const float* ref_logp;
    const float* adv;
    const double* seq_weight;
    const int64_t* cu_seqlens;
    int64_t M;
    int64_t row0;
    const uint8_t* mask;
    int64_t T;
    int32_t V;
    float eps, beta, grad_scale;
    float* logp;
    uint16_t* dlogits;
    int64_t ldd;
    double* row_loss;      // workspace [T]: mask_t w_i loss_t
    RowPrep* prep;         // workspace [T]: the rows' scalar inputs (cluster path)
    uint32_t* status;
    int vec_ok;            // 16-byte aligned rows: 128-bit path
    int precise;           // small chunk: the sum of exponentials is also taken in fp64 (see exact_sum_threshold)
};

// Chunks of at most this many logits are bound by launch latency, not by bandwidth: there the row-tile and
// the general row kernel also take the sum of exponentials in fp64 with the library exponential, so that the
// log-probs carry fp64 accuracy and a loss that is a nearly cancelling sum of rollout terms (zero-sum
// advantages) keeps its relative accuracy.  The gradient rows are the same either way.
constexpr int64_t kExactSumMaxLogits = 1 << 20;

// Sum over a vector's eight values of e^(x - mx) in fp64; `skip_first_max` leaves out the first value equal to mx.
static __device__ __noinline__ double exact_exp_sum(uint4 q, float mx, bool skip_first_max) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    double s = 0.0;
    bool skipped = !skip_first_max;
#pragma unroll 1
    for (int i = 0; i < 8; ++i) {
        const uint32_t word = w[i >> 1];
        const float v = (i & 1) ? bf16_hi(word) : bf16_lo(word);
        const bool skip = !skipped && v == mx;
        skipped |= skip;
        if (!skip && v != -INFINITY) s += exp((double)v - (double)mx);
    }
    return s;
}

// Rollout of packed row r: the i with cu_seqlens[i] <= r < cu_seqlens[i+1].
__device__ __forceinline__ int64_t find_rollout(const int64_t* cu, int64_t M, int64_t r) {
    int64_t lo = 0, hi = M;            // invariant: cu[lo] <= r, answer in [lo, hi)
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (cu[mid] <= r) lo = mid; else hi = mid;
    }
    return lo;
}

// The inputs of one row that do not depend on its logits.
struct RowInputs {
    double w;        // mask_t / (M |o_i|)
    double adv;
    double old_logp;
    double ref_logp;
    int has_ref;
};

__device__ __forceinline__ RowInputs load_row_inputs(const RowArgs& a, int64_t t) {
    RowInputs in;
    const int64_t i = find_rollout(a.cu_seqlens, a.M, a.row0 + t);
    const bool live = a.mask == nullptr || a.mask[t] != 0;
    in.w = live ? a.seq_weight[i] : 0.0;
    in.adv = (double)a.adv[i];
    in.old_logp = (double)a.old_logp[t];
    in.has_ref = a.ref_logp != nullptr && a.beta != 0.0f;
    in.ref_logp = in.has_ref ? (double)a.ref_logp[t] : 0.0;
    return in;
}

// The token term of the objective (Section 3.2) from the token's log-prob, fp64:
//   rho = exp(logp - old),  loss = -min(rho a, clip(rho) a) + beta kl,  g = grad_scale w dloss/dlogp.
struct TokenTerms {
    double weighted_loss, g;
};

__device__ __forceinline__ TokenTerms token_terms(double logp, const RowInputs& in, float eps_f, float beta_f,
                                                  float grad_scale) {
    TokenTerms r;
    const double eps = (double)eps_f, beta = (double)beta_f;
    const double rho = exp(logp - in.old_logp);
    const double clipped = rho < 1.0 - eps ? 1.0 - eps : (rho > 1.0 + eps ? 1.0 + eps : rho);
    const double s1 = rho * in.adv, s2 = clipped * in.adv;
    double loss = -(s1 < s2 ? s1 : s2);
    double dl = (s1 <= s2) ? -in.adv * rho : 0.0;
    if (in.has_ref) {
        const double d = in.ref_logp - logp;
        const double ed = exp(d);
        loss += beta * (ed - d - 1.0);
        dl += beta * (1.0 - ed);
    }
    r.g = (in.w != 0.0) ? (double)grad_scale * in.w * dl : 0.0;
    r.weighted_loss = (in.w != 0.0) ? in.w * loss : 0.0;     // a masked row adds nothing, whatever its inputs
    return r;
}

// The scalar part of the objective for one row of logits:
//   logp = (x_tok - M) - log(1 + Z'),  the token's terms,  1 - p accurate even when p -> 1.
struct RowScalars {
    double logp, weighted_loss, g, one_minus_p, Z;
};

__device__ __forceinline__ RowScalars row_scalars(const RowArgs& a, const RowInputs& in, float x_tok, float mx,
                                                  double zp) {
    RowScalars r;
    r.Z = 1.0 + zp;
    r.logp = ((double)x_tok - (double)mx) - log1p(zp);
    const TokenTerms tt = token_terms(r.logp, in, a.eps, a.beta, a.grad_scale);
    r.g = tt.g;
    r.weighted_loss = tt.weighted_loss;
    r.one_minus_p = (x_tok == mx) ? zp / r.Z : -expm1(r.logp);
    return r;
}

// grpo_loss.cu: fixed-order sum of per-row loss terms, added to *loss_acc (one CTA).
int launch_loss_reduce(const double* row_loss, int64_t T, double* loss_acc, cudaStream_t stream);

// grpo_loss_cluster.cu: runs the rows on the cluster-resident path when their shape allows it.
int launch_grpo_loss_cluster(const RowArgs& a, cudaStream_t stream, bool* launched);

}  // namespace pods_loss

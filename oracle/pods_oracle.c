/*
 * CPU oracle for the PODS hot path (arxiv 2504.13818).  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, readable implementation of what the CUDA library computes,
 * written from the paper so that a reader can check it against the text:
 *
 *   oracle_select      Algorithm 2 (max-variance down-sampling) with the prefix
 *                      sums of Theorem 1's proof, the three baseline rules of
 *                      Section 3.2, and the advantages a_{S,i} of Section 3.2
 *                      (or the full-group statistics of Appendix A.3, "Before").
 *   oracle_seq_weights 1/(M |o_i|) of the L_PODS formula, Section 3.2.
 *   oracle_grpo_rows   per-token terms of L_PODS (Section 3.2) with a KL penalty
 *                      (Table 2 "KL Coefficient"), and the gradient w.r.t. logits.
 *   oracle_grpo_loss   the two outer sums of L_PODS, in the paper's order.
 *
 * Nothing here is shared with the CUDA path: no headers, tables, helpers or
 * generators.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may load this file; the product never routes through it.
 *
 * Precision: fp64 throughout; the split scores of Algorithm 2 are evaluated in
 * __float128 on rewards centred on the group minimum so that ties between
 * splits are decided as in real arithmetic for fp32 inputs of ordinary range.
 * OpenMP parallelises over independent groups / rows only; there is no blocking,
 * fusion or reordering inside a group or a row.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef __float128 quad;

enum { RULE_MAXVAR = 0, RULE_MAXREWARD = 1, RULE_RANDOM = 2, RULE_PERCENTILE = 3 };
enum { FLAG_ADV_BEFORE = 1u, FLAG_STD_SAMPLE = 2u };

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as   */
/* easy as 1, 2, 3", SC'11), used only by the random down-sampling rule.      */
/* ------------------------------------------------------------------------- */
static void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Exposed so that a test can check the generator against published vectors. */
void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}

/* The random word of rollout i of group g under a seed: the first output word. */
static uint64_t random_key(uint64_t seed, int64_t g, int32_t i) {
    uint32_t ctr[4] = {(uint32_t)i, 0u, (uint32_t)((uint64_t)g & 0xffffffffu), (uint32_t)((uint64_t)g >> 32)};
    uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return (uint64_t)out[0];
}

/* ------------------------------------------------------------------------- */
/* Selection                                                                 */
/* ------------------------------------------------------------------------- */

typedef struct { float r; int32_t i; } reward_index;
typedef struct { uint64_t u; int32_t i; } key_index;

/* Total order used by argsort: by reward, then by original index (stable).
 * -0.0 and +0.0 compare equal; NaN sorts above +inf so that the order is total. */
static int cmp_reward_index(const void* pa, const void* pb) {
    const reward_index* a = (const reward_index*)pa;
    const reward_index* b = (const reward_index*)pb;
    int an = isnan(a->r), bn = isnan(b->r);
    if (an != bn) return an ? 1 : -1;
    if (!an) {
        if (a->r < b->r) return -1;
        if (a->r > b->r) return 1;
    }
    return (a->i > b->i) - (a->i < b->i);
}

static int cmp_key_index(const void* pa, const void* pb) {
    const key_index* a = (const key_index*)pa;
    const key_index* b = (const key_index*)pb;
    if (a->u != b->u) return a->u < b->u ? -1 : 1;
    return (a->i > b->i) - (a->i < b->i);
}

static int cmp_int(const void* pa, const void* pb) {
    int a = *(const int*)pa, b = *(const int*)pb;
    return (a > b) - (a < b);
}

/* m^2 Var of S_k = {ind_1..ind_{m-k}} U {ind_{n-k+1}..ind_n} from the prefix
 * sums P1, P2 of the sorted centred rewards (Theorem 1's proof):
 * Var = E[x^2] - E[x]^2, hence m^2 Var = m * sum x^2 - (sum x)^2. */
static quad split_score(const quad* P1, const quad* P2, int n, int m, int k) {
    quad s1 = P1[m - k] + (P1[n] - P1[n - k]);
    quad s2 = P2[m - k] + (P2[n] - P2[n - k]);
    return (quad)m * s2 - s1 * s1;
}

/*
 * rewards [G,n] fp32 row-major.  Outputs: idx [G,m] (ascending original index),
 * adv [G,m] fp64 aligned with idx, k_out [G] (number of highest-reward rollouts
 * taken; -1 for rules that are not a split), gap [G] (relative distance between
 * the best and the second-best distinct score of Algorithm 2, or +inf).  Any
 * output pointer may be NULL.  Returns 0, or 1 on invalid sizes.
 */
int oracle_select(const float* rewards, int64_t G, int32_t n, int32_t m, int32_t rule, uint64_t seed,
                  uint32_t flags, int32_t* idx, double* adv, int32_t* k_out, double* gap) {
    if (G < 0 || n < 1 || m < 1 || m > n) return 1;
    if (rule < 0 || rule > 3) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t g = 0; g < G; ++g) {
        const float* r = rewards + g * (int64_t)n;
        int32_t* S = (int32_t*)malloc(sizeof(int32_t) * (size_t)m);
        int32_t* ind = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
        int32_t kbest = -1;
        double rel_gap = INFINITY;

        if (rule == RULE_RANDOM) {
            /* D_rand: a uniformly random m-subset = the m smallest of n i.i.d. 32-bit words
             * (equal words, probability ~n^2 2^-33 per group, fall back to index order). */
            key_index* ki = (key_index*)malloc(sizeof(key_index) * (size_t)n);
            for (int i = 0; i < n; ++i) { ki[i].u = random_key(seed, g, i); ki[i].i = i; }
            qsort(ki, (size_t)n, sizeof(key_index), cmp_key_index);
            for (int j = 0; j < m; ++j) S[j] = ki[j].i;
            free(ki);
        } else {
            /* Algorithm 2, step 1: ind <- argsort(r). */
            reward_index* ri = (reward_index*)malloc(sizeof(reward_index) * (size_t)n);
            for (int i = 0; i < n; ++i) { ri[i].r = r[i]; ri[i].i = i; }
            qsort(ri, (size_t)n, sizeof(reward_index), cmp_reward_index);
            for (int j = 0; j < n; ++j) ind[j] = ri[j].i;
            free(ri);

            if (rule == RULE_MAXVAR) {
                /* prefix sums of r and r^2 over the sorted order (Theorem 1) */
                quad* P1 = (quad*)malloc(sizeof(quad) * (size_t)(n + 1));
                quad* P2 = (quad*)malloc(sizeof(quad) * (size_t)(n + 1));
                quad rmin = (quad)r[ind[0]];
                P1[0] = 0; P2[0] = 0;
                for (int j = 0; j < n; ++j) {
                    quad x = (quad)r[ind[j]] - rmin;
                    P1[j + 1] = P1[j] + x;
                    P2[j + 1] = P2[j] + x * x;
                }
                /* step 2: S_ans <- the m lowest (k = 0) */
                kbest = 0;
                quad best = split_score(P1, P2, n, m, 0);
                quad second = -1;   /* best distinct score below `best`, if any */
                /* steps 3-6: replace only on a strictly larger variance */
                for (int k = 1; k <= m; ++k) {
                    quad v = split_score(P1, P2, n, m, k);
                    if (v > best) { second = best; best = v; kbest = k; }
                    else if (v < best && v > second) second = v;
                }
                if (second >= 0 && best > 0) rel_gap = (double)((best - second) / best);
                free(P1); free(P2);
                for (int j = 0; j < m - kbest; ++j) S[j] = ind[j];
                for (int j = 0; j < kbest; ++j) S[m - kbest + j] = ind[n - kbest + j];
            } else if (rule == RULE_MAXREWARD) {
                /* D_maxr: the m highest rewards. */
                kbest = m;
                for (int j = 0; j < m; ++j) S[j] = ind[n - m + j];
            } else {
                /* D_perc: the (j + 0.5)/m quantiles, j = 0..m-1, read as sorted
                 * position floor((j + 0.5) n / m) = floor((2j + 1) n / (2m)). */
                for (int j = 0; j < m; ++j) S[j] = ind[((2 * (int64_t)j + 1) * n) / (2 * (int64_t)m)];
            }
        }

        /* The output is a set: report it in ascending original index. */
        qsort(S, (size_t)m, sizeof(int32_t), cmp_int);
        if (idx) memcpy(idx + g * (int64_t)m, S, sizeof(int32_t) * (size_t)m);
        if (k_out) k_out[g] = kbest;
        if (gap) gap[g] = rel_gap;

        if (adv) {
            /* a_i = (r_i - mu) / sigma over the kept subset (Section 3.2), or over
             * the whole group when FLAG_ADV_BEFORE (Appendix A.3).  Two-pass fp64. */
            int cnt = (flags & FLAG_ADV_BEFORE) ? n : m;
            double mu = 0.0;
            for (int j = 0; j < cnt; ++j) mu += (double)r[(flags & FLAG_ADV_BEFORE) ? j : S[j]];
            mu /= (double)cnt;
            double ss = 0.0;
            for (int j = 0; j < cnt; ++j) {
                double d = (double)r[(flags & FLAG_ADV_BEFORE) ? j : S[j]] - mu;
                ss += d * d;
            }
            double denom = (flags & FLAG_STD_SAMPLE) ? (double)(cnt - 1) : (double)cnt;
            double sigma = (denom > 0.0) ? sqrt(ss / denom) : 0.0;
            for (int j = 0; j < m; ++j)
                adv[g * (int64_t)m + j] = (sigma > 0.0) ? ((double)r[S[j]] - mu) / sigma : 0.0;
        }
        free(S); free(ind);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Loss                                                                      */
/* ------------------------------------------------------------------------- */

static double bf16_bits_to_double(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* w_i = 1 / (M |o_i|), |o_i| = number of unmasked tokens; 0 for an empty sequence. */
void oracle_seq_weights(const uint8_t* mask, const int64_t* cu_seqlens, int64_t M, double* w) {
    for (int64_t i = 0; i < M; ++i) {
        int64_t L = 0;
        for (int64_t t = cu_seqlens[i]; t < cu_seqlens[i + 1]; ++t) L += mask[t] ? 1 : 0;
        w[i] = (L > 0) ? 1.0 / ((double)M * (double)L) : 0.0;
    }
}

/*
 * One token position.  x[0..V) are the logits of the row in fp64.
 *   logp   = log pi_theta(token)                  (log-softmax, two passes)
 *   rho    = pi_theta / pi_theta_fixed = exp(logp - old_logp)
 *   obj    = min(rho a, clip(rho, 1-eps, 1+eps) a)          (Section 3.2)
 *   kl     = exp(d) - d - 1,  d = ref_logp - logp           (penalty; beta = Table 2)
 *   ell    = -obj + beta kl
 *   dl/dlogp = -a rho [rho a <= clip(rho) a] + beta (1 - exp(d))
 *   dlogits[v] = gscale * dl/dlogp * ([v = token] - softmax_v)
 * margin = |rho a - clip(rho) a|: how far the min is from switching branch.
 */
static void grpo_row(const double* x, int32_t V, int32_t token, double old_logp, double ref_logp, int has_ref,
                     double a, double eps, double beta, double gscale,
                     double* logp_out, double* ell_out, double* dldlogp_out, double* margin_out,
                     double* dlogits /* [V] or NULL */) {
    double mx = x[0];
    for (int v = 1; v < V; ++v) if (x[v] > mx) mx = x[v];
    double Z = 0.0;
    for (int v = 0; v < V; ++v) Z += exp(x[v] - mx);
    double lse = mx + log(Z);
    double logp = x[token] - lse;

    double rho = exp(logp - old_logp);
    double clipped = rho < 1.0 - eps ? 1.0 - eps : (rho > 1.0 + eps ? 1.0 + eps : rho);
    double s1 = rho * a, s2 = clipped * a;
    double obj = s1 < s2 ? s1 : s2;
    double ell = -obj;
    double dl = (s1 <= s2) ? -a * rho : 0.0;
    if (has_ref && beta != 0.0) {
        double d = ref_logp - logp;
        ell += beta * (exp(d) - d - 1.0);
        dl += beta * (1.0 - exp(d));
    }
    *logp_out = logp;
    *ell_out = ell;
    *dldlogp_out = dl;
    *margin_out = fabs(s1 - s2);
    if (dlogits) {
        double gs = gscale * dl;
        for (int v = 0; v < V; ++v) {
            double p = exp(x[v] - lse);
            dlogits[v] = gs * ((v == token ? 1.0 : 0.0) - p);
        }
    }
}

/*
 * Rows t = 0..T-1 of a block of bf16 logits (row pitch ldl elements).
 * seq_of_row[t] names the kept sequence i of the row; adv [M] fp32 as the
 * library takes it; seq_weight [M] from oracle_seq_weights.  eps and beta are
 * fp32 values widened to double.  Outputs (any may be NULL): logp [T],
 * ell [T] (per-token loss term), g [T] = mask w_i dl/dlogp (the factor that
 * multiplies (onehot - softmax) in dlogits), margin [T], dlogits [T,V] fp64.
 * A row with mask 0 has g = 0 and a zero dlogits row.  Returns the number of
 * rows whose token id was outside [0,V) (those rows are computed with token 0).
 */
int64_t oracle_grpo_rows(const uint16_t* logits, int64_t ldl, int64_t T, int32_t V, const int32_t* tokens,
                         const float* old_logp, const float* ref_logp, const float* adv,
                         const double* seq_weight, const int32_t* seq_of_row, const uint8_t* mask,
                         float eps, float beta, double* logp, double* ell, double* g, double* margin,
                         double* dlogits) {
    int64_t bad = 0;
#pragma omp parallel for schedule(dynamic, 4) reduction(+ : bad)
    for (int64_t t = 0; t < T; ++t) {
        double* x = (double*)malloc(sizeof(double) * (size_t)V);
        for (int v = 0; v < V; ++v) x[v] = bf16_bits_to_double(logits[t * ldl + v]);
        int32_t tok = tokens[t];
        if (tok < 0 || tok >= V) { tok = 0; bad += 1; }
        int32_t i = seq_of_row[t];
        double w = mask[t] ? seq_weight[i] : 0.0;
        double lp, el, dl, mg;
        grpo_row(x, V, tok, (double)old_logp[t], ref_logp ? (double)ref_logp[t] : 0.0, ref_logp != NULL,
                 (double)adv[i], (double)eps, (double)beta, w, &lp, &el, &dl, &mg,
                 dlogits ? dlogits + t * (int64_t)V : NULL);
        if (!mask[t] || w == 0.0) {
            /* not a token of any rollout's sum: no gradient, whatever old/ref hold there */
            dl = 0.0;
            if (dlogits) memset(dlogits + t * (int64_t)V, 0, sizeof(double) * (size_t)V);
        }
        if (logp) logp[t] = lp;
        if (ell) ell[t] = el;
        if (g) g[t] = w * dl;
        if (margin) margin[t] = mg;
        free(x);
    }
    return bad;
}

/* The same row computation on fp64 logits, for finite-difference checks. */
void oracle_grpo_rows_f64(const double* logits, int64_t T, int32_t V, const int32_t* tokens,
                          const double* old_logp, const double* ref_logp, const double* adv,
                          const double* seq_weight, const int32_t* seq_of_row, const uint8_t* mask,
                          double eps, double beta, double* logp, double* ell, double* g, double* dlogits) {
    for (int64_t t = 0; t < T; ++t) {
        int32_t i = seq_of_row[t];
        double w = mask[t] ? seq_weight[i] : 0.0;
        double lp, el, dl, mg;
        grpo_row(logits + t * (int64_t)V, V, tokens[t], old_logp[t], ref_logp ? ref_logp[t] : 0.0,
                 ref_logp != NULL, adv[i], eps, beta, w, &lp, &el, &dl, &mg,
                 dlogits ? dlogits + t * (int64_t)V : NULL);
        if (!mask[t] || w == 0.0) {
            dl = 0.0;
            if (dlogits) memset(dlogits + t * (int64_t)V, 0, sizeof(double) * (size_t)V);
        }
        if (logp) logp[t] = lp;
        if (ell) ell[t] = el;
        if (g) g[t] = w * dl;
    }
}

/* L = (1/M) sum_i (1/|o_i|) sum_t ell_{i,t}: the outer sums of L_PODS over the
 * concatenated kept rollouts, taken sequence by sequence, token by token. */
double oracle_grpo_loss(const double* ell, const uint8_t* mask, const int64_t* cu_seqlens, int64_t M) {
    double loss = 0.0;
    for (int64_t i = 0; i < M; ++i) {
        int64_t L = 0;
        double s = 0.0;
        for (int64_t t = cu_seqlens[i]; t < cu_seqlens[i + 1]; ++t)
            if (mask[t]) { s += ell[t]; L += 1; }
        if (L > 0) loss += s / (double)L;
    }
    return loss / (double)M;
}

/*
 * pods.h - C ABI of the B200 (sm_100a) hot path of PODS, "Policy Optimization with
 * Down-Sampling" (arxiv 2504.13818): per prompt group, max-variance down-sampling of n
 * rollout rewards to m rollouts, GRPO advantages on the kept subset, concatenation of the
 * kept rollouts, and the GRPO-PODS token objective with its gradient w.r.t. the logits.
 *
 * Conventions for every call
 *   - Pointers marked [dev] are device pointers on the current CUDA device, [host] are host
 *     pointers.  The caller owns every buffer.  Three things outlive a call and are described
 *     where they are declared: the object pods_host_step_create allocates, the fixed scratch
 *     array grpo_loss_chunk_static uses, and the process-wide tuning value of
 *     pods_set_loss_cluster_min_vocab.  No other call allocates device memory or keeps state.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work and return; outputs are valid once the stream has reached that point.
 *   - The return value is a pods_status.  Errors that the host can see (sizes, null or
 *     misaligned pointers, workspace too small) are returned before anything is launched.
 *   - Anomalies only the device can see (non-finite reward, token id outside [0,V), packed
 *     output capacity exceeded) OR a bit into *status [dev, uint32, may be NULL, never
 *     cleared by the library] and the kernel carries on with a defined substitute.  No kernel
 *     traps or waits without bound.
 *   - Notation follows the paper: G prompt groups, n rollouts per group, m kept per group,
 *     M = G*m kept rollouts, T kept tokens, V vocabulary size, |o_i| tokens of rollout i.
 */
#ifndef PODS_H_
#define PODS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PODS_OK = 0,
    PODS_ERR_INVALID_ARG = 1,   /* bad size, null pointer, misaligned pointer */
    PODS_ERR_UNSUPPORTED = 2,   /* n above PODS_MAX_N, unknown rule */
    PODS_ERR_WORKSPACE = 3,     /* workspace missing or too small */
    PODS_ERR_CUDA = 4,          /* a CUDA runtime call failed (launch, copy) */
    PODS_ERR_STATIC_CAPACITY = 5 /* grpo_loss_chunk_static: more rows than the built-in scratch holds */
} pods_status;

/* Bits of the device status word. */
#define PODS_STATUS_NONFINITE_REWARD 0x1u  /* a reward was NaN or +-inf (sorted as NaN > +inf > finite) */
#define PODS_STATUS_TOKEN_RANGE      0x2u  /* a token id was outside [0,V); token 0 was used instead      */
#define PODS_STATUS_CAPACITY         0x4u  /* pods_compact: T exceeded T_cap (the excess was not written),
                                              or a length exceeded src_ld (it was cut to src_ld)          */
#define PODS_STATUS_NEG_LENGTH       0x8u  /* pods_compact: a negative length was treated as 0            */
#define PODS_STATUS_TIMEOUT          0x10u /* a bounded wait inside a kernel ran out (asynchronous copy never
                                              completed); the results of that call are not valid           */
#define PODS_STATUS_INTERNAL         0x40u /* checked build only (-DPODS_BOUNDS_CHECK): an index computed inside a
                                              kernel left its extent; the access was skipped               */
#define PODS_STATUS_INDEX_RANGE      0x20u /* pods_compact: an entry of idx was outside [0,n); rollout 0 of the
                                              group was used instead                                        */

/* Down-sampling rules D(o, r; m) of Section 3.2 / 3.3. */
typedef enum {
    PODS_RULE_MAXVAR = 0,      /* max-variance down-sampling, Section 3.3, Algorithm 2 */
    PODS_RULE_MAXREWARD = 1,   /* the m highest rewards, Section 3.2                   */
    PODS_RULE_RANDOM = 2,      /* uniform m-subset, Section 3.2                        */
    PODS_RULE_PERCENTILE = 3   /* the (j+0.5)/m quantiles, Section 3.2                 */
} pods_rule;

#define PODS_FLAG_ADV_BEFORE 0x1u  /* advantages from full-group statistics (Appendix A.3 "Before") */
#define PODS_FLAG_STD_SAMPLE 0x2u  /* divide by (count-1) instead of count in the standard deviation  */
#define PODS_FLAG_EXACT_TIES 0x4u  /* max-variance rule: settle near-equal split scores in ~106-bit arithmetic (see pods_select) */

#define PODS_MAX_N 1024            /* largest supported group size n */

const char* pods_version(void);
const char* pods_status_string(int status);

/* Copy the device status word to *host_value [host]; synchronises `stream`. */
int pods_read_status(const uint32_t* status /*dev*/, uint32_t* host_value /*host*/, void* stream);

/*
 * pods_select - down-sampling rule D(o, r; m) -> S (Definition 3.1) for G groups at once, and
 * the advantages a_{S,i} = (r_i - mu_S) / sigma_S of Section 3.2.
 *
 * PODS_RULE_MAXVAR is Algorithm 2 with the prefix sums of Theorem 1's proof: argsort the
 * rewards (ties by index, -0 == +0), and over k = 0..m take the k highest and m-k lowest whose
 * variance is largest, the smallest such k on ties (Algorithm 2 replaces only on a strictly
 * larger variance).  Split scores are evaluated in fp64 on rewards centred on the group minimum.
 * Ties: splits that keep the same multiset of rewards, and the mirror pair of a two-valued kept subset
 * (j of a and m-j of b against m-j of a and j of b), tie for any reward values and are recognised from the
 * sorted rewards themselves; these are the only ties that do not depend on the values.  Every other tie is
 * decided by the fp64 scores, which is exact whenever the sums are (rewards on a coarse dyadic grid such as
 * {0, 0.5, 1}) but not for coincidences among rewards like 0.1, 0.2, 0.4; PODS_FLAG_EXACT_TIES re-evaluates
 * such near-ties in double-double arithmetic (about 10 % slower).
 * PODS_RULE_RANDOM keeps the m rollouts with the smallest 32-bit Philox4x32-10 words (counter
 * (i, 0, g lo, g hi), key = seed, first output word; ties by index).  PODS_RULE_PERCENTILE keeps
 * sorted positions floor((j+0.5) n/m), j = 0..m-1.
 *
 *   rewards [dev] fp32 [G,n] row-major            idx   [dev] int32 [G,m], ascending original index
 *   adv     [dev] fp32 [G,m] aligned with idx     k_out [dev] int32 [G] or NULL: highest-reward count k
 *                                                       (m for MAXREWARD, -1 for RANDOM/PERCENTILE)
 * sigma_S is the population (divide by m) standard deviation unless PODS_FLAG_STD_SAMPLE; if it
 * is 0 every advantage of the group is 0.  Requires 1 <= m <= n <= PODS_MAX_N, G >= 0.
 */
int pods_select(const float* rewards, int64_t G, int32_t n, int32_t m, int32_t rule, uint64_t seed,
                uint32_t flags, int32_t* idx, float* adv, int32_t* k_out, uint32_t* status, void* stream);

/*
 * pods_compact - concatenation of the kept rollouts of all prompt groups into one packed batch
 * (text after Algorithm 1).  Rollout j of group g is row g*n+j of the padded storage;
 * kept rollout number i = g*m+j' is rollout idx[g,j'].
 *
 *   idx        [dev] int32 [G,m]                   lengths   [dev] int32 [G*n] tokens per rollout
 *   src_tokens [dev] int32 [G*n, src_ld]           src_f32   [host] array of n_f32 (<= 4) [dev] fp32
 *   dst_tokens [dev] int32 [T_cap]                            [G*n, src_ld] per-token streams (or NULL)
 *   dst_f32    [host] array of n_f32 [dev] fp32 [T_cap]
 *   cu_seqlens [dev] int64 [M+1]: exclusive prefix sums of the kept lengths; cu_seqlens[M] = T
 * Tokens beyond T_cap are not written and PODS_STATUS_CAPACITY is raised.
 */
int pods_compact(const int32_t* idx, int64_t G, int32_t n, int32_t m, const int32_t* lengths,
                 const int32_t* src_tokens, int64_t src_ld, const float* const* src_f32, int32_t n_f32,
                 int64_t* cu_seqlens, int32_t* dst_tokens, float* const* dst_f32, int64_t T_cap,
                 uint32_t* status, void* stream);

/*
 * grpo_seq_weights - the factor 1/(M |o_i|) in front of the token sum of L_PODS (Section 3.2; the
 * 1/m of one prompt becomes 1/M over the concatenated batch).  |o_i| counts tokens with mask != 0
 * (all tokens if mask is NULL); an empty rollout gets weight 0.
 *   mask [dev] uint8 [T] or NULL    cu_seqlens [dev] int64 [M+1]    seq_weight [dev] fp64 [M]
 */
int grpo_seq_weights(const uint8_t* mask, const int64_t* cu_seqlens, int64_t M, double* seq_weight, void* stream);

/* Bytes of workspace grpo_loss_chunk needs for a chunk of T_chunk rows. */
size_t grpo_loss_chunk_workspace_bytes(int64_t T_chunk);

/*
 * grpo_loss_chunk - the token terms of L_PODS(theta, S) (Section 3.2) and d loss / d logits for
 * rows [row0, row0 + T_chunk) of the packed kept tokens, in one kernel.  Per row t of rollout i:
 *   logp = log softmax(logits[t,:])[token]        rho = exp(logp - old_logp)
 *   loss_t = -min(rho a_i, clip(rho, 1-eps, 1+eps) a_i) + beta (exp(d) - d - 1),  d = ref_logp - logp
 *   g_t = grad_scale mask_t w_i (-a_i rho [rho a_i <= clip(rho) a_i] + beta (1 - exp(d)))
 *   dlogits[t,v] = g_t ([v == token] - softmax(logits[t,:])[v])   rounded to bf16 (nearest even)
 * and sum_t mask_t w_i loss_t is ADDED to *loss_acc (the caller zeroes it before the first chunk;
 * the loss is minimised, i.e. it is minus the paper's objective, plus the KL penalty whose
 * coefficient is Table 2's "KL Coefficient").  Rows with mask 0 get logp but a zero dlogits row.
 *
 *   logits  [dev] bf16 [T_chunk, V], row pitch ldl elements.  Fast path: 16-byte aligned base and
 *           ldl % 8 == 0; anything else takes a slower element-wise path.
 *   tokens, old_logp, ref_logp (NULL allowed iff beta == 0), mask (NULL = all ones), logp:
 *           [dev] arrays of T_chunk entries for this chunk's rows (int32, fp32, fp32, uint8, fp32 out)
 *   adv [dev] fp32 [M]; seq_weight [dev] fp64 [M]; cu_seqlens [dev] int64 [M+1]: row0 + t is mapped
 *           to its rollout through cu_seqlens
 *   dlogits [dev] bf16 [T_chunk, V] pitch ldd; may be the same buffer as logits (in place, ldd == ldl),
 *           must not overlap it otherwise
 *   loss_acc [dev] fp64 scalar; workspace [dev] of grpo_loss_chunk_workspace_bytes(T_chunk), 16-byte aligned
 */
int grpo_loss_chunk(const void* logits, int64_t ldl, const int32_t* tokens, const float* old_logp,
                    const float* ref_logp, const float* adv, const double* seq_weight,
                    const int64_t* cu_seqlens, int64_t M, int64_t row0, const uint8_t* mask, int64_t T_chunk,
                    int32_t V, float eps, float beta, float grad_scale, double* loss_acc, float* logp,
                    void* dlogits, int64_t ldd, void* workspace, size_t workspace_bytes, uint32_t* status,
                    void* stream);

/* Bytes of workspace grpo_loss_fwd_bwd needs. */
size_t grpo_loss_workspace_bytes(int64_t T, int64_t M, int64_t chunk_rows);

/*
 * grpo_loss_fwd_bwd - L_PODS(theta, S) over the whole packed batch (Section 3.2):
 *   (logits, tokens, old_logp, ref_logp, adv, mask, eps, beta) -> loss, logp, dlogits.
 * Computes the rollout weights, runs grpo_loss_chunk over chunks of chunk_rows rows (<= 0: one
 * chunk) and writes loss [dev] fp32 scalar = (1/M) sum_i (1/|o_i|) sum_t mask_t loss_t.
 * Arguments as in grpo_loss_chunk, with per-token arrays of T entries.
 */
int grpo_loss_fwd_bwd(const void* logits, int64_t ldl, const int32_t* tokens, const float* old_logp,
                      const float* ref_logp, const float* adv, const int64_t* cu_seqlens, int64_t M,
                      const uint8_t* mask, int64_t T, int32_t V, float eps, float beta, int64_t chunk_rows,
                      float* loss, float* logp, void* dlogits, int64_t ldd, void* workspace,
                      size_t workspace_bytes, uint32_t* status, void* stream);

/*
 * grpo_loss_chunk_static - grpo_loss_chunk without a workspace argument, for callers that must not
 * allocate device memory and have none to spare: code running inside a framework's memory-planned
 * region or a plug-in that is handed only its inputs and outputs, an embedder that forbids cudaMalloc
 * after start-up, a process whose allocator is frozen while a profiler or checkpointer is attached.
 * (The paper has no counterpart; this is a packaging variant of the same computation.)
 *
 * What grpo_loss_chunk keeps in the caller's workspace (per row: its loss term and a 32-byte record
 * of its scalar inputs) is kept here in a fixed array inside the library image, sized for
 * grpo_loss_chunk_static_max_rows() rows (16384): 640.5 KB, resident on every GPU that loads the
 * library until the process exits.  The call itself
 * calls no cudaMalloc, cudaFree or allocating library routine.  Same arguments, outputs and status
 * bits as grpo_loss_chunk, minus workspace/workspace_bytes.
 *
 *   - T_chunk above grpo_loss_chunk_static_max_rows() returns PODS_ERR_STATIC_CAPACITY and launches
 *     nothing: split the rows into more chunks.
 *   - The first call on each device looks up the array's device address (a host-side runtime query,
 *     with that device current) and remembers it; make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the last call's contents.  Nothing in it
 *     needs clearing: each call overwrites the T_chunk slots it later reads.  Two calls that can run
 *     at the same time on the GPU (different streams, no ordering between them) race on it and give
 *     a wrong loss_acc; order them, or use grpo_loss_chunk with separate workspaces.
 */
int64_t grpo_loss_chunk_static_max_rows(void);
int grpo_loss_chunk_static(const void* logits, int64_t ldl, const int32_t* tokens, const float* old_logp,
                           const float* ref_logp, const float* adv, const double* seq_weight,
                           const int64_t* cu_seqlens, int64_t M, int64_t row0, const uint8_t* mask,
                           int64_t T_chunk, int32_t V, float eps, float beta, float grad_scale,
                           double* loss_acc, float* logp, void* dlogits, int64_t ldd, uint32_t* status,
                           void* stream);

/*
 * grpo_logp_from_hidden - log pi_theta(o_t | p, o_<t), the policy term of L_GRPO (Section 3.1) and L_PODS
 * (Section 3.2), computed from the last hidden states without ever storing the logits:
 *   logits[t, :] = hidden[t, :] . W^T  (bf16 inputs, fp32 accumulation on the tensor cores, not rounded to bf16)
 *   lse[t] = log sum_v exp(logits[t, v])        logp[t] = logits[t, tokens[t]] - lse[t]
 * This is the forward-only half of fusing the LM-head projection into the objective: it serves the passes that
 * need no gradient - the frozen sampling policy's old_logp and the reference policy's ref_logp, which
 * grpo_loss_chunk takes as inputs - and saves them the write and the re-read of [T,V] logits.
 *
 *   hidden [dev] bf16 [T, d], row pitch ldh elements      W [dev] bf16 [V, d], row pitch ldw elements
 *   tokens [dev] int32 [T] (an id outside [0,V) raises PODS_STATUS_TOKEN_RANGE and is read as 0)
 *   logp   [dev] fp32 [T]                                 lse [dev] fp32 [T] or NULL
 *   workspace [dev] of grpo_logp_from_hidden_workspace_bytes(T, V, d), 16-byte aligned (the size follows from
 *             the SM count of the device that is current at the query: ask on the device that will run the call)
 * Requires d >= 8 and d % 8 == 0, ldh % 8 == 0, ldw % 8 == 0, 16-byte aligned hidden and W (so that every row
 * starts on a 16-byte boundary); anything else returns PODS_ERR_INVALID_ARG.  Both matrices must live in the
 * current device's own memory.
 */
size_t grpo_logp_from_hidden_workspace_bytes(int64_t T, int32_t V, int32_t d);
int grpo_logp_from_hidden(const void* hidden, int64_t ldh, const void* W, int64_t ldw, const int32_t* tokens,
                          int64_t T, int32_t V, int32_t d, float* logp, float* lse, void* workspace,
                          size_t workspace_bytes, uint32_t* status, void* stream);

/*
 * grpo_loss_from_hidden - the token terms of L_PODS(theta, S) (Section 3.2) for rows [row0, row0 + T) of the packed
 * kept tokens when the logits are the LM-head projection of the last hidden states, together with the gradient
 * carried back through that projection; neither the [T,V] logits nor their gradient is ever stored in full:
 *   logits[t, :] = hidden[t, :] . W^T  (bf16 inputs, fp32 accumulation on the tensor cores, not rounded to bf16)
 *   logp, loss_t, g_t as in grpo_loss_chunk;   dlogits[t, v] = g_t ([v == token] - softmax(logits[t, :])[v])
 *   dhidden[t, :]  = sum_v dlogits[t, v] W[v, :]           (written: fp32 [T, d], row pitch lddh elements)
 *   dW[v, :]      += sum_t dlogits[t, v] hidden[t, :]      (ADDED to fp32 [V, d], row pitch lddw elements: the
 *                                                           caller zeroes it before the first chunk of a batch)
 * and sum_t mask_t w_i loss_t is ADDED to *loss_acc.  dlogits is rounded to bf16 (nearest even) before it is
 * contracted, as the gradient grpo_loss_chunk writes is; it exists only one panel of the vocabulary at a time,
 * inside the workspace (at most 512 MB, whatever T and V).  The logits are formed twice (once for the row
 * statistics, once for the gradient): the second pass is the price of not storing them.
 * This is the gradient half of fusing the LM-head projection into the objective; grpo_logp_from_hidden is the
 * half for passes that need no gradient.
 *
 *   hidden [dev] bf16 [T, d] pitch ldh; W [dev] bf16 [V, d] pitch ldw (d >= 8, d % 8 == 0, ldh % 8 == 0,
 *          ldw % 8 == 0, 16-byte aligned bases), both in the current device's own memory
 *   tokens, old_logp, ref_logp (NULL allowed iff beta == 0), mask (NULL = all ones), logp (out): [dev] arrays of T
 *   adv [dev] fp32 [M]; seq_weight [dev] fp64 [M]; cu_seqlens [dev] int64 [M+1]; row0: first packed row of the chunk
 *   dhidden, dW: [dev] fp32, 16-byte aligned, lddh % 4 == 0, lddw % 4 == 0; they must not overlap anything else
 *   loss_acc [dev] fp64 scalar; workspace [dev] of grpo_loss_from_hidden_workspace_bytes(T, V, d), 256-byte
 *   aligned (the size follows from the SM count of the current device: ask on the device that runs the call)
 * A token id outside [0,V) raises PODS_STATUS_TOKEN_RANGE and is read as 0; a wait that runs out raises
 * PODS_STATUS_TIMEOUT.  Invalid sizes or pointers return PODS_ERR_INVALID_ARG before anything is launched.
 */
size_t grpo_loss_from_hidden_workspace_bytes(int64_t T, int32_t V, int32_t d);
int grpo_loss_from_hidden(const void* hidden, int64_t ldh, const void* W, int64_t ldw, const int32_t* tokens,
                          const float* old_logp, const float* ref_logp, const float* adv, const double* seq_weight,
                          const int64_t* cu_seqlens, int64_t M, int64_t row0, const uint8_t* mask, int64_t T,
                          int32_t V, int32_t d, float eps, float beta, float grad_scale, double* loss_acc,
                          float* logp, float* dhidden, int64_t lddh, float* dW, int64_t lddw, void* workspace,
                          size_t workspace_bytes, uint32_t* status, void* stream);

/*
 * pods_set_loss_from_hidden_panel_bytes - tuning knob (the paper has no counterpart): the most bytes of workspace
 * grpo_loss_from_hidden may spend on the piece of the logits gradient that exists at one time (default 512 MB; at
 * least one 256-column tile per panel is always taken; values below 64 KB are raised to 64 KB).  Smaller panels
 * mean less memory and more passes over dhidden.  Process-wide; changes what grpo_loss_from_hidden_workspace_bytes
 * returns; returns the previous value.  Results meet the same tolerances at any setting.
 */
size_t pods_set_loss_from_hidden_panel_bytes(size_t bytes);

/*
 * pods_set_loss_cluster_min_vocab - tuning knob (the paper has no counterpart): grpo_loss_chunk runs rows of
 * V >= min_vocab (V % 8 == 0, 16-byte aligned rows) on the cluster-resident kernel and shorter rows on the
 * row-tile (V <= 4096) or the general row kernel.  The default, 8192, is the measured cross-over on B200; values
 * below 2048 are raised to 2048.  Process-wide; returns the previous value.  Results of either kernel meet the same tolerances.
 */
int32_t pods_set_loss_cluster_min_vocab(int32_t min_vocab);

/*
 * pods_selftest_bounded_wait - diagnostic (the paper has no counterpart): one small kernel waits, with the
 * same bounded poll loop the loss kernel uses for its barriers, on a barrier that nothing completes.
 * After `polls` (1 .. 2^20) failed polls it must give up, OR PODS_STATUS_TIMEOUT into *status [dev]
 * and return normally, leaving the context usable.  Shows that a lost signal ends in a status bit,
 * not in a hang.
 */
int pods_selftest_bounded_wait(uint32_t polls, uint32_t* status, void* stream);

/* Convert the fp64 accumulator of grpo_loss_chunk calls to the fp32 loss.  Both [dev]. */
int grpo_loss_finalize(const double* loss_acc, float* loss, void* stream);

/*
 * pods_host_step - the whole path of one training batch for callers whose data is in HOST memory:
 * D(o, r; m) and a_{S,i} (Sections 3.2-3.3), concatenation of the kept rollouts (text after
 * Algorithm 1) and L_PODS with its gradient (Section 3.2), i.e. pods_select -> pods_compact ->
 * grpo_seq_weights -> grpo_loss_chunk per chunk -> grpo_loss_finalize, with the copies around them.
 *
 * pods_host_step_create allocates, on the current device, every buffer the step needs (the only
 * calls of this library that allocate): rollout storage for G*n rollouts of src_ld tokens, packed
 * per-token arrays of T_cap entries, two staging buffers of chunk_rows x V bf16 logits, the
 * gradient [T_cap, V] bf16, the loss workspace, two streams and four events.  V % 8 == 0 is
 * required.  pods_host_step_destroy frees them.  One object serves one thread at a time.
 *
 * pods_host_step_run, all pointers [host] (pinned memory makes the copies asynchronous):
 *   rewards fp32 [G,n]; lengths int32 [G*n]; src_tokens int32, src_old, src_ref fp32 [G*n, src_ld]
 *   (src_ref may be NULL iff beta == 0); logits bf16 [T_logits, V], densely packed: the rows of the
 *   kept rollouts in kept order - the caller must know which rollouts the rule keeps (it does when the
 *   logits come from a forward pass over the kept rollouts only); if the device finds another T the
 *   call stops after the compaction, *T_out holds the device's T and PODS_ERR_INVALID_ARG is returned.
 *   Outputs: loss_out fp32 [1]; logp_out fp32 [T] or NULL; idx_out int32 [G,m] or NULL; adv_out
 *   fp32 [G,m] or NULL; T_out, status_out (the device status word) or NULL.
 * The logits are uploaded chunk by chunk on a second stream while the previous chunk's loss kernel
 * runs.  dlogits [T, V] (row pitch V) stays on the device for the backward pass that consumes it:
 * pods_host_step_dlogits returns its [dev] address, valid until the next run or destroy.  The call
 * returns when every result is in place.
 */
typedef struct pods_host_step pods_host_step;
int pods_host_step_create(int64_t G, int32_t n, int32_t m, int64_t src_ld, int64_t T_cap, int32_t V,
                          int64_t chunk_rows, pods_host_step** out);
int pods_host_step_run(pods_host_step* step, const float* rewards, const int32_t* lengths,
                       const int32_t* src_tokens, const float* src_old, const float* src_ref, const void* logits,
                       int64_t T_logits, float eps, float beta, int32_t rule, uint64_t seed, uint32_t flags,
                       float* loss_out, float* logp_out, int32_t* idx_out, float* adv_out, int64_t* T_out,
                       uint32_t* status_out);
void* pods_host_step_dlogits(pods_host_step* step);
int pods_host_step_destroy(pods_host_step* step);

#ifdef __cplusplus
}
#endif
#endif /* PODS_H_ */

/* asyncflow.h -- C ABI of the B200 (sm_100a) scoring path for streaming GRPO post-training.
 *
 * The library implements the device-side hot path shared by the actor-inference,
 * reference-inference and actor-update tasks of AsyncFlow (arXiv 2507.01663): micro-batches of
 * variable-length responses are gathered from a sample-indexed columnar store, scored by the LM
 * head with a fused online log-softmax, and reduced to the clipped GRPO policy loss (forward and
 * backward).  The paper fixes the data flow; it prints no formula for the numerics, which are
 * the textbook definitions stated with each entry point below.
 *
 * Conventions
 *   - "dev" pointers are device pointers on the context's device, "host" pointers are host
 *     pointers.  All buffers are owned by the caller; the library owns only its context and
 *     the workspace inside it.
 *   - Every call enqueues its kernels on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream) and returns without synchronising, unless noted.
 *   - The return code reports what the host can see (null pointers, sizes, alignment, capacity,
 *     index lists, CUDA launch errors).  Conditions only the device can see (a target id outside
 *     [0, V), a watchdog expiry inside a kernel) set bits of a sticky device error word that
 *     af_check_device_errors reads; affected outputs are NaN; no kernel traps.
 *   - A context serves one stream at a time: calls on one context must not overlap on the GPU
 *     (they share its workspace).  Use one context per concurrent stream.
 *   - Workspace grows on demand with cudaMalloc (which may synchronise).  Call af_reserve once
 *     with the largest sizes to keep allocation out of the hot calls.
 *   - Stream capture: once af_reserve has covered the sizes (and the tuning is unchanged), every
 *     call except af_pack_microbatch, af_unpack_microbatch, af_check_device_errors, af_reserve and
 *     af_destroy issues only kernel launches and asynchronous memsets on `stream`, so a sequence
 *     of them may be recorded into a CUDA graph and replayed on new contents of the same buffers.
 *     af_pack_microbatch and af_unpack_microbatch build a table from their host index list (and
 *     for large batches stage it through pinned host memory, waiting on an event of their own);
 *     they are not meant to be recorded.  Nothing is claimed for
 *     af_token_logprob_static.
 *   - Only compute capability 10.0 devices are accepted.  There is no CPU path.
 *   - Every entry point that enqueues work opens an NVTX range named after itself (a no-op unless
 *     a profiler that reads NVTX is attached).
 */
#ifndef ASYNCFLOW_H_
#define ASYNCFLOW_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct af_ctx af_ctx;

typedef enum {
  AF_OK = 0,
  AF_ERR_INVALID_ARG = -1,        /* null pointer, negative size, bad enum value            */
  AF_ERR_SHAPE = -2,              /* size outside what the kernels support (see each call)   */
  AF_ERR_ALIGNMENT = -3,          /* pointer or row pitch not 16-byte aligned                */
  AF_ERR_CAPACITY = -4,           /* caller's output buffers too small                       */
  AF_ERR_INDEX = -5,              /* sample index outside [0, N)                             */
  AF_ERR_WORKSPACE = -6,          /* workspace allocation failed                             */
  AF_ERR_CUDA = -7,               /* a CUDA runtime / driver call failed                     */
  AF_ERR_UNSUPPORTED_DEVICE = -8, /* device is not compute capability 10.0                   */
  AF_ERR_DEVICE_FLAGGED = -9      /* af_check_device_errors found the error word non-zero    */
} af_status;

/* bits of the device error word */
#define AF_DEVERR_TARGET_RANGE 1u /* a target id was outside [0, V): that token's outputs are NaN */
#define AF_DEVERR_WATCHDOG 2u     /* a bounded wait inside a kernel ran out; results invalid      */
#define AF_DEVERR_CU_SEQLENS 4u   /* cu_seqlens not non-decreasing from 0 to T                     */
#define AF_DEVERR_SAMPLE_INDEX 8u /* af_controller_put met an index outside [0, N): entry skipped  */
#define AF_DEVERR_GROUP_ID 16u    /* af_grpo_advantage met a group id outside [0, n_groups): NaN    */

/* Create / destroy a context on CUDA device `device`.  af_create fails with
 * AF_ERR_UNSUPPORTED_DEVICE unless the device is compute capability 10.0.  af_destroy
 * synchronises the device and frees the workspace. */
af_status af_create(af_ctx** out, int device);
af_status af_destroy(af_ctx* ctx);
const char* af_status_string(af_status s);

/* Pre-size the workspace for micro-batches of up to max_T tokens and max_B sequences at head
 * shape (d, V), and for af_grpo_advantage by group id with up to max_B groups (pass the number of
 * stored responses as max_B if advantages are taken over the whole store).  with_backward != 0
 * also reserves the scratch of af_policy_loss_backward, and with_backward == 2 that of
 * af_policy_update too.  Synchronous (allocates). */
af_status af_reserve(af_ctx* ctx, int64_t max_T, int32_t max_B, int32_t d, int32_t V,
                     int32_t with_backward);

/* Bytes of device workspace currently held by the context. */
int64_t af_workspace_bytes(const af_ctx* ctx);

/* Tuning knobs of the fused LM-head kernels (0 keeps the default): `v_splits` = number of
 * vocabulary ranges one token tile is split into across CTAs; `bwd_token_block` = tokens per
 * backward block, a multiple of 128 (scratch is proportional to it); `gemm_variant` selects the
 * main loop of every tensor-core GEMM of the context: 0 (the default) and 3 = CTA pairs -- two
 * SMs share one 256 x 256 tile, each staging half of the weight tile, the pairs pace one another
 * so that a weight tile fetched once serves them all, and the row tiles are dealt to the pairs by
 * the die they run on (see af_die_split), so that a hidden-state panel occupies one half of L2
 * only; 2 = CTA pairs dealt without regard to dies; 1 = one CTA per 128 x 256 tile.
 * Results agree within the stated tolerances either way. */
af_status af_set_tuning(af_ctx* ctx, int32_t v_splits, int32_t bwd_token_block, int32_t gemm_variant);

/* Self-test of the bounded waits (the paper has no counterpart; failure handling of this library).
 * Every wait inside the kernels gives up after a time limit, sets AF_DEVERR_WATCHDOG and lets the
 * kernel return; nothing traps or spins without bound.  This call runs that same wait for one warp
 * on a barrier nobody arrives at, with a limit of one millisecond, synchronises `stream` and returns
 * how long the warp waited (microseconds, nullable).  Afterwards af_check_device_errors reports (and
 * clears) AF_DEVERR_WATCHDOG, and the context is as usable as before. */
af_status af_selftest_bounded_wait(af_ctx* ctx, uint32_t* waited_us, void* stream);

/* How af_create found the SMs split over the two dies of the part (each die has its own half of
 * L2): the number of SMs that share a die with the first SM probed, and the rest.  When the latency
 * measurement behind it was not clear-cut after several attempts (then work is dealt without regard
 * to dies), *die0_sms is 0 and *die1_sms is minus the reason: 1 a CUDA call failed, 2 SM ids out of
 * range or repeated, 3 an SM between the two groups, 4 an SM pair straddling the dies, 5 a lopsided
 * split. */
af_status af_die_split(const af_ctx* ctx, int32_t* die0_sms, int32_t* die1_sms);

/* Data-parallel actor update (Section 4.1: the training batch is streamed to the DP groups of the
 * actor-update task; each computes the gradient of its share).  The one exchange of the path is
 * the sum of the ranks' d_W.  Register a cudaEvent_t (as void*; NULL clears it; the event stays the
 * caller's) and af_policy_loss_backward, its shard form and af_policy_update record it on their
 * stream at the point where d_W is complete: the last token block then runs its dW product BEFORE
 * its dH product, so a collective that waits on the event on another stream overlaps with the
 * remaining dH product, the loss record and whatever the caller enqueues next.  Results do not
 * depend on it (the two products of a block are independent).  While an event is registered the
 * three calls cannot be recorded into a CUDA graph of a single stream. */
af_status af_set_dw_ready_event(af_ctx* ctx, void* event);

/* Synchronise `stream`, read and clear the sticky device error word.  Returns AF_OK when it was
 * zero, else AF_ERR_DEVICE_FLAGGED with the bits in *flags (nullable). */
af_status af_check_device_errors(af_ctx* ctx, uint32_t* flags, void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_pack_microbatch -- sample-index list -> cu_seqlens-packed tensors.
 *
 * The store is the paper's 2-D columnar structure restricted to one device (Section 4.3 "Data
 * Plane"): rows are samples addressed by a global index, columns are task-specific components,
 * and a task reads only the columns it asks for (NULL = not requested).  The index list is the
 * metadata a controller hands out; the worker on the device fetches the data (Section 4.2
 * "Interaction Interface").  Sample i owns token rows tok_offset[i] .. tok_offset[i+1]-1 of every
 * per-token column.
 *
 * For j in [0, B): cu_seqlens[j+1] = cu_seqlens[j] + len(idx[j]); the rows of sample idx[j] are
 * copied, bit for bit, to packed rows cu_seqlens[j] .. cu_seqlens[j+1]-1 of each requested
 * column; adv_seq[j] = adv[idx[j]]; seq_id[t] = j.  Duplicate indices are gathered twice.
 *
 * Errors: AF_ERR_INDEX for an index outside [0, N); AF_ERR_CAPACITY if T or B exceed the output
 * capacities or T >= 2^31; AF_ERR_ALIGNMENT unless d % 8 == 0 and hidden pointers are 16-byte
 * aligned.  *T_out (host) receives the packed token count before the call returns.  B == 0 is
 * valid and writes cu_seqlens[0] = 0 only.
 *
 * The sequence table the kernels work from (first row, length and packed offset of each indexed
 * sample) is built on the host in O(B).  For up to 512 sequences whose hidden rows are at most
 * 32 KB it travels in the parameters of the one kernel that does the whole gather -- the call
 * then waits for nothing and stages nothing; larger batches (or a call without the hidden
 * column) stage it through pinned host memory, from where a small kernel brings it to the device.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int64_t n_samples;               /* N                                                       */
  int32_t d;                       /* hidden size (elements per token row)                    */
  int32_t reserved;
  const int64_t* tok_offset_host;  /* [N+1] host: lets the host size the batch without a sync */
  const void* hidden;              /* [sum L, d] bf16, dev, row-major                         */
  const int32_t* target;           /* [sum L] dev, or NULL                                    */
  const float* old_logp;           /* [sum L] dev, or NULL                                    */
  const float* ref_logp;           /* [sum L] dev, or NULL                                    */
  const float* adv;                /* [N] dev, or NULL                                        */
} af_store_view;

typedef struct {
  int64_t token_capacity;          /* rows available in the per-token outputs                 */
  int32_t seq_capacity;            /* cu_seqlens holds seq_capacity + 1 entries               */
  int32_t reserved;
  int32_t* cu_seqlens;             /* [B+1] dev (required)                                    */
  void* hidden;                    /* [T, d] bf16 dev, or NULL iff store.hidden is NULL       */
  int32_t* target;                 /* [T] dev, NULL iff store.target is NULL                  */
  float* old_logp;                 /* [T] dev, NULL iff store.old_logp is NULL                */
  float* ref_logp;                 /* [T] dev, NULL iff store.ref_logp is NULL                */
  float* adv_seq;                  /* [B] dev, NULL iff store.adv is NULL                     */
  int32_t* seq_id;                 /* [T] dev, or NULL                                        */
} af_packed;

af_status af_pack_microbatch(af_ctx* ctx, const af_store_view* store, const int32_t* idx_host,
                             int32_t B, const af_packed* out, int64_t* T_out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_token_logprob -- LM-head projection fused with an online log-softmax (the last stage of
 * the `compute_log_prob` task of the paper's backend interface, Appendix "Backend-level
 * interface"; forward-only for reference / actor inference, Section 7.4).
 *
 * For each token t:  z_tv = sum_k hidden[t,k] * W[v,k]  (bf16 x bf16, fp32 accumulation; the
 * [T,V] logits are never written to memory);  lse_t = log sum_v exp z_tv;
 * logp_t = z_{t,target[t]} - lse_t;  entropy_t = lse_t - sum_v softmax_tv * z_tv.
 *
 * hidden [T,d] bf16 dev, W [V,d] bf16 dev (one row per vocabulary id), both row-major and
 * 16-byte aligned, d % 8 == 0, 1 <= d, 1 <= V, 0 <= T < 2^31.  logp (required), entropy and lse
 * (nullable) are [T] fp32 dev.  A target outside [0,V) yields NaN logp and AF_DEVERR_TARGET_RANGE.
 * ------------------------------------------------------------------------------------------- */
af_status af_token_logprob(af_ctx* ctx, const void* hidden, const void* W, const int32_t* target,
                           int64_t T, int32_t d, int32_t V, float* logp, float* entropy,
                           float* lse, void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_token_logprob_shard / af_merge_logprob_shards -- the same scoring with the LM head split by
 * vocabulary rows over model-parallel ranks.
 *
 * The paper's instances combine tensor parallelism with the other strategies (Section 2.1); it
 * says nothing about the head.  These two calls are what a vocabulary-parallel head needs on the
 * forward path (af_policy_loss_backward_shard is their counterpart for the actor update).  Rank r holds the rows [v_offset, v_offset + V_shard) of W and computes, per token, the
 * four statistics of its logits z_v = hidden[t,:] . W_shard[v,:]:
 *     m = max_v z_v,  s = sum_v exp(z_v - m),  u = sum_v exp(z_v - m) z_v,
 *     zy = z at the target if target[t] lies in the shard, else -inf
 * written as partial_out[t] = (m, s, u, zy), fp32, [T][4], 16-byte aligned.  The ranks exchange
 * these 16 bytes per token (one all-gather) into partials
 * [R][T][4], and af_merge_logprob_shards gives, with M = max_r m_r, S = sum_r s_r e^{m_r - M},
 * U = sum_r u_r e^{m_r - M}:  lse = M + log S,  logp = max_r zy_r - lse,  entropy = lse - U / S
 * -- the full-vocabulary result of af_token_logprob up to fp32 rounding.  target holds global ids;
 * one outside [0, V_total) gives a NaN log-prob and AF_DEVERR_TARGET_RANGE at the merge.
 * Arguments, alignment and errors as for af_token_logprob; entropy and lse may be NULL.
 * ------------------------------------------------------------------------------------------- */
af_status af_token_logprob_shard(af_ctx* ctx, const void* hidden, const void* W_shard,
                                 const int32_t* target, int64_t T, int32_t d, int32_t V_shard,
                                 int32_t v_offset, float* partial_out, void* stream);
af_status af_merge_logprob_shards(af_ctx* ctx, const float* partials, const int32_t* target, int32_t R,
                                  int64_t T, int32_t V_total, float* logp, float* entropy, float* lse,
                                  void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_grpo_advantage -- group-normalised advantages: GRPO has no critic and takes each response's
 * advantage from its reward relative to the other responses to the same prompt (paper Section
 * 7.1 "RL algorithms").
 *
 * For each group g with members I_g (n_g = |I_g|):  mu = mean r;  sigma = sqrt(sum (r-mu)^2 /
 * (n_g - ddof));  adv_i = (r_i - mu) / (sigma + eps_adv).  A group of equal rewards gets zeros.
 *
 * reward [N] fp32 dev.  group_id [N] int32 dev with values in [0, n_groups) in any order, or
 * NULL for contiguous equal groups (sample i belongs to group i / (N / n_groups); then
 * N % n_groups must be 0).  With group_id given the work is O(N) whatever n_groups is: the group
 * sums are exact fixed-point sums taken with integer atomics, so the result does not depend on the
 * order of the members and is bit-reproducible; N < 2^31 (AF_ERR_SHAPE); a per-group accumulator
 * table (64 B per group) is kept in the context's workspace (grown on demand, or ahead of time by
 * af_reserve for max_B groups); a sample whose id lies outside
 * [0, n_groups) gets a NaN advantage and raises AF_DEVERR_GROUP_ID; groups without members are fine.
 * ddof is 0 or 1.  eps_adv must be > 0 (AF_ERR_INVALID_ARG otherwise: with eps_adv = 0 a group of
 * equal rewards would divide 0 by 0).  adv [N] fp32 dev.
 * ------------------------------------------------------------------------------------------- */
af_status af_grpo_advantage(af_ctx* ctx, const float* reward, const int32_t* group_id, int64_t N,
                            int32_t n_groups, float eps_adv, int32_t ddof, float* adv,
                            void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_policy_loss -- clipped-ratio GRPO policy loss with a k3 KL penalty against the reference
 * log-probs (the loss of the paper's actor-update task, Section 7.4; GRPO, Section 7.1).
 *
 * Token t of sequence i, A = adv_seq[i]:
 *   rho = exp(logp - old);  pg = -min(rho*A, clip(rho, 1-clip_lo, 1+clip_hi)*A);
 *   delta = ref - logp;  k3 = exp(delta) - delta - 1;  l = pg + kl_coef*k3.
 *   A token counts as clipped iff clip(rho)*A < rho*A (strict).
 * agg_mode 0: loss = loss_scale * mean_i( mean_{t in i} l_t ); agg_mode 1: loss_scale * mean_t l_t.
 * pg_loss and kl_mean aggregate pg and k3 the same way; clip_frac = #clipped / T;
 * entropy_mean = sum entropy / T (0 if entropy is NULL).
 * dlogp[t] = w_t * ( clipped ? 0 : -A*rho ) + w_t * kl_coef * (1 - exp(delta)), w_t the weight of
 * token t in the aggregation (loss_scale/(B*L_i) or loss_scale/T).  Entropy carries no gradient.
 *
 * logp, old_logp, ref_logp, entropy (nullable), dlogp (nullable): [T] fp32 dev; adv_seq [B] fp32
 * dev; cu_seqlens [B+1] int32 dev, non-decreasing, cu_seqlens[0] = 0, cu_seqlens[B] = T.
 * `out` is a device struct, valid when the stream reaches the end of the call.  Sums are taken
 * in a fixed order: results are bit-reproducible from run to run.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  float clip_lo, clip_hi;
  float kl_coef;
  int32_t agg_mode;
  float loss_scale;
} af_loss_params;

typedef struct {
  float loss, pg_loss, kl_mean, clip_frac, entropy_mean;
  int32_t reserved;
  int64_t n_tokens;
} af_loss_out;

af_status af_policy_loss(af_ctx* ctx, const float* logp, const float* old_logp,
                         const float* ref_logp, const float* entropy, const float* adv_seq,
                         const int32_t* cu_seqlens, int32_t B, int64_t T,
                         const af_loss_params* params, af_loss_out* out, float* dlogp,
                         void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_policy_loss_backward -- gradient of the loss through log-softmax and the LM head (the
 * forward-backward actor-update task, paper Section 7.4), without materialising [T,V].
 *
 *   dZ_tv = dlogp[t] * ( 1{v == target[t]} - exp(z_tv - lse[t]) )      (z recomputed per block)
 *   d_hidden[t,:] = sum_v dZ_tv * W[v,:]          -> [T,d] bf16
 *   d_W[v,:]      = sum_t dZ_tv * hidden[t,:]     -> [V,d] fp32 (added to d_W if accumulate_dW)
 *
 * dZ is rounded to bf16 for the two tensor-core products (fp32 accumulation).  Tokens are
 * processed in blocks; the only scratch is the dZ of one block (token block x V bf16) in the
 * context's workspace, independent of T.  No operand is transposed in memory.
 * Requirements: d % 8 == 0, V % 8 == 0, 16-byte aligned pointers, 0 <= T < 2^31.
 * ------------------------------------------------------------------------------------------- */
af_status af_policy_loss_backward(af_ctx* ctx, const void* hidden, const void* W,
                                  const int32_t* target, const float* lse, const float* dlogp,
                                  int64_t T, int32_t d, int32_t V, void* d_hidden, float* d_W,
                                  int32_t accumulate_dW, void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_policy_loss_backward_shard -- the same backward on one vocabulary shard of the head (the
 * counterpart of af_token_logprob_shard for the actor update; Section 2.1 names tensor parallelism,
 * the paper says nothing about the head).
 *
 * The rank holds rows [v_offset, v_offset + V_shard) of W.  lse is the logsumexp over the WHOLE
 * vocabulary (from af_merge_logprob_shards), target holds global ids, dlogp comes from
 * af_policy_loss on the merged log-probs.  Over the shard's columns only:
 *   dZ_tv = dlogp[t] * ( 1{target[t] == v_offset + v} - exp(z_tv - lse[t]) )
 *   d_hidden_partial[t,:] = sum_v dZ_tv * W_shard[v,:]   -> [T,d] bf16: this shard's contribution;
 *                                                           the ranks' contributions add up to
 *                                                           d_hidden (one all-reduce)
 *   d_W_shard[v,:]        = sum_t dZ_tv * hidden[t,:]    -> [V_shard,d] fp32: the rank's own rows
 * Requirements as for af_policy_loss_backward with V_shard in place of V; v_offset >= 0.
 * ------------------------------------------------------------------------------------------- */
af_status af_policy_loss_backward_shard(af_ctx* ctx, const void* hidden, const void* W_shard,
                                        const int32_t* target, const float* lse, const float* dlogp,
                                        int64_t T, int32_t d, int32_t V_shard, int32_t v_offset,
                                        void* d_hidden_partial, float* d_W_shard,
                                        int32_t accumulate_dW, void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_policy_update -- forward, loss and backward of one packed micro-batch in one call (the
 * forward-backward actor-update task of Section 7.4).
 *
 * Computes what af_token_logprob, af_policy_loss and af_policy_loss_backward compute when called
 * one after the other on the same micro-batch -- logp, entropy, lse [T]; the loss record; dlogp
 * [T]; d_hidden [T,d] bf16; d_W [V,d] fp32 -- but evaluates the logits once per token instead of
 * twice: tokens are processed in blocks, a block's fp32 logits stay in scratch between the
 * log-softmax statistics and dZ, and the per-token loss gradient is taken in between with the
 * arithmetic of af_policy_loss.  Scratch: one block of logits (fp32) and of dZ (bf16), independent
 * of T; [T,V] is never materialised.  af_reserve with with_backward = 2 pre-sizes it.
 * entropy and dlogp may be NULL; every other pointer is required when T > 0.  Requirements and
 * errors as for the three calls (d % 8 == 0, V % 8 == 0, 16-byte aligned matrices, 0 <= T < 2^31).
 * ------------------------------------------------------------------------------------------- */
af_status af_policy_update(af_ctx* ctx, const void* hidden, const void* W, const int32_t* target,
                           const float* old_logp, const float* ref_logp, const float* adv_seq,
                           const int32_t* cu_seqlens, int32_t B, int64_t T, int32_t d, int32_t V,
                           const af_loss_params* params, af_loss_out* out, float* logp, float* entropy,
                           float* lse, float* dlogp, void* d_hidden, float* d_W, int32_t accumulate_dW,
                           void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_controller_put / af_controller_get / af_controller_clear -- the status table of the
 * streaming store and one read request against it.
 *
 * The paper's TransferQueue controller keeps, per sample, a binary "written" indicator for every
 * column and a consumption record per RL task; a `get` request builds the mask of the requested
 * columns, finds the samples whose requested columns are all written and that the requesting
 * task has not been handed yet, selects the required number of them, returns their metadata and
 * marks them consumed; storage units report finished writes, which turns indicators on (Section
 * 4.4 "Control Plane: Panoramic Data Admin" with its figure of the get procedure; Section 4.2).
 * Here the table lives on the device next to the store it describes:
 *   ready[i]    bit c set  <=>  column c of sample i has been written       (c in 0..31)
 *   consumed[i] bit t set  <=>  sample i has been handed to task t           (t in 0..31)
 *   length[i]   tokens of sample i (only needed for token budgets)
 *
 * put:   ready[idx[j]] |= column_bits for j in [0, n); idx is a DEVICE array (for instance the
 *        out_idx of the get that handed the samples out).  An index outside [0, N) is skipped
 *        and sets AF_DEVERR_SAMPLE_INDEX.
 * get:   sample i is eligible iff (ready[i] & column_mask) == column_mask and
 *        (consumed[i] & task_bit) == 0.  The paper does not say how "the required number" is
 *        chosen; this call takes eligible samples in increasing index and returns the longest
 *        prefix of them with at most max_samples entries and, when token_budget > 0, at most
 *        token_budget tokens in total -- except that a first eligible sample longer than the
 *        whole budget is returned alone.  out_idx[0 .. count) (device, capacity max_samples)
 *        receives the indices in increasing order, *out (device) the record below, and the
 *        returned samples get task_bit set in consumed.  The result is unique (integer work).
 * clear: ready[i] &= ~column_bits, consumed[i] &= ~task_bits for every sample (a new iteration).
 *
 * All three enqueue on `stream` and return; read *out / out_idx after synchronising (or place
 * them in mapped pinned memory).  Calls on one table must not overlap on the GPU.
 * Errors: AF_ERR_INVALID_ARG for null pointers, negative sizes, max_samples < 0, a task_bit that
 * is not a single bit, or token_budget > 0 without length; AF_ERR_SHAPE for N >= 2^31.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int64_t n_samples;        /* N                                       */
  uint32_t* ready;          /* [N] dev                                 */
  uint32_t* consumed;       /* [N] dev                                 */
  const int32_t* length;    /* [N] dev, or NULL (no token budgets)     */
} af_controller_view;

typedef struct {
  int32_t count;            /* samples returned                                         */
  int32_t eligible;         /* eligible samples in the table when the request was made  */
  int64_t tokens;           /* their token total (0 without length)                     */
} af_get_result;

af_status af_controller_put(af_ctx* ctx, const af_controller_view* table, const int32_t* idx,
                            int64_t n, uint32_t column_bits, void* stream);
af_status af_controller_get(af_ctx* ctx, const af_controller_view* table, uint32_t column_mask,
                            uint32_t task_bit, int32_t max_samples, int64_t token_budget,
                            int32_t* out_idx, af_get_result* out, void* stream);
af_status af_controller_clear(af_ctx* ctx, const af_controller_view* table, uint32_t column_bits,
                              uint32_t task_bits, void* stream);

/* ---------------------------------------------------------------------------------------------
 * af_unpack_microbatch -- per-token results of a task, in packed order -> the store, by metadata.
 *
 * The inverse of af_pack_microbatch for results (Section 4.2 "Interaction Interface": when a task
 * has computed, it writes its results to the storage units according to the metadata, and the
 * controllers learn that the data at these locations can now be consumed).  For j in [0, B) and
 * every listed column k, the packed values at cu[j] .. cu[j+1]-1 (cu as af_pack_microbatch builds
 * it from the same list) are copied, bit for bit, to rows tok_offset[idx[j]] ..
 * tok_offset[idx[j]+1]-1 of the store column; rows of samples not listed keep their contents.
 * Columns hold 4-byte elements (fp32 log-probs, int32 ids).  If `table` is given, the bits
 * `column_bits` of ready[idx[j]] are set afterwards on the same stream (what af_controller_put
 * does), so that a later af_controller_get on that stream sees data and status together.
 *
 * Errors: AF_ERR_INDEX for an index outside [0, N); AF_ERR_INVALID_ARG for an index listed twice
 * (two writers of one row have no defined order), for n_cols outside [0, AF_MAX_WRITE_COLS], a
 * NULL column pointer while there are tokens to move, or a table whose n_samples differs from
 * N; AF_ERR_CAPACITY if the listed samples hold 2^31 tokens or more.  *T_out (host, nullable) receives the token count.  B == 0 is
 * valid and writes nothing.  The call stages its sequence table through pinned host memory (it may
 * wait for the staging slot it reuses) and cannot be recorded into a CUDA graph.
 * ------------------------------------------------------------------------------------------- */
#define AF_MAX_WRITE_COLS 4
typedef struct {
  int32_t n_cols;                          /* columns to write: 0 .. AF_MAX_WRITE_COLS              */
  int32_t reserved;
  const void* packed[AF_MAX_WRITE_COLS];   /* [T] dev, 4-byte elements in packed order               */
  void* store[AF_MAX_WRITE_COLS];          /* [sum L] dev, the store's column of the same element   */
} af_write_cols;

af_status af_unpack_microbatch(af_ctx* ctx, const int64_t* tok_offset_host, int64_t n_samples,
                               const int32_t* idx_host, int32_t B, const af_write_cols* cols,
                               const af_controller_view* table, uint32_t column_bits,
                               int64_t* T_out, void* stream);


/* ---------------------------------------------------------------------------------------------
 * af_plan_token_logprob / af_plan_units -- how af_token_logprob cuts its work (host calls, no GPU).
 *
 * The paper leaves kernel design to the platform; this is the library's own work decomposition,
 * exposed so that it can be inspected and checked without a device.  The fused LM-head kernel
 * processes units: a unit is one row tile of tokens (256 rows for CTA pairs, 128 for single CTAs)
 * times one of v_splits contiguous ranges of 256-column vocabulary tiles; unit u is row tile
 * u / v_splits, range u % v_splits.  `workers` persistent CTA pairs (or CTAs) share the units.
 * Dealt plainly, worker r takes units r, r + workers, ...  Dealt by die (die0_workers > 0), the first
 * die0_workers workers share the units of the first die0_row_tiles row tiles among themselves and
 * the others the rest, so that a row tile's hidden-state panel is cached in one half of L2 only.
 *
 * af_plan_token_logprob fills *plan for a batch of T >= 1 tokens at head shape (d, V) on a part
 * with sm_count SMs of which die0_sms share a die (0: unknown, deal plainly); v_splits and
 * gemm_variant as in af_set_tuning (0 = the library's choice).  af_plan_units gives the units of
 * worker `rank` in [0, workers): *first, *first + *stride, ... below *end.  Over all ranks these
 * lists hold every unit in [0, m_tiles * v_splits) exactly once.  AF_ERR_INVALID_ARG for null
 * pointers, sizes below 1, die0_sms outside [0, sm_count] or a rank outside [0, workers).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int32_t m_tiles;         /* row tiles of the batch                                          */
  int32_t n_tiles;         /* vocabulary tiles of 256 columns                                 */
  int32_t v_splits;        /* vocabulary ranges per row tile                                  */
  int32_t workers;         /* CTA pairs (or CTAs) the launch starts                           */
  int32_t die0_workers;    /* > 0: dealt by die, workers running on the first die             */
  int32_t die0_row_tiles;  /* row tiles whose units the first die's workers share             */
} af_gemm_plan;

af_status af_plan_token_logprob(int64_t T, int32_t d, int32_t V, int32_t sm_count, int32_t die0_sms,
                                int32_t v_splits, int32_t gemm_variant, af_gemm_plan* plan);
af_status af_plan_units(const af_gemm_plan* plan, int32_t rank, int32_t* first, int32_t* stride,
                        int32_t* end);

/* ---------------------------------------------------------------------------------------------
 * af_balance_partitions -- token-balanced split of a batch over k groups (host call, no GPU).
 *
 * The controller's load balancing (Section 4.4, last paragraph): a one-dimensional bin-packing
 * problem solved with the Karmarkar-Karp largest differencing method.  equal_size != 0 is the
 * data-parallel variant (every group gets the same number of samples, up to one when k does not
 * divide n, and the spread of token totals is minimised under that constraint); equal_size == 0
 * is the pipeline-parallel variant (sample counts free).
 *
 * Method: partial solutions are lists of k groups in decreasing order of token sum.  Start with
 * one per sample (equal_size: one per run of k consecutive samples in decreasing length, one
 * sample per group); repeatedly merge the two partial solutions of largest spread (largest minus
 * smallest sum), joining the j-th largest group of the first with the j-th smallest of the
 * second, until one is left.  Ties: samples by (length descending, index ascending); equal
 * spreads in order of creation; equal sums keep their order.  Group g of the result has the
 * g-th largest token total.
 *
 * length_host [n] >= 0 (host) in; part_host [n] (host) out, values in [0, k);
 * group_tokens_host [k] (host, nullable) out.  AF_ERR_INVALID_ARG for null pointers, n < 0,
 * k < 1 or a negative length.
 * ------------------------------------------------------------------------------------------- */
af_status af_balance_partitions(const int32_t* length_host, int32_t n, int32_t k, int32_t equal_size,
                                int32_t* part_host, int64_t* group_tokens_host);

/* ---------------------------------------------------------------------------------------------
 * af_token_logprob_static -- af_token_logprob for callers that are not allowed to allocate.
 *
 * (The paper has no counterpart for this call; it exists for the sake of embedding.)  Some hosts
 * of this library cannot call cudaMalloc on the path that scores tokens: code running while a
 * memory pool owns the whole device, a serving loop with a frozen memory plan, a plug-in handed
 * only the buffers its caller chose to give it.  For them this entry point computes what
 * af_token_logprob computes, with the same arguments, but takes no context and keeps its only
 * scratch (the per-range online-softmax partials) in a fixed array inside the library's device
 * image: 2 MiB + 256 B that every GPU loading the library holds until the process exits.  The call
 * itself never calls cudaMalloc, cudaFree or an allocating library routine.
 *
 * Kernel and results: always the one-CTA-per-tile main loop (gemm_variant 1 of af_set_tuning),
 * with the number of vocabulary ranges cut down to what the fixed array holds (4 x 32768 partials).
 * Its results agree with af_token_logprob within the log-prob tolerance (2e-3 absolute); they are
 * bit-equal only to a context set to gemm_variant 1 that happens to use the same number of ranges.
 *
 * Limit: 0 <= T <= 32768 tokens per call (AF_ERR_CAPACITY above that); d, V, pointers and
 * alignment as for af_token_logprob.  Runs on the current CUDA device, which must be compute
 * capability 10.0.
 * First call on a device: resolves the array's device address (cudaGetSymbolAddress), reads the SM
 * count, fetches the tensor-map encoder and sets the kernel's shared-memory limit.  With lazy
 * module loading this is also when the driver loads the library's kernels and materialises the
 * array, which allocates device memory inside the driver; so make that first call during start-up,
 * before memory is frozen and before any stream capture begins.
 * Sharing: every call on a device uses the same array.  Nothing in it has to start at zero (a
 * call overwrites each partial before reading it, so stale contents of an earlier call are
 * harmless), but two calls that overlap on the GPU -- different streams, no ordering -- race on
 * it and corrupt each other's results.  Serialise them (one stream, or events).
 * device_flags: optional device pointer to a caller-owned uint32 that receives the AF_DEVERR_*
 * bits (OR-ed in; clear it yourself).  With NULL the bits are OR-ed into a word of the fixed
 * array's header that nothing reads: they are lost, and a target outside [0, V) then shows only as
 * a NaN log-prob.  entropy and lse are optional; a NULL one is not written.
 * ------------------------------------------------------------------------------------------- */
af_status af_token_logprob_static(const void* hidden, const void* W, const int32_t* target,
                                  int64_t T, int32_t d, int32_t V, float* logp, float* entropy,
                                  float* lse, uint32_t* device_flags, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ASYNCFLOW_H_ */

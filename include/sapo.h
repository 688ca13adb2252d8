/*
 * sapo.h — C ABI of the SAPO policy-scoring library for NVIDIA B200 (sm_100a).
 *
 * One SAPO node's policy update (paper Algorithm 1: the steps that put the training set
 * together and update the policy) scores a batch made of I locally generated and J swarm-sampled
 * rollouts per question.  This library runs the data-parallel part of that update:
 *
 *   sapo_pack_rollouts     training set T^n = {local picks} U {external picks}
 *                          (Section 3.2, training-set equation) as a varlen layout
 *   sapo_group_advantages  GRPO group-relative advantages (Section 4.2)
 *   sapo_policy_loss_fwd   LM-head log-probs of the chosen tokens (Section 3.2: rollouts
 *                          are re-encoded and their token-level values computed under the
 *                          node's own policy) + clipped-ratio surrogate, KL weight 0,
 *                          separate lower/upper clip thresholds (Section 4.2)
 *   sapo_policy_loss_bwd   gradient of that loss w.r.t. the final hidden states and the
 *                          LM-head weight (Algorithm 1, the policy-gradient step)
 *   sapo_policy_loss_fwd_bwd  the two above in one call that passes over the logits once
 *                          (bf16 operands; the fastest way through a training step)
 *
 * and, around them:
 *   sapo_select_external            filter and sample the shared pool (Section 3.2 / Section 5)
 *   sapo_policy_loss_bwd_active     backward over the tokens with a gradient only
 *   sapo_policy_loss_fwd_bwd_gather the single-pass call reading the hidden states in place from the
 *                                   rollout stores (the pack then copies none)
 *   sapo_lmhead_lse_partial, sapo_policy_loss_from_partials, sapo_policy_loss_bwd_shard
 *                                   the same loss with W_head sharded by vocabulary over ranks
 *   sapo_adam_step                  the optimiser step of Section 4.2 on the LM head
 *   sapo_policy_loss_fwd_static     the forward for callers that may not allocate device memory
 *   sapo_group_advantages_warp, sapo_workspace_bytes[_min], sapo_status_string, sapo_timing_*,
 *   sapo_launch_count, sapo_debug_wait_timeout, sapo_debug_bounds_violations
 *                                   sizes, texts, measurement and test hooks
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its name starts with h_.  The caller owns
 *     all buffers; the library allocates and frees nothing and keeps no pointer after a
 *     call returns.  Scratch memory is passed in as `workspace`.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *     synchronising.  Results are valid once the stream has drained.
 *   - Return value: SAPO_OK or a negative host-detected error.  Conditions only the device
 *     can see (capacity overflow, index out of range, a bounded wait that ran out) are
 *     OR-ed as SAPO_ST_* bits into *status (int32 in device memory, zeroed by the caller);
 *     the kernels never trap and never spin without a limit.
 *   - Matrices are row-major with the H (hidden) index contiguous.  Base pointers of
 *     hidden / W_head / dhidden / dW_head / workspace must be 16-byte aligned and the
 *     leading dimensions, in bytes, multiples of 16.
 *   - There is no CPU fallback: without a CUDA device every call returns SAPO_ERR_CUDA.
 *   - Threads.  The calls keep a few per-device values they look up on first use (the driver's
 *     tensor-map encoder, the SM count, the shared-memory opt-in and resident CTA pairs of each
 *     kernel, the address of the built-in scratch of sapo_policy_loss_fwd_static) without locks.
 *     Make the first call of each entry point on each device from one thread (a warm-up step does
 *     it); after that, calls from several threads are safe as long as each uses its own stream,
 *     workspace and outputs.  sapo_timing_* and sapo_launch_count are for one thread only.
 */
#ifndef SAPO_H_
#define SAPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* host-detected errors (return values) */
#define SAPO_OK                      0
#define SAPO_ERR_INVALID_ARG        -1
#define SAPO_ERR_UNSUPPORTED_SHAPE  -2
#define SAPO_ERR_WORKSPACE_TOO_SMALL -3
#define SAPO_ERR_CUDA               -4
#define SAPO_ERR_STATIC_SCRATCH_EXCEEDED -5  /* sizes beyond the built-in scratch of the _static call */

/* device-detected conditions (bits of *status) */
#define SAPO_ST_TOKEN_OVERFLOW   0x01  /* packed tokens exceed max_tokens; output truncated   */
#define SAPO_ST_SEQ_OVERFLOW     0x02  /* selected sequences exceed max_seqs; nothing packed  */
#define SAPO_ST_BAD_INDEX        0x04  /* a selection index is outside its rollout buffer     */
#define SAPO_ST_EMPTY_SEQUENCE   0x08  /* a selected rollout has no tokens                    */
#define SAPO_ST_BAD_TOKEN_ID     0x10  /* ids[t] outside [0, V): token scored as masked       */
#define SAPO_ST_WAIT_TIMEOUT     0x20  /* a bounded in-kernel wait ran out; results invalid   */
#define SAPO_ST_NONFINITE_REWARD 0x40  /* a reward is NaN or infinite                         */
#define SAPO_ST_EXP_RANGE        0x80  /* fused call: old_logp[t] is so far from the current
                                          log-prob that exp(z - c_t) left the safe range; the
                                          token is scored as masked: use the separate calls   */
#define SAPO_ST_NONFINITE_INPUT  0x100 /* old_logp[t] or the advantage of its sequence is NaN or
                                          infinite: the token is scored as masked               */

/* element types of hidden / W_head */
#define SAPO_DTYPE_BF16 0
#define SAPO_DTYPE_F32  1  /* converted on the device to split bf16; see sapo_policy_loss_fwd */

/* `which` of sapo_workspace_bytes */
#define SAPO_WS_FWD 0
#define SAPO_WS_BWD 1
#define SAPO_WS_BWD_ACTIVE 2
#define SAPO_WS_FUSED 3
#define SAPO_WS_OUT_BF16 0x100   /* OR into `which`: the gradients will be asked for in bf16 */
#define SAPO_WS_GATHER   0x200   /* OR into `which`: for sapo_policy_loss_fwd_bwd_gather          */

/* A rollout store: n_rollouts completions laid end to end (Section 3.1: a node's answers
 * to its questions; Section 3.2: the tuples other nodes broadcast).
 *   hidden   [n_tokens, H]  final hidden state at the position that predicts ids[t]
 *   ids      [n_tokens]     chosen token
 *   old_logp [n_tokens]     log-prob of ids[t] under the pre-update policy
 *   offsets  [n_rollouts+1] token offset of each completion (offsets[0] = 0)
 *   rewards  [n_rollouts]   reward of each completion */
typedef struct sapo_rollout_buf {
  const void*    hidden;
  const int32_t* ids;
  const float*   old_logp;
  const int64_t* offsets;
  const float*   rewards;
  int32_t        n_rollouts;
} sapo_rollout_buf;

/* Which rollouts enter the training set: for question q the local picks are
 * local_idx[q_offsets_local[q] .. q_offsets_local[q+1]) and the external picks
 * ext_idx[q_offsets_ext[q] .. q_offsets_ext[q+1]).  Either side may be empty. */
typedef struct sapo_selection {
  const int32_t* q_offsets_local;  /* [Q+1] */
  const int32_t* local_idx;
  const int32_t* q_offsets_ext;    /* [Q+1] */
  const int32_t* ext_idx;
  int32_t        Q;
} sapo_selection;

/* Output of sapo_pack_rollouts.  Capacities max_tokens / max_seqs are set by the caller.
 *   hidden [max_tokens, H], ids, old_logp [max_tokens], rewards [max_seqs]
 *   cu_seqlens [max_seqs+1] exclusive prefix sum of sequence lengths
 *   seq_group [max_seqs] question of each sequence;  seq_is_ext [max_seqs] 0 local / 1 external
 *   seq_src [max_seqs] index of the rollout inside its buffer
 *   tok_seq [max_tokens] sequence of each token;  tok_mask [max_tokens] 1 for t < T else 0
 *   group_offsets [Q+1] first sequence of each question
 *   n_tokens, n_seqs: device scalars T and S
 *   tok_src [max_tokens] (optional, may be NULL): where each packed token's row lives in its source
 *     buffer: row index, plus 2^62 when it is the external buffer; -1 for unused slots.  With it the
 *     loss can read the hidden states in place (sapo_policy_loss_fwd_bwd_gather) and `hidden` may
 *     be NULL: the pack then copies no hidden rows at all. */
typedef struct sapo_packed {
  void*    hidden;
  int32_t* ids;
  float*   old_logp;
  float*   rewards;
  int32_t* cu_seqlens;
  int32_t* seq_group;
  uint8_t* seq_is_ext;
  int32_t* seq_src;
  int32_t* tok_seq;
  uint8_t* tok_mask;
  int32_t* group_offsets;
  int32_t* n_tokens;
  int32_t* n_seqs;
  int64_t  max_tokens;
  int32_t  max_seqs;
  int64_t* tok_src;
} sapo_packed;

/* Loss parameters.  The paper's run uses eps_low 0.2, eps_high 0.28 and no KL term
 * (Section 4.2).  grad_scale multiplies the per-token gradient factor (upstream dL).
 * loss_agg: 0 = mean over sequences of the token mean (the default reading), 1 = mean over all
 * tokens (the aggregation of DAPO, which Section 4.2 cites).  kl_beta: weight of a penalty
 * towards a reference policy, per token exp(d) - d - 1 with d = ref_logp[t] - logp[t], aggregated
 * like the surrogate; 0 (the paper's choice) leaves ref_logp unused.  ref_logp: device pointer,
 * [T], may be NULL when kl_beta is 0.  entropy: device pointer [T] or NULL; when given, the forward
 * also writes the entropy of the policy's next-token distribution at every scored position,
 * H_t = - sum_v p[t,v] log p[t,v] (nats), a by-product of the same pass over the logits that RL
 * runs log beside the reward; it does not enter the loss.  Tokens that belong to no sequence get 0. */
typedef struct sapo_loss_cfg {
  float eps_low;
  float eps_high;
  float grad_scale;
  int32_t loss_agg;
  float kl_beta;
  const float* ref_logp;
  float* entropy;
} sapo_loss_cfg;

/* Section 3.2, training-set equation / Algorithm 1, where the training set is put together.
 * Gathers the selected rollouts into one token-major batch.  Sequence order: questions in
 * order; inside a question its local picks in list order, then its external picks in list
 * order.  Copies are byte-exact.  H is the row width in elements, `dtype` a SAPO_DTYPE_*.
 * Slots [T, max_tokens) of hidden, ids and old_logp are zero-filled (tok_mask 0, tok_seq -1),
 * so a caller that must not read n_tokens back can score the whole capacity: the loss calls
 * treat tokens that belong to no sequence as masked.
 * Errors: a NULL struct, a NULL array that the sizes say will be touched (outputs when the
 * capacities are positive, the members of a rollout buffer that holds rollouts; the index lists
 * may be NULL when empty) or a negative size returns SAPO_ERR_INVALID_ARG before anything is
 * launched; a bad index, an empty rollout or a capacity overflow sets the matching status bit
 * (bad or empty picks are packed as length-0 sequences, tokens beyond max_tokens are dropped). */
int sapo_pack_rollouts(const sapo_rollout_buf* h_local, const sapo_rollout_buf* h_ext,
                       const sapo_selection* h_sel, int32_t H, int32_t dtype,
                       const sapo_packed* h_out, int32_t* status, void* stream);

/* Section 4.2 (GRPO): for each question g with members group_offsets[g]..group_offsets[g+1):
 *   mean_g = average reward, std_g = sqrt(sum (r-mean_g)^2 / (G - ddof)),
 *   adv[s] = (rewards[s] - mean_g) / (std_g + adv_eps).
 * The group covers all its completions, local and external alike.  fp32 in, fp32 out; the sums
 * carry their rounding errors along (compensated fp32), so an advantage is within 6 fp32 ulp of
 * the exactly computed value for groups of up to 16 rewards whatever their common offset, and an
 * all-equal group gives exactly 0.  mean / std may be NULL.  A non-finite reward sets
 * SAPO_ST_NONFINITE_REWARD.  Up to 4095 questions run on the warp-level kernel (two lanes per
 * question, a 16-byte vector of rewards each), more on a thread-per-question kernel; sapo_group_advantages_warp always takes the
 * warp-level one (same arguments and results; it exists so that kernel can be measured alone). */
int sapo_group_advantages(const float* rewards, const int32_t* group_offsets, int32_t Q,
                          float adv_eps, int32_t ddof, float* adv, float* mean, float* std,
                          int32_t* status, void* stream);
int sapo_group_advantages_warp(const float* rewards, const int32_t* group_offsets, int32_t Q,
                               float adv_eps, int32_t ddof, float* adv, float* mean, float* std,
                               int32_t* status, void* stream);

/* Section 3.2 (token-level values under the node's own policy) + Section 4.2 (clipped
 * surrogate, KL weight 0).  For T packed tokens in S sequences:
 *   z[t,v] = <hidden[t,:], W_head[v,:]>,  lse[t] = log sum_v exp z[t,v],
 *   logp[t] = z[t, ids[t]] - lse[t],      ratio[t] = exp(logp[t] - old_logp[t]),
 *   surr[t] = min(ratio*A, clip(ratio, 1-eps_low, 1+eps_high)*A),  A = adv[seq of t],
 *   loss    = -(1/S) sum_s (1/T_s) sum_{t in s} surr[t]   (variants: see sapo_loss_cfg),
 *   gscale[t] = dloss/dlogp[t] = -grad_scale * A * ratio / (S*T_s) where the unclipped term
 *               is the min (ties included), else 0.
 * The [T,V] logits are never written to memory: the projection runs on the tensor cores and
 * its epilogue keeps a running max / sum-exp / target logit per token.
 * hidden [T, ld_hidden], W_head [V, ld_W] of `dtype`; for SAPO_DTYPE_F32 the operands are
 * split on the device into bf16 high and low parts (3 products), which keeps log-probs at
 * fp32 accuracy.  adv [S], cu_seqlens [S+1].  Outputs logp, lse, ratio, surr, gscale [T]
 * and loss [1] (float32); seq_surr [S] (token-mean surrogate per sequence) may be NULL.
 * cu_seqlens must be non-decreasing with every entry in [0, T]; normally cu_seqlens[0] = 0 and
 * cu_seqlens[S] = T, but T may also be the capacity of the buffers (sapo_pack_rollouts leaves the
 * token count on the device): tokens of [0, T) before cu_seqlens[0] or from cu_seqlens[S] on
 * belong to no sequence and are scored as masked (all five per-token outputs 0, no gradient).
 * Their hidden rows are still read by the projection and must hold finite numbers
 * (sapo_pack_rollouts zero-fills them).  An entry of cu_seqlens outside [0, T] or below its
 * predecessor is clamped and sets SAPO_ST_BAD_INDEX.  A NaN or infinite old_logp[t] or adv[s]
 * sets SAPO_ST_NONFINITE_INPUT and masks the token(s) (ratio = surr = gscale = 0).
 * workspace: at least sapo_workspace_bytes(SAPO_WS_FWD, ...) bytes.
 * Errors: bad arguments / unaligned pointers -> SAPO_ERR_INVALID_ARG; H or V beyond the
 * supported range -> SAPO_ERR_UNSUPPORTED_SHAPE; small workspace ->
 * SAPO_ERR_WORKSPACE_TOO_SMALL; ids outside [0,V) -> SAPO_ST_BAD_TOKEN_ID and the token
 * gets logp = 0 contribution (surr = gscale = 0). */
int sapo_policy_loss_fwd(const void* hidden, const void* W_head, int32_t dtype,
                         int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                         const int32_t* ids, const float* old_logp, const float* adv,
                         const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                         float* logp, float* lse, float* ratio, float* surr, float* gscale,
                         float* seq_surr, float* loss,
                         void* workspace, size_t workspace_bytes,
                         int32_t* status, void* stream);

/* Algorithm 1 "Policy update" (gradient of the loss above through the LM head):
 *   dz[t,v]      = gscale[t] * ([v == ids[t]] - exp(z[t,v] - lse[t]))
 *   dhidden[t,:] = sum_v dz[t,v] W_head[v,:]        [T, H] of out_dtype
 *   dW_head[v,:] = sum_t dz[t,v] hidden[t,:]        [V, H] of out_dtype
 * Logit tiles are recomputed on the tensor cores; dz is rounded to bf16 and kept in a
 * bounded panel inside `workspace` (token chunks x vocab padded to 128, stored as 16 KB tiles
 * of 128 tokens x 64 vocab entries), from which two tensor-core contractions form dhidden and
 * dW_head.  accumulate_dW != 0 adds into dW_head instead of
 * overwriting it.  lse and gscale come from sapo_policy_loss_fwd.  For SAPO_DTYPE_F32 the
 * operands are rounded to bf16.
 * out_dtype: SAPO_DTYPE_F32, or SAPO_DTYPE_BF16 for gradients that feed a bf16 backward pass and
 * optimiser: contiguous [T, H] / [V, H] of that type, 16-byte aligned; sums are always formed in
 * fp32 and rounded once (when the panel holds fewer than T tokens, or accumulate_dW is set,
 * dW_head is summed in an fp32 copy inside `workspace` and rounded, or added to the caller's
 * values and rounded, at the end: ask sapo_workspace_bytes for SAPO_WS_BWD | SAPO_WS_OUT_BF16).
 * workspace: sapo_workspace_bytes(SAPO_WS_BWD, ...) is the preferred size; any size down to
 * the one for 128 tokens works (smaller panels mean more passes over dW_head). */
int sapo_policy_loss_bwd(const void* hidden, const void* W_head, int32_t dtype,
                         int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                         const int32_t* ids, const float* lse, const float* gscale,
                         void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                         void* workspace, size_t workspace_bytes,
                         int32_t* status, void* stream);

/* The loss over a vocabulary that is sharded across ranks (no counterpart in the paper, whose
 * nodes each hold a whole model; it lets one node's LM head span several GPUs).  Rank r holds
 * W_shard = rows [vocab_offset, vocab_offset + V_shard) of W_head and every token's hidden state.
 *   1. sapo_lmhead_lse_partial: the projection of the shard on the tensor cores, reduced per token
 *      to triple[0][t] = max_v z log2(e), triple[1][t] = sum_v 2^(z log2(e) - max), triple[2][t] =
 *      z[t, ids[t]] if the chosen token lies in the shard, else 0   (float32 [3][T]).
 *      workspace: sapo_workspace_bytes(SAPO_WS_FWD, T, H, V_shard, dtype).
 *   2. the caller gathers the triples of all ranks into local memory, [n_parts][3][T] (one
 *      all-gather of 12 T bytes per rank);
 *   3. sapo_policy_loss_from_partials: merges them (log-sum-exp over the parts) and evaluates the
 *      loss tail exactly as sapo_policy_loss_fwd does; every rank computes the same values.
 *      ids are the global token ids, V the whole vocabulary.  h_cfg->entropy must be NULL.
 *   4. sapo_policy_loss_bwd_shard: sapo_policy_loss_bwd on the shard with the global lse:
 *      dW_shard [V_shard, H] is this rank's rows of dW_head; dhidden is this shard's share of
 *      the sum over the vocabulary, to be added up over the ranks (one all-reduce of T H values).
 * The library itself moves nothing between GPUs; a kernel only ever reads local memory. */
int sapo_lmhead_lse_partial(const void* hidden, const void* W_shard, int32_t dtype,
                            int64_t T, int32_t H, int32_t V_shard, int64_t ld_hidden, int64_t ld_W,
                            const int32_t* ids, int32_t vocab_offset, float* triple,
                            void* workspace, size_t workspace_bytes, int32_t* status, void* stream);
int sapo_policy_loss_from_partials(const float* triples, int32_t n_parts, int64_t T, int32_t V,
                                   const int32_t* ids, const float* old_logp, const float* adv,
                                   const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                   float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                   float* seq_surr, float* loss, int32_t* status, void* stream);
int sapo_policy_loss_bwd_shard(const void* hidden, const void* W_shard, int32_t dtype,
                               int64_t T, int32_t H, int32_t V_shard, int64_t ld_hidden, int64_t ld_W,
                               const int32_t* ids, int32_t vocab_offset, const float* lse,
                               const float* gscale, void* dhidden, void* dW_shard, int32_t out_dtype,
                               int32_t accumulate_dW, void* workspace, size_t workspace_bytes,
                               int32_t* status, void* stream);

/* The same gradient, computed over the active tokens only (gscale[t] != 0).  Sequences of a
 * zero-advantage group — which the paper's experiments drop from the shared pool as
 * uninformative (Section 5) — and tokens clipped on the binding side have gscale = 0 and add
 * nothing to either gradient; this call compacts them away first (order kept), gathers the
 * hidden rows of the rest, runs the three contractions on those rows and writes dhidden rows
 * back to their token positions (inactive rows are zero).  The active count is read on the
 * device by the kernels, so the call does not synchronise; if n_active_out (device int32) is not
 * NULL the count is also copied there.  Results equal sapo_policy_loss_bwd up to fp32 summation
 * order.  workspace: sapo_workspace_bytes(SAPO_WS_BWD_ACTIVE, ...) (the regular backward's plus
 * a compacted copy of hidden and four per-token vectors). */
int sapo_policy_loss_bwd_active(const void* hidden, const void* W_head, int32_t dtype,
                                int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                const int32_t* ids, const float* lse, const float* gscale,
                                void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                                int32_t* n_active_out,
                                void* workspace, size_t workspace_bytes,
                                int32_t* status, void* stream);

/* Loss (Section 3.2 + Section 4.2) and both gradients (Algorithm 1 "Policy update") in ONE call
 * that passes over the logits once.  Same definitions and outputs as sapo_policy_loss_fwd followed
 * by sapo_policy_loss_bwd; what changes is how the softmax is carried from the forward to the
 * backward contraction.  With a per-token reference
 *   c_t = z[t, ids[t]] - old_logp[t]          (one dot product per token, computed first)
 * — equal to lse[t] if the policy has not moved since old_logp was taken, and off by
 * log ratio[t] otherwise — the forward epilogue forms e[t,v] = exp(z[t,v] - c_t), adds it up per
 * token in fp32 (lse[t] = c_t + log sum_v e[t,v]; no running maximum is needed) and keeps e,
 * rounded to bf16, in a panel inside `workspace` (token chunks x vocab padded to 128, 16 KB tiles
 * of 128 tokens x 64 vocab entries).  Then, with sum_t = sum_v e[t,v] and a_t = -gscale[t] / sum_t,
 *   dz[t,v] = gscale[t] ([v == ids[t]] - e[t,v] / sum_t) = a_t e'[t,v],  e' = e - [v == ids[t]] sum_t,
 * so after patching one panel entry per token
 *   dhidden[t,:] = a_t sum_v e'[t,v] W_head[v,:]     (row scale in the epilogue)
 *   dW_head[v,:] = sum_t e'[t,v] (a_t hidden[t,:])   (scaled bf16 copy of hidden as operand)
 * are two tensor-core contractions over the panel: 6 T V H flops instead of the 8 T V H of the
 * separate calls, which recompute the logits.  The price is the range of e: if old_logp[t] is so
 * stale that |log ratio| approaches 69 (the sum of e reaches 2^100 or drops below 2^-100), the token
 * is scored as masked (surr = gscale = 0) and SAPO_ST_EXP_RANGE is set; such batches need the
 * separate calls.  bf16 operands only (SAPO_DTYPE_F32 returns SAPO_ERR_UNSUPPORTED_SHAPE).
 * Arguments as in the two separate calls.  workspace: sapo_workspace_bytes(SAPO_WS_FUSED, ...)
 * is the preferred size (a panel of up to 32768 tokens); any size down to
 * sapo_workspace_bytes_min(SAPO_WS_FUSED, ...) works, the batch is then processed in token
 * chunks and dW_head accumulated over them.  seq_surr may be NULL (then S <= T is required). */
int sapo_policy_loss_fwd_bwd(const void* hidden, const void* W_head, int32_t dtype,
                             int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                             const int32_t* ids, const float* old_logp, const float* adv,
                             const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                             float* logp, float* lse, float* ratio, float* surr, float* gscale,
                             float* seq_surr, float* loss,
                             void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                             void* workspace, size_t workspace_bytes,
                             int32_t* status, void* stream);

/* sapo_policy_loss_fwd_bwd with the hidden states read in place.  The training set is a union of
 * index picks (Section 3.2, training-set equation), so it need not be copied: every packed token
 * names its row in the local or the external rollout store (tok_src, written by
 * sapo_pack_rollouts, which then copies no hidden rows when its `hidden` output is NULL), the
 * projection's row loads follow the runs of consecutive rows that whole sequences form, and the
 * per-token kernels read their row through the same map.  local_hidden [n_local_tokens, ld_hidden],
 * ext_hidden [n_ext_tokens, ld_hidden] (bf16, the same row pitch, 16-byte aligned; fewer than 2^31
 * rows each); everything else, results included, as in sapo_policy_loss_fwd_bwd.  A packed slot
 * without a token (tok_src -1) is scored as masked; a tok_src that points outside its store sets
 * SAPO_ST_BAD_INDEX.  workspace: sapo_workspace_bytes(SAPO_WS_FUSED | SAPO_WS_GATHER, ...). */
int sapo_policy_loss_fwd_bwd_gather(const void* local_hidden, int64_t n_local_tokens,
                                    const void* ext_hidden, int64_t n_ext_tokens, const int64_t* tok_src,
                                    const void* W_head, int32_t dtype,
                                    int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                    const int32_t* ids, const float* old_logp, const float* adv,
                                    const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                    float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                    float* seq_surr, float* loss,
                                    void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* status, void* stream);

/* Section 3.2 (nodes filter and sample what the swarm shares) / Section 5 (the experiments'
 * policy: discard rollouts with zero advantage, then sample uniformly from the rest).
 * The pool holds n_entries rollouts; entry g is a question's group of completions with rewards
 * rewards[group_offsets[g] .. group_offsets[g+1]).  An entry whose rewards are all equal has zero
 * advantage throughout and is dropped; of the others, J are drawn uniformly without replacement
 * (all of them if there are fewer than J): entry g gets the key
 * (philox4x32-10(counter = (g,0,0,0), key = (seed low, seed high))[0] << 32) | g and the J
 * smallest keys win, so the draw depends only on the seed and the pool.  selected [J] receives
 * the chosen entries in pool order, *n_selected how many there are, *n_candidates how many passed
 * the filter (all device memory).  workspace: sapo_select_workspace_bytes(n_entries), 8-byte
 * aligned. */
int sapo_select_external(const float* rewards, const int32_t* group_offsets, int32_t n_entries,
                         int32_t J, uint64_t seed, int32_t* selected, int32_t* n_selected,
                         int32_t* n_candidates, void* workspace, size_t workspace_bytes, void* stream);
size_t sapo_select_workspace_bytes(int32_t n_entries);

/* Section 4.2: the policy is updated with Adam (default hyper-parameters, learning rate 0.001).
 * One Adam step (Kingma & Ba, Algorithm 1) on a [rows, cols] weight such as W_head, from the
 * fp32 gradient sapo_policy_loss_bwd wrote:
 *   m <- beta1 m + (1-beta1) g;  v <- beta2 v + (1-beta2) g^2;
 *   master <- master - lr * (m / (1-beta1^step)) / (sqrt(v / (1-beta2^step)) + eps).
 * master, m, v, grad: fp32 [rows, cols], contiguous, 16-byte aligned, updated in place (grad is
 * only read).  w_bf16 (may be NULL): bf16 [rows, ld_w] copy of the new master weight, rounded to
 * nearest even — the operand the next forward reads.  step counts from 1.  cols % 4 == 0. */
int sapo_adam_step(float* master, float* m, float* v, const float* grad, void* w_bf16,
                   int64_t rows, int32_t cols, int64_t ld_w, int32_t step,
                   float lr, float beta1, float beta2, float eps, void* stream);

/* Bytes of scratch the forward (SAPO_WS_FWD), backward (SAPO_WS_BWD, SAPO_WS_BWD_ACTIVE) or
 * fused (SAPO_WS_FUSED) call wants for these sizes; OR SAPO_WS_OUT_BF16 into `which` for a call
 * with bf16 gradient outputs.  Returns 0 for invalid arguments. */
size_t sapo_workspace_bytes(int32_t which, int64_t T, int32_t H, int32_t V, int32_t dtype);

/* Smallest backward or fused workspace that still works (one 128-token panel). */
size_t sapo_workspace_bytes_min(int32_t which, int64_t T, int32_t H, int32_t V, int32_t dtype);

/* Forward pass without caller-provided scratch (the paper has no counterpart; this exists for
 * hosts that are not allowed to allocate device memory: a component embedded in a process whose
 * memory pool is fixed once at start-up, or a loop that must never reach cudaMalloc because it
 * synchronises the whole device).  Same arguments and results as sapo_policy_loss_fwd, and the
 * same argument checks in the same order, except that `workspace` is gone: the scratch is an
 * array of SAPO_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that loads
 * the library carries it until the process ends.  The call itself allocates and frees nothing.
 * Limits, checked after the common argument checks: bf16 operands only
 * (SAPO_ERR_UNSUPPORTED_SHAPE otherwise), and
 *     24 * T bytes  (+ 4 * S, rounded up to 256, when seq_surr is NULL)  <=  SAPO_STATIC_SCRATCH_BYTES,
 * i.e. up to 174,762 tokens (32 * T and 131,072 tokens when h_cfg->entropy is given); beyond that
 * the call does nothing and returns SAPO_ERR_STATIC_SCRATCH_EXCEEDED.  The forward keeps 24 (32)
 * bytes per token and vocab split; this
 * entry takes as many of the splits the regular call would use as fit in the array.  When all of
 * them fit the results are bit-identical to sapo_policy_loss_fwd; with fewer splits they agree up
 * to the order in which a token's partial sums are added (and large batches of few tokens per SM
 * pair run somewhat slower).
 * The first call on each device looks up the array's device address (that device must be
 * current); make that first call outside any stream capture, and from one thread.  All calls on
 * a device share the one array and it keeps whatever the previous call left: nothing in it needs
 * clearing between calls, but two calls that may run on the GPU at the same time (different
 * streams, or different threads) race on it and must be ordered by the caller. */
#define SAPO_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int sapo_policy_loss_fwd_static(const void* hidden, const void* W_head, int32_t dtype,
                                int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                const int32_t* ids, const float* old_logp, const float* adv,
                                const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                float* seq_surr, float* loss, int32_t* status, void* stream);

/* Optional per-kernel timing for benchmarks (no counterpart in the paper).  While enabled,
 * every kernel launch of the library is bracketed by two CUDA events recorded on the call's
 * stream.  sapo_timing_read waits for the recorded events, writes the summed milliseconds and
 * the number of launches per kernel id (arrays of SAPO_K_COUNT) and forgets them; at most 16384
 * launches are kept between reads.  The events are created on the first enable.  Not thread-safe.
 * sapo_launch_count returns how many kernels the library has launched in this process. */
#define SAPO_K_PACK_SCAN  0
#define SAPO_K_PACK_COPY  1
#define SAPO_K_GROUP_ADV  2
#define SAPO_K_SPLIT_BF16 3
#define SAPO_K_FWD_GEMM   4
#define SAPO_K_LOSS_TAIL  5
#define SAPO_K_LOSS_FINAL 6
#define SAPO_K_BWD_DZ     7
#define SAPO_K_BWD_DH     8
#define SAPO_K_BWD_DW     9
#define SAPO_K_STREAMK_FIXUP 10
#define SAPO_K_COMPACT   11
#define SAPO_K_SELECT    12
#define SAPO_K_ADAM      13
#define SAPO_K_TARGET_LOGIT 14
#define SAPO_K_FWD_EXP   15
#define SAPO_K_FUSED_TAIL 16
#define SAPO_K_COUNT      17
int sapo_timing_enable(int32_t on);
int sapo_timing_read(float* h_ms, int32_t* h_launches);
int64_t sapo_launch_count(void);

/* The library's in-kernel waits (on the barriers between the copy, tensor-core and epilogue
 * roles of the GEMM kernels) are bounded: a wait that runs out makes the kernel set
 * SAPO_ST_WAIT_TIMEOUT, let its copies in flight land, free its tensor memory and return, so the
 * context stays usable.  This call (no counterpart in the paper) exercises exactly that code on a
 * barrier nobody arrives at: one thread waits limit_clocks SM clocks (at most 10^8, about 50 ms),
 * then sets the bit in *status.  For tests of a caller's error handling. */
int sapo_debug_wait_timeout(int64_t limit_clocks, int32_t* status, void* stream);

/* Checked builds (the library compiled with -DSAPO_BOUNDS_CHECK, see build.py): the kernels compare
 * every index they compute before a global-memory access with the extent of its array, count a
 * violation and leave the access out.  Returns the number of violations counted so far in this
 * process, or -1 when the library is a regular build. */
int64_t sapo_debug_bounds_violations(void);

/* Text for a return code. */
const char* sapo_status_string(int32_t code);

#ifdef __cplusplus
}
#endif
#endif /* SAPO_H_ */

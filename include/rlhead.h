/* rlhead.h - C ABI of the fused LM-head log-probability + GRPO policy-loss library (sm_100a).
 *
 * The library evaluates, for a batch of token positions, the quantities of the policy-update
 * step of Algorithm 1 (its advantage-estimation step and its policy-update step, Eq. 6): GRPO
 * group-normalised advantages (section 4.2), the
 * log-probability of every sampled token under the next-token policy over the vocabulary
 * (section 2.2), its entropy (section 2.2 "Regularization"), the clipped importance-ratio
 * surrogate (section 3.1) with a KL-to-reference regulariser, and the gradient of the resulting
 * loss with respect to the hidden states H and the LM-head weight W.  The [T,V] logits are
 * never written to memory.
 *
 * Conventions
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.
 *     The library allocates only inside rl_ctx (a few KB of device memory for counters and the
 *     status word) and otherwise works in the caller-provided workspace.
 *   - All functions return rl_status; 0 is success.  Nothing throws, traps or aborts.
 *   - Calls enqueue work on the context's stream and return; argument errors are reported
 *     synchronously, errors found on the device (token id outside [0,V) on a valid row, a
 *     bounded wait that ran out) are latched in a device status word read by
 *     rl_last_device_status().
 *   - H is [T,d] bf16 row-major with row stride ldH elements, W is [V,d] bf16 row-major with
 *     row stride ldW elements (the layout of a linear layer's weight).  Row t of H is the hidden
 *     state whose next-token distribution scores tokens[t].  d must be a multiple of 64; ldH
 *     and ldW multiples of 8; H and W base addresses 16-byte aligned (TMA requirements).
 *   - mask is one byte per row (non-zero = the token takes part in the loss); NULL means all
 *     valid.  Rows with mask 0 are skipped entirely (padding-free execution, section 4.4):
 *     their outputs are 0 and their token ids are ignored.
 *   - T = 0 or an all-zero mask is not an error: loss 0, gradients 0.
 *   - A context is not thread-safe: use one context per host thread (contexts are cheap), or
 *     serialise the calls on it.  Calls on different contexts may run concurrently as long as
 *     their workspaces differ.
 */
#ifndef RLHEAD_H_
#define RLHEAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RL_OK = 0,
  RL_ERR_INVALID_ARG = 1,      /* NULL required pointer, negative size, bad hyper-parameter   */
  RL_ERR_SHAPE = 2,            /* d not a multiple of 64, group_size does not divide n_seq ... */
  RL_ERR_ALIGNMENT = 3,        /* base pointer or leading dimension breaks the TMA rules       */
  RL_ERR_WORKSPACE = 4,        /* workspace missing or smaller than rl_workspace_bytes()       */
  RL_ERR_CUDA = 5,             /* a CUDA runtime / driver call failed                          */
  RL_ERR_UNSUPPORTED_ARCH = 6, /* device is not compute capability 10.x                        */
  RL_ERR_TOKEN_RANGE = 7,      /* device: token id outside [0,V) on a valid row                */
  RL_ERR_TIMEOUT = 8           /* device: a bounded wait inside a kernel ran out               */
} rl_status;

typedef struct rl_ctx rl_ctx;  /* opaque; one per device and stream */

/* Context.  rl_create checks that `device` is compute capability 10.x, allocates the context's
 * small device block and uses the legacy default stream until rl_set_stream is called. */
rl_status rl_create(rl_ctx** out, int device);
rl_status rl_destroy(rl_ctx* ctx);
rl_status rl_set_stream(rl_ctx* ctx, void* cuda_stream);
const char* rl_status_string(rl_status s);

/* Bytes of scratch needed by any call with at most T rows, hidden size d, vocabulary V.  The
 * size does not grow with T*V: the gradient with respect to the logits only ever exists for a
 * bounded slab of rows x vocabulary columns. */
rl_status rl_workspace_bytes(rl_ctx* ctx, int64_t T, int64_t d, int64_t V, size_t* bytes);
/* The same for calls that set rl_loss_opts.kl_full with a reference model of hidden size d_ref
 * (adds the compacted reference rows and five per-row arrays). */
rl_status rl_workspace_bytes_kl(rl_ctx* ctx, int64_t T, int64_t d, int64_t V, int64_t d_ref, size_t* bytes);
/* Size of the slab the backward pass works in: at most max_rows token rows x max_cols vocabulary
 * columns of the gradient with respect to the logits exist at a time (bf16, in the workspace).
 * max_rows a multiple of 128, max_cols a multiple of 256, max_rows * max_cols at most 2^31; 0 restores a
 * default (32768 x 37888: 2.5 GB of slab at most, chosen so that the tile counts of the dlogits and dW
 * passes are multiples of the 74 SM pairs for d = 2048, 2560 and 3584; half as many columns cost 0.5-1.7 %
 * of a step in launch ramps and accumulator traffic).  Changes what rl_workspace_bytes() returns: call it
 * first. */
rl_status rl_set_slab_limits(rl_ctx* ctx, int max_rows, int max_cols);
/* Tile shape of the tensor-core passes: 1 = one CTA per 128x256 output tile, 2 = CTA pairs
 * (clusters of two SMs, tcgen05 cta_group::2) on 256x256 tiles, which halves the shared-memory
 * and L2 traffic of the B operand.  2 is the default when the device can co-schedule CTA pairs;
 * asking for 2 when it cannot returns RL_ERR_UNSUPPORTED_ARCH.  Results are identical up to fp32 summation order inside the tensor core. */
rl_status rl_set_cta_group(rl_ctx* ctx, int cta_group);
/* Upper bound (1..4, default 1) on the number of slices the K range of a dH tile may be cut
 * into.  With more than one slice the dH pass picks, on the device, the slice count that evens
 * out its last wave of tiles; every slice accumulates into its own fp32 buffer and the buffers
 * are summed in slice order when dH is written, so results stay reproducible.  Costs
 * (max_slices - 1) extra [slab rows x d] fp32 buffers of workspace: call before
 * rl_workspace_bytes().  On the measured workloads the gain was within 1 %. */
rl_status rl_set_dh_k_slices(rl_ctx* ctx, int max_slices);
/* Tile shape of the two long-K gradient products, dH = G W and dW = G^T H (default on, used when the
 * tensor-core passes run as CTA pairs and neither rl_set_dh_k_slices nor rl_set_dh_stream_k is in
 * effect): 256 x 512 output tiles that fill both accumulators of tensor memory, so a CTA pulls a
 * quarter fewer operand bytes from L2 per flop, at the price of not overlapping a tile's epilogue
 * with the next tile's main loop (about 1 % of a tile at K of 17-19 thousand).  Off: 256 x 256 tiles
 * with a double-buffered accumulator, as the forward and gradient-of-logits passes always use.
 * Results are bit-identical either way.  Measured: 3.4-4.1 % of a step on the four large workloads. */
rl_status rl_set_wide_tiles(rl_ctx* ctx, int on);
/* L2 working set of the two passes that walk their tiles rows-first (forward statistics and the
 * gradient-of-logits slab).  Every CTA of such a pass re-reads its panel of compacted hidden rows
 * (256 rows x d, bf16) once per vocabulary tile; when the panels of all row tiles together exceed
 * what L2 keeps (126 MB shared with the streamed operand), each re-read goes to DRAM.  The row
 * tiles are therefore taken in equal groups whose panels fit `bytes` (default 36 MiB), and all
 * vocabulary tiles are walked for one group before the next group starts; the rows of W are then
 * read once per group instead of once per launch.  0 = one group.  Results do not depend on it.
 * Measured: 2 % (16896 rows, d = 2048) to 11 % (32768-row slabs, d = 2560 / 3584) of a step. */
rl_status rl_set_row_group_bytes(rl_ctx* ctx, int64_t bytes);
/* Load balancing of the dH pass (default off).  The pass has (row tiles x d/256) output tiles; when
 * that count is not a multiple of the number of SM pairs the last wave of tiles leaves most SMs
 * idle (7.14 waves at d = 2048 with 16896 rows).  With stream-K on, the last full wave and the
 * ragged wave are instead cut, by tile x k-block iterations, into equal contiguous shares, one per
 * SM pair; a tile that straddles two shares is completed in a second fp32 accumulator buffer,
 * summed when dH is written.  Every element still has one writer per buffer and launch, so
 * results stay reproducible run to run.  Costs one extra [slab rows x d] fp32 buffer of
 * workspace: call before rl_workspace_bytes().  Ignored while rl_set_dh_k_slices() asks for more
 * than one slice.  Measured: the dH pass itself gets about 7 % faster at 16896 rows, but a
 * whole step on a board that sits at its power limit does not (the other passes slow down by as
 * much), which is why it is opt-in. */
rl_status rl_set_dh_stream_k(rl_ctx* ctx, int on);
/* Upper bound on the CTAs of the persistent tensor-core grids (default: one per SM).  A caller that
 * overlaps a collective with the backward pass (sections 4.3 / 4.4: sharded training engines) can
 * leave a few SMs to the collective's kernels this way; an odd bound is rounded down to whole CTA
 * pairs.  0 restores the default.  Results do not depend on it except where the forward pass
 * chooses its vocabulary split from the number of workers (summation order of the merge).
 * Errors: max_ctas < 0 or, after rounding, fewer than 2 -> RL_ERR_INVALID_ARG. */
rl_status rl_set_max_ctas(rl_ctx* ctx, int max_ctas);
/* Gradient hand-over for data-parallel training (the paper has no kernel-level counterpart; its
 * training engines all-reduce gradients after the backward pass).  The backward pass finishes dW
 * one slab of vocabulary rows at a time.  When a hook is set, rl_policy_loss_fwd_bwd[_ex] calls
 * hook(user, slab, row_begin, row_end) on the calling host thread right after it has ENQUEUED the
 * launch that completes rows [row_begin, row_end) of dW: work the hook enqueues behind an event
 * recorded on the context's stream at that moment (for instance an all-reduce of those rows on
 * another stream) runs while the remaining slabs are still being computed.  Slabs are reported in
 * ascending order and cover [0, V) exactly once per call; nothing is reported for T = 0 (dW is then
 * zero, or untouched when accumulating).  hook = NULL removes it.  The hook must not call into
 * this context. */
typedef void (*rl_dw_slab_hook)(void* user, int slab, int64_t row_begin, int64_t row_end);
rl_status rl_set_dw_slab_hook(rl_ctx* ctx, rl_dw_slab_hook hook, void* user);
/* Caller-owned device scratch, 256-byte aligned; must outlive the calls that use it. */
rl_status rl_set_workspace(rl_ctx* ctx, void* dev_ptr, size_t bytes);

/* Synchronises the context's stream and returns the latched device status (RL_OK,
 * RL_ERR_TOKEN_RANGE or RL_ERR_TIMEOUT), then clears it.  detail (host, may be NULL) receives a
 * kernel-specific word describing where the first error was seen. */
rl_status rl_last_device_status(rl_ctx* ctx, int32_t* detail);

/* GRPO advantages - the advantage-estimation step of Algorithm 1; section 3.2.2 advantage
 * estimation stage; section 4.2 (normalisation of the rewards within each group of responses).
 * rewards[n_seq] holds one scalar per response (section 3.2.2 scoring stage), the group_size
 * responses of a prompt stored consecutively.  adv_seq[i] = (r_i - mean_g) / (std_g + eps_std);
 * a group whose rewards are all equal gets exactly 0.  The basic call uses the sample standard
 * deviation (ddof = 1) and eps_std = 1e-6.  With seq_offsets[n_seq+1] (row range of each
 * response) and adv_tok[T] non-NULL the per-response value is also broadcast to every row of
 * the response (rows outside every range get 0); T = seq_offsets[n_seq].
 * Errors: group_size < 2 or n_seq % group_size != 0 -> RL_ERR_SHAPE; ddof not 0/1, eps_std < 0,
 * NULL rewards/adv_seq -> RL_ERR_INVALID_ARG. */
rl_status rl_grpo_advantages(rl_ctx* ctx, const float* rewards, int64_t n_seq, int group_size,
                             float* adv_seq);
rl_status rl_grpo_advantages_ex(rl_ctx* ctx, const float* rewards, int64_t n_seq, int group_size,
                                int ddof, float eps_std, const int32_t* seq_offsets,
                                int64_t T, float* adv_seq, float* adv_tok);

/* The other critic-free advantage estimators that section 4.2 names (the leave-one-out baseline
 * of RLOO, the length-weighted baseline of OPO, REINFORCE++) on the same grouped layout.  The
 * paper prints no formula for them; the readings are
 *   RL_ADV_GRPO          as rl_grpo_advantages (sample std, eps_std as given)
 *   RL_ADV_RLOO          A_i = r_i - mean of the other responses of the group (group_size >= 2)
 *   RL_ADV_OPO           A_i = r_i - sum_j(len_j r_j) / sum_j(len_j) over the group; lengths[n_seq]
 *                        (int32, valid tokens per response) required
 *   RL_ADV_REINFORCE_PP  c_i = r_i - group mean, then A_i = (c_i - mean(c)) / (std(c) + eps_std) over
 *                        the whole batch (population std, fp64 fixed-order reduction)
 * Errors as rl_grpo_advantages_ex. */
typedef enum { RL_ADV_GRPO = 0, RL_ADV_RLOO = 1, RL_ADV_OPO = 2, RL_ADV_REINFORCE_PP = 3 } rl_adv_estimator;
rl_status rl_advantages(rl_ctx* ctx, int estimator, const float* rewards, const int32_t* lengths,
                        int64_t n_seq, int group_size, float eps_std, float* adv_seq);

/* Token-level KL reward shaping - section 2.2 "Regularization": the KL-to-reference regulariser
 * applied as per-token rewards rather than (or beside) a loss term.  The paper prints no formula;
 * the reading is: every valid row t of response i gets the shaped reward r_t = -beta * kl_t, the
 * last valid row of the response additionally seq_value[i] (the trajectory reward of the scoring
 * stage, section 3.2.2, or a group-normalised advantage from rl_grpo_advantages), and
 * returns[t] = r_t + gamma * returns[next valid row of the same response] (gamma = 1: the reverse
 * cumulative sum), to be used as the per-row adv[T] of the loss calls.  kl_t is chosen by
 * kl_estimate: RL_KL_K1 the signed log-ratio logp[t] - ref_logp[t]; RL_KL_K3 exp(delta) - delta - 1
 * with delta = ref_logp[t] - logp[t] (the estimator the loss uses); RL_KL_GIVEN kl_tok[t] as handed
 * in (for instance rl_loss_opts.kl_out of a full-distribution pass).
 * seq_value[n_seq], seq_offsets[n_seq+1] (ascending row ranges, seq_offsets[n_seq] <= T), logp,
 * ref_logp, kl_tok, mask (NULL = all valid), returns[T] and shaped_reward[T] (may be NULL) are
 * device pointers; the arrays a kl_estimate does not read may be NULL.  Rows with mask 0 and rows
 * outside every range get 0, carry no reward and do not count as a discount step; a response
 * without a valid row drops its seq_value.  Sums run in double precision, one warp per response,
 * in a fixed order (reproducible).  Needs no workspace.
 * Errors: beta < 0, gamma < 0, unknown kl_estimate, NULL required pointer -> RL_ERR_INVALID_ARG. */
typedef enum { RL_KL_K1 = 0, RL_KL_K3 = 1, RL_KL_GIVEN = 2 } rl_kl_estimate;
rl_status rl_kl_shaped_returns(rl_ctx* ctx, const float* seq_value, const float* logp, const float* ref_logp,
                               const float* kl_tok, const uint8_t* mask, const int32_t* seq_offsets,
                               int64_t n_seq, int64_t T, float beta, float gamma, int kl_estimate,
                               float* shaped_reward, float* returns);

/* The per-token loss arithmetic on its own: Eq. 6 (negated) with the clipped importance-ratio surrogate of
 * section 3.1 and the k3 estimate of the KL-to-reference term of section 2.2, from per-token quantities the
 * caller already holds (for instance the merged output of the vocabulary-parallel calls, or log-probabilities
 * scored by another engine):
 *     rho_t = exp(logp_t - old_logp_t),   s_t = min(rho_t A_t, clip(rho_t, 1 - eps_low, 1 + eps_high) A_t),
 *     delta_t = ref_logp_t - logp_t,      k3_t = exp(delta_t) - delta_t - 1,
 *     loss = sum_t w_t (-s_t + beta k3_t - ent_coef Ent_t),
 * w_t = token_weight[t] if given, else mask_t / (number of rows with mask != 0, or *token_count if given: the
 * data-parallel global count, a device int64).  All arrays are device pointers of T floats in the original row
 * order; mask[T] bytes or NULL (every row valid); entropy may be NULL when ent_coef == 0 (the entropy metric
 * is then 0); ref_logp NULL iff beta == 0.  Outputs: loss[1]; dlogp[T] = d loss / d logp_t and dentropy[T] =
 * d loss / d Ent_t = -w_t ent_coef (either may be NULL; rows with mask 0 get 0); metrics_out[8] or NULL, laid
 * out as rl_loss_opts.metrics_out.  A count pass over the mask, one pass of four rows per thread (16-byte
 * loads and stores when every array is 16-byte aligned) and a fixed-order reduction in double: reproducible.
 * Needs no workspace (the context owns 64 KB for the block sums).  T == 0: loss 0, RL_OK.
 * Errors: eps_low outside [0, 1), eps_high < 0, beta < 0, ent_coef < 0, NULL required pointer -> RL_ERR_INVALID_ARG. */
rl_status rl_token_loss(rl_ctx* ctx, const float* logp, const float* entropy, const float* old_logp,
                        const float* ref_logp, const float* adv, const uint8_t* mask, int64_t T, float eps_low,
                        float eps_high, float beta, float ent_coef, const float* token_weight, const void* token_count,
                        float* loss, float* dlogp, float* dentropy, float* metrics_out);

/* Padding-free row map on its own (section 4.4, training without padding tokens): row_map[i] = index of
 * the i-th row with mask != 0, ascending, for i < *n_valid; entries past that are left untouched.
 * mask NULL = all rows valid.  row_map[T] (int32) and n_valid[1] (int32) are device pointers; the
 * workspace needs (T / 4096 + 3) * 4 bytes.  Every other call of this library runs the same
 * three kernels internally; this entry exists so that the map can be checked and timed by itself.
 * Errors: T < 0 or T >= 2^31, NULL outputs -> RL_ERR_INVALID_ARG; RL_ERR_WORKSPACE. */
rl_status rl_mask_scan(rl_ctx* ctx, const uint8_t* mask, int64_t T, int32_t* row_map, int32_t* n_valid);

/* Per-token log-probability of the sampled token, entropy and log-sum-exp of the next-token
 * distribution softmax(W h_t) - section 2.2 (policy over the vocabulary; importance ratio
 * numerator) and section 2.2 "Regularization" (entropy).  Natural logarithms.
 * logp[T] required; entropy[T] and lse[T] may be NULL.  Masked rows get 0. */
rl_status rl_token_logprobs(rl_ctx* ctx, const void* H, int64_t ldH, const void* W, int64_t ldW,
                            const int32_t* tokens, const uint8_t* mask,
                            int64_t T, int64_t d, int64_t V,
                            float* logp, float* entropy, float* lse);

/* Loss of Eq. 6 (negated, to be minimised) and its gradients.
 *   rho_t  = exp(logp_t - old_logp_t)                                   (section 2.2)
 *   s_t    = min(rho_t A_t, clip(rho_t, 1-eps_low, 1+eps_high) A_t)     (section 3.1)
 *   k3_t   = exp(delta_t) - delta_t - 1, delta_t = ref_logp_t - logp_t  (KL-to-reference)
 *   loss   = sum_t w_t (-s_t + beta k3_t - ent_coef Ent_t),  w_t = mask_t / sum(mask)
 * loss[1] is a device scalar.  dH[T,d] (bf16, row stride d; masked rows 0) and dW[V,d] (fp32,
 * row stride d) are fully overwritten.  adv is per row [T].  ref_logp may be NULL iff beta == 0.
 * Errors: eps_low outside [0,1), eps_high < 0, beta < 0, NULL required pointer ->
 * RL_ERR_INVALID_ARG; shape/alignment/workspace as above. */
rl_status rl_policy_loss_fwd_bwd(rl_ctx* ctx, const void* H, int64_t ldH, const void* W,
                                 int64_t ldW, const int32_t* tokens, const float* old_logp,
                                 const float* ref_logp, const float* adv, const uint8_t* mask,
                                 int64_t T, int64_t d, int64_t V,
                                 float eps_low, float eps_high, float beta,
                                 float* loss, void* dH, float* dW);

/* Options of the extended call.  Zero-initialise, set struct_size = sizeof(rl_loss_opts). */
typedef struct {
  size_t struct_size;
  float ent_coef;             /* entropy bonus coefficient (section 2.2), >= 0                 */
  const float* token_weight;  /* [T] or NULL: replaces w_t = mask_t/sum(mask) by               */
                              /* token_weight[t]*mask_t (the length normalisation by token     */
                              /* weights that section 2.2 lists among the regularisers)        */
  int accumulate_dW;          /* non-zero: dW += gradient instead of overwrite                 */
  float* logp_out;            /* [T] or NULL                                                   */
  float* entropy_out;         /* [T] or NULL                                                   */
  float* metrics_out;         /* [8] or NULL: pg_loss, kl_mean, entropy_mean, clip_frac,       */
                              /* ratio_mean, ratio_max, n_valid, reserved                      */
  int agg_mode;               /* token weights when token_weight is NULL: 0 token mean over    */
                              /* the call; 1 mean over responses of each response's token mean */
                              /* (w = mask/(n_seq*len_i)); 2 mean over responses of the token  */
                              /* sum over the longest row range (w = mask/(n_seq*L_max))       */
  int sequence_level;         /* non-zero: sequence-level importance ratio (the GSPO variant   */
                              /* named in section 4.2; reading: rho_i = exp(mean               */
                              /* token log-ratio over the valid tokens of response i), used    */
                              /* and clipped for every token of the response                   */
  int dH_dtype;               /* 0: dH is bf16 [T,d]; 1: dH is fp32 [T,d]                      */
  const int32_t* seq_offsets; /* [n_seq+1] ascending row range of every response, needed by    */
  int64_t n_seq;              /* agg_mode 1/2 and sequence_level; seq_offsets[n_seq] <= T;     */
                              /* valid rows outside every range then take no part in the loss  */
                              /* (the token mean of agg_mode 0 is over the rows inside ranges; */
                              /* metrics_out[6] still counts every valid row)                  */
  int kl_full;                /* non-zero: the regulariser is the full-distribution            */
                              /* KL(pi_theta(.|s_t) || pi_ref(.|s_t)) = sum_j p_j (log p_j -   */
                              /* log q_j) over the vocabulary, as sections 2.2 and 3.1 print   */
                              /* it, instead of the sampled-token k3 estimate; q = softmax(    */
                              /* W_ref h_ref_t) is recomputed tile by tile next to p, never    */
                              /* stored.  ref_logp is then unused (may be NULL).  Not          */
                              /* combined with sequence_level / agg_mode 1, 2 (INVALID_ARG).   */
  const void* H_ref;          /* [T, d_ref] bf16 device, row stride ldH_ref: hidden states of  */
  int64_t ldH_ref;            /* the frozen reference model for the same rows                  */
  const void* W_ref;          /* [V, d_ref] bf16 device, row stride ldW_ref: its LM head       */
  int64_t ldW_ref;
  int64_t d_ref;              /* multiple of 64 (whole 128-byte k-slices), strides multiples   */
                              /* of 8, bases 16-byte aligned; the reference model is a         */
                              /* constant: no gradient flows to H_ref / W_ref                  */
  float* kl_out;              /* [T] or NULL: per-token KL_t of the kl_full mode (masked rows 0) */
  const int64_t* token_count; /* device scalar or NULL: the token mean (agg_mode 0 without          */
                              /* token_weight) divides by *token_count instead of this call's own  */
                              /* number of valid rows.  Data-parallel ranks pass the count summed   */
                              /* over ranks, so that the per-rank losses and gradients add up to    */
                              /* those of the global batch; it is read on the device in stream      */
                              /* order, the host never sees it.  Not used by the response-aware     */
                              /* paths (sequence_level, agg_mode 1 / 2).                            */
} rl_loss_opts;

rl_status rl_policy_loss_fwd_bwd_ex(rl_ctx* ctx, const void* H, int64_t ldH, const void* W,
                                    int64_t ldW, const int32_t* tokens, const float* old_logp,
                                    const float* ref_logp, const float* adv, const uint8_t* mask,
                                    int64_t T, int64_t d, int64_t V,
                                    float eps_low, float eps_high, float beta,
                                    float* loss, void* dH, float* dW, const rl_loss_opts* opts);

/* One whole step with the per-step inputs in HOST memory (pinned memory gives asynchronous
 * copies): H, tokens, old_logp, ref_logp, mask and either adv (per row) or rewards[n_seq] +
 * seq_offsets[n_seq+1] are host pointers, copied to the device inside the call; when adv_host is
 * NULL the advantages are computed on the device from the rewards as rl_grpo_advantages does and
 * broadcast over seq_offsets.  W, dH and dW stay device pointers (weights and gradients live on
 * the device); loss_host[1] and metrics_host[8] (may be NULL) are written on the host.  ldH must
 * equal d.  The call synchronises the context's stream before returning.  The workspace must
 * have been sized with rl_workspace_bytes_host(). */
rl_status rl_workspace_bytes_host(rl_ctx* ctx, int64_t T, int64_t d, int64_t V, size_t* bytes);
rl_status rl_policy_loss_fwd_bwd_host(rl_ctx* ctx, const void* H_host, int64_t ldH, const void* W,
                                      int64_t ldW, const int32_t* tokens_host,
                                      const float* old_logp_host, const float* ref_logp_host,
                                      const float* adv_host, const float* rewards_host,
                                      int64_t n_seq, int group_size,
                                      const int32_t* seq_offsets_host, const uint8_t* mask_host,
                                      int64_t T, int64_t d, int64_t V,
                                      float eps_low, float eps_high, float beta, float ent_coef,
                                      float* loss_host, float* metrics_host, void* dH, float* dW);

/* Scoring with several models in one call - Algorithm 1 evaluates the same sampled tokens under
 * the old policy pi_theta_old (its old-policy refresh step; importance-ratio denominator of
 * section 2.2) and under the frozen reference pi_ref (section 3.2.1, Reference role) before the
 * update.  Model i has hidden states H[i] ([T, d[i]] bf16, row stride ldH[i]) and LM head W[i]
 * ([V, d[i]] bf16, row stride ldW[i]); tokens, mask, T and V are shared.  The arrays H, ldH, W,
 * ldW, d, logp, entropy are HOST arrays of n_models (1..16) entries holding device pointers /
 * sizes; logp[i][T] required, entropy (the array, or single entries) may be NULL.  The mask is
 * scanned once and every model reuses the row map; each model then takes one sweep over its own
 * W.  Workspace: rl_workspace_bytes() with the largest d[i].  Errors as rl_token_logprobs. */
rl_status rl_token_logprobs_multi(rl_ctx* ctx, int n_models, const void* const* H, const int64_t* ldH,
                                  const void* const* W, const int64_t* ldW, const int64_t* d,
                                  const int32_t* tokens, const uint8_t* mask, int64_t T, int64_t V,
                                  float* const* logp, float* const* entropy);

/* Vocabulary-parallel LM head - for training engines that shard the model states so that the
 * head weight is never resident on one GPU in full (the sharded training engines of section 4.3
 * and the memory discussion of section 4.4).  The rows of W are partitioned over ranks; this rank
 * holds W_shard[V_shard, d] =
 * rows [vocab_offset, vocab_offset + V_shard) of the V_total-row head.  tokens are ids in
 * [0, V_total) (checked against V_total; an id outside this rank's slice simply has no logit
 * here).  The three calls compute exactly what rl_token_logprobs and rl_policy_loss_fwd_bwd_ex
 * compute on one device; between them the caller moves 16 bytes per row (all-gather of the
 * statistics) and the partial dH (all-reduce).
 *
 * rl_shard_logit_stats: stats[T][4] (fp32, 16-byte aligned) receives per row (M, S, A, z_y) over the
 *   slice: M = max_j z_j, S = sum_j exp(z_j - M), A = sum_j exp(z_j - M) z_j, z_y = the logit of
 *   the sampled token if its id lies in the slice, else 0.  Masked rows get four zeros.
 * rl_merge_logit_stats: stats[n_shards][T][4] -> logp[T], entropy[T] (may be NULL), lse[T] (may be
 *   NULL) over the whole vocabulary; masked rows 0.  Slices are combined in index order, so every
 *   rank that merges the same gathered array gets the same bits.
 * rl_policy_loss_shard_bwd: arguments as rl_policy_loss_fwd_bwd_ex plus the slice position and the
 *   merged logp, entropy, lse ([T] each, as rl_merge_logit_stats wrote them).  loss[1] is the loss
 *   of the whole vocabulary (every rank computes the same value: do not sum it over ranks);
 *   dH_partial[T,d] is this slice's contribution to dH (sum over ranks = dH; ask for fp32 with
 *   opts->dH_dtype = 1 when it is to be all-reduced); dW_shard[V_shard,d] is this rank's rows of dW.
 *   opts->kl_full is not supported here (RL_ERR_INVALID_ARG).
 * Errors: vocab_offset < 0 or vocab_offset + V_shard > V_total -> RL_ERR_SHAPE; the rest as the
 * single-device calls.  Workspace: rl_workspace_bytes(T, d, V_shard). */
rl_status rl_shard_logit_stats(rl_ctx* ctx, const void* H, int64_t ldH, const void* W_shard, int64_t ldW,
                               const int32_t* tokens, const uint8_t* mask, int64_t T, int64_t d,
                               int64_t V_shard, int64_t vocab_offset, int64_t V_total, float* stats);
rl_status rl_merge_logit_stats(rl_ctx* ctx, const float* stats, int n_shards, const uint8_t* mask,
                               int64_t T, float* logp, float* entropy, float* lse);
rl_status rl_policy_loss_shard_bwd(rl_ctx* ctx, const void* H, int64_t ldH, const void* W_shard,
                                   int64_t ldW, const int32_t* tokens, const float* old_logp,
                                   const float* ref_logp, const float* adv, const uint8_t* mask,
                                   int64_t T, int64_t d, int64_t V_shard, int64_t vocab_offset,
                                   int64_t V_total, const float* logp, const float* entropy,
                                   const float* lse, float eps_low, float eps_high, float beta,
                                   float* loss, void* dH_partial, float* dW_shard,
                                   const rl_loss_opts* opts);

/* The same step split in two, so that the host-to-device copies of one step overlap the kernels of
 * the step before it (a trainer that receives rollout batches in host memory: Algorithm 1 runs
 * mu policy updates per sampled batch).  rl_policy_loss_fwd_bwd_host_submit copies the inputs of a
 * step on a copy stream that belongs to the context into staging slot `slot` (0 or 1), makes the
 * context's stream wait for them, enqueues the step there and returns without synchronising;
 * rl_policy_loss_fwd_bwd_host_wait blocks until the step submitted to that slot has finished and
 * returns its loss and metrics.  A slot must be waited for before it is submitted to again
 * (RL_ERR_INVALID_ARG otherwise); steps run in submission order and share dH / dW as the caller
 * passes them, so a step's dH and dW are valid between its wait and the submit after next at the
 * latest - with one dH / dW pair, read them before submitting the next step, or alternate two pairs.
 * The host buffers of a step must stay untouched until its wait returns; pinned memory is needed for
 * the copies to be asynchronous.  Workspace: rl_workspace_bytes_host_pipelined() (two staging
 * slots).  The first submit on a context creates the copy stream, four events and 128 bytes of
 * pinned memory, released by rl_destroy. */
rl_status rl_workspace_bytes_host_pipelined(rl_ctx* ctx, int64_t T, int64_t d, int64_t V, size_t* bytes);
rl_status rl_policy_loss_fwd_bwd_host_submit(rl_ctx* ctx, int slot, const void* H_host, int64_t ldH,
                                             const void* W, int64_t ldW, const int32_t* tokens_host,
                                             const float* old_logp_host, const float* ref_logp_host,
                                             const float* adv_host, const float* rewards_host,
                                             int64_t n_seq, int group_size,
                                             const int32_t* seq_offsets_host, const uint8_t* mask_host,
                                             int64_t T, int64_t d, int64_t V,
                                             float eps_low, float eps_high, float beta, float ent_coef,
                                             void* dH, float* dW);
rl_status rl_policy_loss_fwd_bwd_host_wait(rl_ctx* ctx, int slot, float* loss_host, float* metrics_host);

/* rl_token_logprobs without any device allocation and without a context (the paper has no
 * counterpart).  It is meant for callers that cannot allocate GPU memory when they need
 * log-probabilities: a scoring pass that shares the GPU with another engine which has already
 * reserved almost all of its memory, so that a cudaMalloc of the workspace would fail, or code
 * that must not pay the device-wide synchronisation cudaMalloc / cudaFree imply.  Inputs and
 * outputs are the caller's device buffers exactly as in
 * rl_token_logprobs; everything in between (compacted rows, row map, per-range softmax
 * statistics, the status word) lives in a fixed 16 MiB device array that is part of the library
 * image, so every GPU on which the library is loaded holds those 16 MiB until the process exits.
 *   Limit: the forward scratch, about Tpad*(2*d + 28 + 16*R) + 70 KB bytes with Tpad = T rounded up
 *   to 128 and R = max(16, ceil(ceil(V/256)/8)) vocabulary ranges, must fit in 16 MiB - 256 B (e.g.
 *   T <= 3712 at d = 2048 for V <= 32768; T <= 3072 at d = 2048 and T <= 1664 at d = 4096 for the
 *   151936-word vocabulary, where R = 75); larger
 *   sizes are rejected with RL_ERR_WORKSPACE before anything is enqueued.
 *   The call runs on the CURRENT device (device ordinal < 16) and enqueues on cuda_stream.  The
 *   first call on each device looks up the array's device address and configures the kernel; make
 *   that first call before any stream capture begins.  No cudaMalloc, cudaFree or other allocating
 *   routine is called, on the first call or later.
 *   All calls on a device share the one array and it keeps the previous call's contents; the call
 *   clears what has to start at zero (status word, valid-row count) itself.  Two calls whose GPU
 *   work overlaps (different streams, or different host threads on different streams) race on the
 *   array: serialise them on one stream or with events.  Host-side the call is thread-safe.
 *   dev_status (device, int32[2], may be NULL) receives {status, detail} as rl_last_device_status
 *   would report them (RL_ERR_TOKEN_RANGE / RL_ERR_TIMEOUT), written in stream order ({0, 0} when
 *   T = 0). */
rl_status rl_token_logprobs_static(void* cuda_stream, const void* H, int64_t ldH, const void* W,
                                   int64_t ldW, const int32_t* tokens, const uint8_t* mask,
                                   int64_t T, int64_t d, int64_t V,
                                   float* logp, float* entropy, float* lse, int32_t* dev_status);

/* Instrumentation.  rl_launch_count: kernels this context has launched so far.
 * rl_set_profiling(on): when on, every kernel (or group of small kernels) is bracketed by a pair of CUDA events
 * on the context's stream (at most 65536 launch groups are kept between two reads; later ones go untimed).
 * rl_profile_read: synchronises the stream and returns, per kernel kind (0 forward statistics,
 * 1 gradient-of-logits slab, 2 dH, 3 dW, 4 mask scan, 5 row gather, 6 merge + per-token loss,
 * 7 dH scatter, 8 advantages), the summed device time in milliseconds ms[9] (host) and the number
 * of timed launch groups launches[9] (host) since the previous read.  The paper has no
 * counterpart; these exist so that a benchmark can report per-kernel roofline figures. */
rl_status rl_launch_count(rl_ctx* ctx, int64_t* n);
rl_status rl_set_profiling(rl_ctx* ctx, int on);
rl_status rl_profile_read(rl_ctx* ctx, double* ms, int64_t* launches);

/* Self-test of the tensor-core GEMM engine the calls above are built from: C[M,N] (fp32,
 * row-major, ldc = N) = A * B with bf16 operands.  a_mn_major = 0: A is [M,K] row-major;
 * 1: A is stored [K,M] row-major.  b_mn_major = 0: B is stored [N,K] row-major; 1: B is stored
 * [K,N] row-major.  M, N multiples of 64, K a multiple of 8.  The paper has no counterpart; this
 * entry exists so that the operand layouts can be checked against a library product. */
rl_status rl_selftest_gemm(rl_ctx* ctx, const void* A, const void* B, float* C,
                           int64_t M, int64_t N, int64_t K, int a_mn_major, int b_mn_major,
                           int accumulate);

/* Measurement of data movement between the CTAs of a thread-block cluster through distributed shared
 * memory (the paper has no counterpart; it prices designs that would keep the gradient with respect
 * to the logits on chip).  mode 0: per round every CTA of a cluster of cluster_size (2, 4 or 8) sums
 * its 128 / cluster_size rows of the 128 x 128 fp32 tiles all CTAs hold (remote loads), rounds to
 * bf16 and writes the result into every CTA's 128 x 128 bf16 tile (remote stores), with two cluster
 * barriers: per CTA (cluster_size - 1) * (128 / cluster_size) * 128 * 4 bytes come in and half as
 * many go out.  mode 1: per round every CTA sends `bytes` (multiple of 16, at most 48 KiB) to the CTA
 * whose rank is its own XOR partner_xor with one bulk shared-to-shared copy that completes on the
 * receiver's barrier, one cluster barrier per round.  The kernel runs `iters` rounds on as many
 * clusters as fit the device (n_clusters_host, may be NULL); ms_host (host) receives the device time
 * of one launch after a warm-up launch.  Synchronises the context's stream. */
rl_status rl_selftest_cluster_exchange(rl_ctx* ctx, int mode, int cluster_size, int iters, int bytes,
                                       int partner_xor, float* ms_host, int* n_clusters_host);

/* Host-only view of how a tensor-core pass distributes its work (no GPU is touched; the paper has
 * no counterpart).  For a pass over n_valid rows (at most rows_cap), K extent k_len, n_tiles column
 * tiles walked n_range at a time (0: split that fills the SMs, or 8 with plenty of work; -h with 1 <= h < 100:
 * chosen in [1, h] as the gradient-of-the-logits pass does; -100 - h: chosen in [8, h] when there is plenty of
 * work, else as 0), with the ordering options
 * of the library (n_fastest, row groups of m_group row tiles, stream-K, K slices) on n_workers
 * workers of cta_group CTAs each, writes one record of eight int32 per work unit, worker by worker
 * in the order the worker walks them: {worker, row tile, first column tile, end column tile,
 * output slice, first k-block, end k-block, k-blocks per tile}.  units (host, may be NULL when
 * max_units is 0) receives at most max_units records, *n_units (host) the total.  It runs the very
 * functions the kernels run, so that a test without a GPU can check that every (tile, k-block) is
 * covered exactly once. */
rl_status rl_debug_schedule(int64_t n_valid, int64_t rows_cap, int64_t k_len, int64_t n_tiles, int n_range,
                            int n_fastest, int m_group, int stream_k, int k_split_max, int cta_group,
                            int n_workers, int32_t* units, int64_t max_units, int64_t* n_units);

/* Self-test of the bounded waits every kernel of this library uses: launches one warp that waits,
 * for at most limit_ms (1..1000) milliseconds, on a barrier nothing ever signals.  The kernel
 * returns by itself with RL_ERR_TIMEOUT latched (detail 0x70000000); rl_last_device_status()
 * reports and clears it and the context stays usable.  The paper has no counterpart. */
rl_status rl_selftest_wait_timeout(rl_ctx* ctx, int limit_ms);

#ifdef __cplusplus
}
#endif
#endif /* RLHEAD_H_ */

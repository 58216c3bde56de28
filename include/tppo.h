/*
 * tppo.h -- C ABI of the B200 (sm_100a) T-PPO token-selective update library.
 *
 * The library computes the part of a Truncated-PPO training step that the paper's method changes:
 * EGAE advantages over possibly truncated responses (Section 3.1, Eq. 6), the policy / value
 * token filter (Section 3.2), and the two losses restricted to the surviving tokens (Eq. 1 and
 * Eq. 4-5; the advantage, policy and value steps of Algorithm 1).
 *
 * Conventions that hold for every entry point
 *   - Every array pointer is a DEVICE pointer unless the comment says "host".  The caller owns all
 *     buffers, the workspace included; the library allocates nothing and keeps no state between
 *     calls -- with one exception, tppo_egae_static, which works in a device array compiled into
 *     the library and remembers that array's address per device (see there).  Scalars are passed
 *     by value.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work and return; they never
 *     synchronise the stream or the device.
 *   - Return value: a tppo_status.  Anything the host can detect (null pointer, negative size,
 *     workspace too small, misalignment, unsupported shape) is reported before any kernel is
 *     launched and leaves all outputs untouched.  Problems only the device can see (a target id
 *     outside [0,V), an index outside its array, a scan wait that ran out, a NaN or infinity in
 *     an input) set bits of a status word in the call's output and the affected outputs are
 *     written as 0 -- never NaN, never a trap.
 *   - Packed token layout: sequence i occupies positions [seq_begin[i], seq_begin[i+1]) laid out
 *     prompt | response tokens of earlier windows | response tokens of this window.
 *   - Workspace: query tppo_workspace_bytes() with the same sizes, pass at least that many bytes,
 *     256-byte aligned.  Contents need no initialisation and are garbage afterwards.  Two calls
 *     that may overlap on the GPU need different workspaces.
 */
#ifndef TPPO_H
#define TPPO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TPPO_OK = 0,
    TPPO_ERR_INVALID_ARG = 1, /* null / negative / inconsistent argument, bad alignment      */
    TPPO_ERR_WORKSPACE = 2,   /* workspace pointer null, misaligned or smaller than required */
    TPPO_ERR_UNSUPPORTED = 3, /* valid request this library cannot serve                     */
    TPPO_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch error, wrong device)     */
    TPPO_ERR_TOO_LARGE = 5    /* problem exceeds a fixed built-in capacity (see *_static)    */
} tppo_status;

/* bits of the device status word */
enum {
    TPPO_DEV_BAD_TARGET = 1,  /* targets[row] outside [0, V): that row contributes nothing   */
    TPPO_DEV_WAIT_TIMEOUT = 2,/* a bounded look-back wait gave up: outputs incomplete        */
    TPPO_DEV_BAD_INDEX = 4,   /* a row / token index outside its array: entry skipped        */
    TPPO_DEV_BAD_SEGMENT = 8, /* segment bounds outside [0, N] or not ascending: skipped     */
    TPPO_DEV_OVERFLOW = 16,   /* an output buffer was too small: the excess was not written  */
    TPPO_DEV_NONFINITE = 32   /* a NaN or infinity was met in an input: see each entry point */
};

typedef enum {
    TPPO_OP_EGAE = 0,
    TPPO_OP_SELECT_TOKENS = 1,
    TPPO_OP_POLICY_LOSS = 2,
    TPPO_OP_VALUE_LOSS = 3,
    TPPO_OP_LMHEAD = 4
} tppo_op;

/* logits element types */
enum { TPPO_BF16 = 0, TPPO_F32 = 1 };

/* where the gradient with respect to the logits goes */
enum {
    TPPO_DLOGITS_NONE = 0,    /* forward only (e.g. the old-policy log-probs of Algorithm 1)  */
    TPPO_DLOGITS_FULL = 1,    /* [R, ld] like the logits; rows that are not selected are     */
                              /* zero-filled; may be the logits buffer itself (in place)     */
    TPPO_DLOGITS_COMPACT = 2  /* [n_max, V] dense, row j belongs to the j-th selected row    */
};

/* Library version (major*10000 + minor*100 + patch). Host call. */
int tppo_version(void);

/* Human-readable name of a status code (static string, host). */
const char *tppo_status_string(int status);

/*
 * For tests of the give-up paths of the two kernels that wait on other thread blocks (the scan of
 * tppo_egae and the compaction of tppo_select_tokens, both decoupled look-back chains).  Host call;
 * it changes a process-wide setting that later calls of those two entry points read:
 *   lookback_polls  >= 0: a look-back gives up after this many failed polls of a round of tiles
 *                   (normally about four million); < 0 restores the normal limit
 *   no_publish      != 0: tiles do not publish their partial results, so that every look-back that
 *                   has to wait runs into the limit -- deterministically, without any fault
 * A call made under these settings returns normally with TPPO_DEV_WAIT_TIMEOUT set; its outputs are
 * incomplete but finite and in bounds.  tppo_test_hooks(-1, 0) restores normal operation.
 */
void tppo_test_hooks(int32_t lookback_polls, int32_t no_publish);

/*
 * Workspace bytes needed by one call of `op`.  N = packed tokens, B = sequences / segments,
 * n_max = capacity of the selected-token list, V = vocabulary (0 where it does not apply).
 * Returns 0 for an unknown op.  Host call, launches nothing.
 */
size_t tppo_workspace_bytes(int op, int64_t N, int32_t B, int64_t n_max, int32_t V);

/*
 * EGAE advantages and Monte-Carlo returns (Section 3.1, Eq. 6 with the TD residual of Eq. 3;
 * R_t as defined after Eq. 5; the advantage step of Algorithm 1).
 *
 * For each response segment [seg_begin[i], seg_end[i]) of the packed arrays, backwards in t:
 *     delta_t = rewards[t] + gamma * V(s_{t+1}) - values[t]
 *     A_t     = delta_t + gamma*lambda * A_{t+1},   A_end = 0
 *     R_t     = rewards[t] + gamma * R_{t+1},       R_end = 0
 * where V(s_{t+1}) = values[t+1] inside the segment and, after the last token, 0 if the response
 * finished, else bootstrap[i] -- or, when bootstrap is NULL, values[seg_end[i]-1], the paper's
 * assumption V(s_l) = V(s_{l-1}) for a response cut at the window length l.
 *
 *   rewards, values  [N] fp32      seg_begin, seg_end  [B] int32, ascending, disjoint,
 *   truncated        [B] u8                            0 <= begin <= end <= N (empty allowed)
 *   bootstrap        [B] fp32 or NULL
 *   advantages       [N] fp32 out; returns [N] fp32 out or NULL.  Positions outside every
 *                    segment are written 0.
 *   status           [1] int32 out: device status bits (0 = clean).
 * A reward, value or used bootstrap value inside a segment that is a NaN or an infinity is read as
 * 0 and raises TPPO_DEV_NONFINITE, so the outputs stay finite.
 * Precision: the advantage is carried as G_t = A_t + values[t] (G_t = rewards[t] + gamma*(1-lambda)*
 * V(s_{t+1}) + gamma*lambda*G_{t+1}, so successive values never cancel).  Everything carried across
 * runs of 16 consecutive positions, warps and tiles is fp64 (the composite map of each run
 * included); inside a run the results are evaluated in fp32 from the entering value rounded once.
 * The error of a result is that rounding plus at most 16 fp32 roundings at the magnitude of |G| or
 * |R| inside its run; it does not grow with the length of a response.  N < 2^31.
 * Arrays that are 16-byte aligned take the fast path (TMA copies); others are still handled.
 * The first call in a process looks up the driver's tensor-map encoder (without it every tile takes
 * the slower plain-load path; no error).
 */
int tppo_egae(const float *rewards, const float *values,
              const int32_t *seg_begin, const int32_t *seg_end,
              const uint8_t *truncated, const float *bootstrap,
              int32_t B, int64_t N, float gamma, float lambda,
              float *advantages, float *returns, int32_t *status,
              void *workspace, size_t workspace_bytes, void *stream);

/*
 * tppo_egae without a caller workspace and without any allocation.  (The paper has no counterpart:
 * this is a packaging variant of tppo_egae, same arithmetic, same outputs.)
 *
 * Who needs it: code that runs where device memory cannot be requested -- a plug-in inside a
 * training or serving runtime that has already reserved the whole device for its own pool (a raw
 * cudaMalloc there fails or fragments the pool), or a latency-critical section that must not pay
 * cudaMalloc's device-wide synchronisation -- and that has no spare buffer of its own to lend as
 * workspace.  The scan's tile descriptors live in a fixed array compiled into the library
 * (TPPO_EGAE_STATIC_MAX_TOKENS / 2048 descriptors of 64 bytes plus one counter, about 128 KB); every
 * GPU that loads the library holds that array until the process exits.
 *
 * Arguments and results are those of tppo_egae minus the workspace pair.  Differences:
 *   - N > TPPO_EGAE_STATIC_MAX_TOKENS returns TPPO_ERR_TOO_LARGE before anything is launched.
 *   - The first call on each device looks up the device address of the built-in array (the device
 *     must be current, as for every call) and caches it; make that first call outside any stream
 *     capture.  Later calls only enqueue a clear of the array and the kernel.  The cached address
 *     belongs to the device's current context: after cudaDeviceReset it is stale, and the entry
 *     point must not be used again in that process.
 *   - All calls on a device share the one array, which still holds the previous call's contents:
 *     each call clears it on `stream` before the scan.  Two calls that can overlap on the GPU
 *     (different streams without an ordering between them) race on it and give undefined results;
 *     order them, or use tppo_egae with separate workspaces.
 * The function calls no cudaMalloc / cudaFree and no allocating library routine.
 */
#define TPPO_EGAE_STATIC_MAX_TOKENS 4194304
int tppo_egae_static(const float *rewards, const float *values,
                     const int32_t *seg_begin, const int32_t *seg_end,
                     const uint8_t *truncated, const float *bootstrap,
                     int32_t B, int64_t N, float gamma, float lambda,
                     float *advantages, float *returns, int32_t *status, void *stream);

/*
 * Token filter and compaction (Section 3.2; "selective filtering of prompt and truncated tokens").
 * With o = p - seq_begin[i] for the sequence i that holds position p:
 *   policy token  iff  prompt_len[i]+prev_len[i] <= o < prompt_len[i]+prev_len[i]+new_len[i]
 *                                                       - (truncated[i] ? drop_i : 0)
 *                      (response tokens generated in the current step, finished or not, minus
 *                      the last drop_i tokens of an unfinished sequence; drop_i = tail_drop_seq[i]
 *                      when that array is given, else tail_drop: the paper leaves the number of
 *                      excluded latest tokens open, so it is a parameter, per call or per sequence)
 *   value token   iff  !truncated[i] and prompt_len[i] <= o < prompt_len[i]+prev_len[i]+new_len[i]
 *                      (all generated tokens of finished sequences)
 * each ANDed with the optional byte masks (non-zero = keep).  Prompt tokens are in neither set.
 *
 *   seq_begin [B+1] int32 ascending; prompt_len, prev_len, new_len [B] int32 >= 0; truncated [B] u8
 *   tail_drop >= 0; tail_drop_seq [B] int32 or NULL (a negative entry is read as 0 and raises
 *   TPPO_DEV_BAD_INDEX)
 *   extra_policy_mask, extra_value_mask  [N] u8 or NULL
 *   policy_idx, value_idx  [N] int32 out: selected positions in ascending order (bit-exact,
 *                          run-to-run deterministic); entries past the count are untouched
 *   counts   [4] int32 out: n_policy, n_value, device status bits, 0
 * The counts stay on the device so that the loss calls can consume them without a host round trip.
 */
int tppo_select_tokens(const int32_t *seq_begin, const int32_t *prompt_len,
                       const int32_t *prev_len, const int32_t *new_len,
                       const uint8_t *truncated, int32_t tail_drop, const int32_t *tail_drop_seq,
                       const uint8_t *extra_policy_mask, const uint8_t *extra_value_mask,
                       int32_t B, int64_t N,
                       int32_t *policy_idx, int32_t *value_idx, int32_t *counts,
                       void *workspace, size_t workspace_bytes, void *stream);

/*
 * Fused per-token log-softmax gather + clipped PPO surrogate, forward and backward to the logits
 * (Eq. 1 with decoupled eps_low / eps_high; token-level mean and no KL term per Section 4.1.1;
 * the policy update of Algorithm 1).  For the j-th selected row r = rows[j] (j < n), a = aux_idx[j]:
 *     logp_j = x[r, y] - log sum_v exp(x[r, v]),            y = targets[r]
 *     rho    = exp(logp_j - old_logp[a])
 *     l_j    = -min(rho*adv[a], clip(rho, 1-eps_low, 1+eps_high)*adv[a])
 *     loss   = (1/denom) * sum_j l_j
 *     dlogits[., v] = (adv[a]*rho*active/denom) * (softmax_v - 1[v == y])
 * with active = 0 exactly when the clipped term is strictly the smaller one (the gradient is then
 * zero), and n = min(*n_sel, n_max).  Each selected logits row is read once from HBM.
 *
 *   logits    [R, ld] elements of logits_dtype (TPPO_BF16 or TPPO_F32), row stride ld >= V
 *   targets   [R] int32: the token scored by logits row r (the caller applies the next-token shift)
 *   rows      [n_max] int32 distinct row indices, or NULL for 0..n_max-1
 *   n_sel     [1] int32 device count (e.g. counts+0 of tppo_select_tokens) or NULL for n_max
 *   aux_idx   [n_max] int32 index into old_logp / adv, or NULL to use the row index
 *   old_logp, adv   fp32, length aux_len (bounds-checked against it)
 *   denom     > 0: divisor of the mean (gradient accumulation / several GPUs); <= 0: n
 *   logp, token_loss  [n_max] fp32 out, compact, either may be NULL
 *   loss      [1] fp32 out
 *   stats     [4] int32 out: n, rows clipped at the lower edge, at the upper edge, status bits
 *   dlogits   per dlogits_mode (same element type as the logits); FULL mode may alias `logits`
 *   kernel_hint  0 = choose automatically; other values select a specific kernel for tuning and
 *                testing and never change the result beyond rounding (see tppo_policy_kernels)
 * Zero selected rows give loss 0 and no gradient writes beyond FULL mode's zero fill.
 * Reductions are done in a fixed order: results are run-to-run identical.
 * Range: exp(x - max) is formed from the difference, so finite logits of any magnitude are handled,
 * and -inf logits (a masked vocabulary entry) count as probability 0.  A selected row that holds a
 * NaN or +inf, or nothing but -inf, has no log-softmax: it contributes nothing (logp, loss term and
 * gradient row 0) and raises TPPO_DEV_NONFINITE.
 */
int tppo_policy_loss_fwd_bwd(const void *logits, int32_t logits_dtype,
                             int64_t R, int32_t V, int64_t ld,
                             const int32_t *targets,
                             const int32_t *rows, const int32_t *n_sel, int64_t n_max,
                             const int32_t *aux_idx,
                             const float *old_logp, const float *adv, int64_t aux_len,
                             float eps_low, float eps_high, float denom,
                             float *logp, float *token_loss, float *loss, int32_t *stats,
                             void *dlogits, int32_t dlogits_mode, int32_t kernel_hint,
                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * Forward-only sweep with statistics: the log-probs of the old-policy snapshot (the step of
 * Algorithm 1 that sets pi_theta_old before the updates; the same gather as above, one read of each
 * selected row, no gradient) together with two diagnostics taken from the same pass.  For the j-th
 * selected row r = rows[j] (j < n = min(*n_sel, n_max)), a = aux_idx[j]:
 *     logp[j]    = x[r, y] - log sum_v exp(x[r, v]),          y = targets[r]
 *     entropy[j] = - sum_v p_v log p_v,  p = softmax(x[r, :])  (an entry of probability 0 adds 0)
 *     means[0]   = (1/n) sum_j entropy[j]
 *     means[1]   = (1/n) sum_j (old_logp[a] - logp[j])         (sample estimate of KL(pi_old || pi))
 *   logits, targets, rows, n_sel, n_max, aux_idx, aux_len: as in tppo_policy_loss_fwd_bwd
 *   old_logp   fp32 [aux_len] or NULL (means[1] is then 0 and aux_idx is not used)
 *   logp       [n_max] fp32 out;  entropy [n_max] fp32 out or NULL;  means [2] fp32 out
 *   stats      [4] int32 out: n, 0, 0, status bits
 *   workspace  tppo_workspace_bytes(TPPO_OP_POLICY_LOSS, R, 0, n_max, V) bytes
 * A row with a bad index or target, or whose logits hold a NaN or +inf (or nothing but -inf), gets
 * logp = entropy = 0, is left out of both sums (n still divides) and raises its status bit.
 * Fixed-order reductions: run-to-run identical.
 */
int tppo_policy_logprob_stats(const void *logits, int32_t logits_dtype,
                              int64_t R, int32_t V, int64_t ld,
                              const int32_t *targets,
                              const int32_t *rows, const int32_t *n_sel, int64_t n_max,
                              const int32_t *aux_idx, const float *old_logp, int64_t aux_len,
                              float *logp, float *entropy, float *means, int32_t *stats,
                              void *workspace, size_t workspace_bytes, void *stream);

/* kernel_hint values of tppo_policy_loss_fwd_bwd */
enum {
    TPPO_POLICY_AUTO = 0,
    TPPO_POLICY_TWO_PASS = 1,     /* any shape / dtype: row read twice from global memory      */
    TPPO_POLICY_CLUSTER_SMEM = 2  /* bf16, V % 8 == 0, 16-byte aligned rows: row held in the    */
                                  /* shared memory of a thread-block cluster, read once         */
};

/*
 * Clipped value regression on the value tokens, forward and backward (Eq. 4-5; the value update
 * of Algorithm 1).  For p = value_idx[j], j < n = min(*n_sel, n_max):
 *     Vc = clip(values[p], old_values[p] - xi_low, old_values[p] + xi_high)
 *     l  = 1/2 * max((values[p]-returns[p])^2, (Vc-returns[p])^2),   loss = (1/denom) sum l
 *     dvalues[p] = (values[p]-returns[p])/denom  if the unclipped term is the max (ties included),
 *                  else (Vc-returns[p])/denom if Vc == values[p], else 0
 *   values, old_values, returns [N] fp32; value_idx [n_max] int32 (distinct) or NULL for 0..n_max-1
 *   loss [1] fp32 out; dvalues [N] fp32 out (zero off the value tokens) or NULL
 *   stats [2] int32 out: n, status bits
 * A value token whose value, old value or return is a NaN or an infinity contributes nothing (loss
 * term and gradient 0) and raises TPPO_DEV_NONFINITE.
 */
int tppo_value_loss(const float *values, const float *old_values, const float *returns,
                    int64_t N, const int32_t *value_idx, const int32_t *n_sel, int64_t n_max,
                    float xi_low, float xi_high, float denom,
                    float *loss, float *dvalues, int32_t *stats,
                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * LM-head variant of the fused policy loss (Eq. 1 as in tppo_policy_loss_fwd_bwd, every one of the
 * M rows selected): the logits x = hidden * weight are a dense [M,K] x [K,V] bf16 contraction on
 * the tensor cores (fp32 accumulation) and are never written to memory.  Outputs are the loss, the
 * per-row log-probs and losses, and the gradients
 *     dhidden = dX * weight^T,   dweight = hidden^T * dX,   dX = (adv*rho*active/denom)(softmax - onehot).
 * The vocabulary is swept twice (statistics, then gradients with the logits recomputed); dX exists
 * only as a bf16 buffer for one chunk of vocabulary columns at a time inside the workspace.
 *
 *   hidden   [M, K] bf16 row-major     weight  [K, V] bf16 row-major     (16-byte aligned)
 *   targets  [M] int32                 aux_idx [M] int32 index into old_logp / adv, or NULL (= row)
 *   old_logp, adv   fp32, length aux_len
 *   logp, token_loss [M] fp32 out or NULL;  loss [1] fp32 out;  stats [4] int32 out as in
 *   tppo_policy_loss_fwd_bwd (n = M)
 *   dhidden  [M, K] bf16 out or NULL;  dweight [K, V] bf16 out or NULL (both NULL: forward only)
 *   chunk_tiles  0 = choose automatically; otherwise the number of 256-column vocabulary tiles per
 *                chunk (low 16 bits), clamped to the automatic choice (which sizes the workspace).
 *                Adding 65536 selects the CTA-pair (cta_group::2) GEMM kernels instead of the single-CTA ones.  For
 *                tuning and testing; changes the result only by the rounding order of dhidden's sum.
 *   workspace    tppo_workspace_bytes(TPPO_OP_LMHEAD, M, K, 0, V) bytes
 * K and V must be multiples of 8 (TPPO_ERR_UNSUPPORTED otherwise).  A row with a target outside
 * [0, V) or an aux index outside [0, aux_len) contributes nothing and raises the status bit.
 * Range: the logits are fp32 sums of K bf16 products and their exponentials are formed as
 * 2^(x*log2(e) - lse*log2(e)), so |x| must stay below 2.3e38 (FLT_MAX / log2 e).  A row whose logits
 * are not finite (a NaN or infinity in its hidden state or in the weight) contributes nothing to
 * the loss and to dweight, gets a zero dX, and raises TPPO_DEV_NONFINITE; dhidden is then only
 * finite where the weight itself is.
 * The first call on a device looks up the driver's tensor-map encoder (TPPO_ERR_CUDA if absent).
 */
int tppo_lmhead_logprob_fwd_bwd(const void *hidden, const void *weight,
                                int64_t M, int32_t K, int32_t V,
                                const int32_t *targets, const int32_t *aux_idx,
                                const float *old_logp, const float *adv, int64_t aux_len,
                                float eps_low, float eps_high, float denom,
                                float *logp, float *token_loss, float *loss, int32_t *stats,
                                void *dhidden, void *dweight, int32_t chunk_tiles,
                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same operation with the vocabulary split across devices (the LM-head weight held as column
 * shards, one per rank; the rows, targets and per-token scalars replicated).  Eq. 1 needs, per row,
 * the maximum logit, the sum of exponentials and the target's logit over the WHOLE vocabulary, so
 * the work is two calls with one exchange between them that the caller performs (the library
 * issues no collective):
 *
 *   1. tppo_lmhead_shard_stats on each rank: over the V_shard columns of its shard (vocabulary ids
 *      v_offset .. v_offset + V_shard - 1), per row r
 *          row_max[r] = max_v x[r,v],  row_sumexp[r] = sum_v exp(x[r,v] - row_max[r]),
 *          row_target_logit[r] = x[r, targets[r]] if the target lies in the shard, else 0.
 *      Rows with a target outside [0, V_total) get (0, 0, 0) and raise the status bit.
 *   2. the merge across ranks, m = max_r m_r;  S = sum_r s_r * exp(m_r - m);  xy = sum_r xy_r:
 *      the caller all-reduces (max) a copy of row_max into row_max_all, calls
 *      tppo_lmhead_shard_rescale, which multiplies row_sumexp[r] by exp(row_max[r] - row_max_all[r])
 *      in place (a skipped row keeps 0), and all-reduces (sum) row_sumexp and row_target_logit.
 *   3. tppo_lmhead_shard_fwd_bwd on each rank with the merged vectors: evaluates Eq. 1 (loss, logp,
 *      token_loss and stats come out identical on every rank), then forms the gradient for its
 *      columns only: dweight_shard [K, V_shard] is complete; dhidden_partial [M, K] holds this
 *      shard's term of dX * weight^T and the caller sums it over the ranks.
 *
 * All arrays live on the device.  row_max, row_sumexp, row_target_logit: [M] fp32.
 *   stats of tppo_lmhead_shard_stats: [4] int32, only the status bits (stats[3]) are written.
 *   workspace for either call: tppo_workspace_bytes(TPPO_OP_LMHEAD, M, K, 0, V_shard) bytes.
 * Every other argument, the limits on K and V_shard (multiples of 8) and the errors are those of
 * tppo_lmhead_logprob_fwd_bwd; 0 <= v_offset <= V_total - V_shard or TPPO_ERR_INVALID_ARG.  With one
 * shard (v_offset = 0, V_shard = V_total) the two calls compute exactly what the unsharded call does.
 */
int tppo_lmhead_shard_stats(const void *hidden, const void *weight_shard,
                            int64_t M, int32_t K, int32_t V_shard, int32_t v_offset, int32_t V_total,
                            const int32_t *targets,
                            float *row_max, float *row_sumexp, float *row_target_logit,
                            int32_t *stats, int32_t chunk_tiles,
                            void *workspace, size_t workspace_bytes, void *stream);
int tppo_lmhead_shard_rescale(const float *row_max, const float *row_max_all, float *row_sumexp,
                              int64_t M, void *stream);
int tppo_lmhead_shard_fwd_bwd(const void *hidden, const void *weight_shard,
                              int64_t M, int32_t K, int32_t V_shard, int32_t v_offset, int32_t V_total,
                              const int32_t *targets, const int32_t *aux_idx,
                              const float *old_logp, const float *adv, int64_t aux_len,
                              float eps_low, float eps_high, float denom,
                              const float *row_max, const float *row_sumexp,
                              const float *row_target_logit,
                              float *logp, float *token_loss, float *loss, int32_t *stats,
                              void *dhidden_partial, void *dweight_shard, int32_t chunk_tiles,
                              void *workspace, size_t workspace_bytes, void *stream);

/*
 * Successive batching between two training steps (Section 3.2 and its batching figure; the step of
 * Algorithm 1 that keeps the unfinished samples of the last step and puts new prompts in the place
 * of the finished ones).  The batch keeps its B slots, visited in ascending order:
 *   - truncated[i] != 0 (no end condition reached): the sequence stays in slot i; the tokens of this
 *     window join those of earlier windows: next_prompt_len = prompt_len, next_prev_len = prev_len +
 *     new_len, slot_source = -1.
 *   - otherwise the slot is freed and listed in free_slots; the k-th freed slot takes queued prompt
 *     k while the queue lasts (k < M): next_prompt_len = its length, next_prev_len = 0, slot_source =
 *     k; later freed slots stay empty (lengths 0, slot_source = -2).
 * The context of the next step (everything known before generation) is packed slot by slot into
 * next_tokens with offsets next_seq_begin: a kept slot's prompt and all its generated tokens copied
 * from `tokens`, a refilled slot's prompt copied from `queue_tokens`.
 *
 *   seq_begin [B+1], prompt_len / prev_len / new_len [B] int32, truncated [B] u8: the finished step
 *   tokens       [N] int32 token ids in that packed layout
 *   queue_begin  [M+1] int32 offsets of the queued prompts inside queue_tokens [queue_total]
 *   next_prompt_len, next_prev_len [B]; next_seq_begin [B+1]; next_tokens [capacity] int32 out
 *   free_slots   [B] int32 out, ascending, first counts[0] entries valid
 *   slot_source  [B] int32 out
 *   counts       [4] int32 out: freed slots, refilled slots, context tokens of the next step, device
 *                status bits (TPPO_DEV_OVERFLOW when the context exceeds `capacity` or 2^31-1: the
 *                excess is not written; TPPO_DEV_BAD_INDEX for negative lengths and for a slot whose
 *                source range does not lie inside `tokens` / `queue_tokens`: its context is then
 *                written as zeros, nothing outside the arrays is read)
 * No workspace and no clear beforehand: the slot walk writes all four counts itself, and the copy
 * kernel is launched as its programmatic dependent (scheduled while the walk still runs, reading its
 * results only after it has finished).  Bit-exact and run-to-run identical.
 */
int tppo_advance_batch(const int32_t *seq_begin, const int32_t *prompt_len,
                       const int32_t *prev_len, const int32_t *new_len,
                       const uint8_t *truncated, const int32_t *tokens, int64_t N,
                       const int32_t *queue_begin, const int32_t *queue_tokens,
                       int64_t queue_total, int32_t B, int32_t M,
                       int32_t *next_prompt_len, int32_t *next_prev_len,
                       int32_t *next_seq_begin, int32_t *next_tokens, int64_t capacity,
                       int32_t *free_slots, int32_t *slot_source, int32_t *counts,
                       void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TPPO_H */

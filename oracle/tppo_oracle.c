/*
 * T-PPO token-selective update path: float64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of what the
 * CUDA library must compute.  Only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg may call it; the product path never does.  It shares no code, header,
 * table or helper with the CUDA sources.
 *
 * Everything is computed in double.  bf16 / fp32 inputs are widened exactly.  Loops are serial
 * inside a segment or a vocabulary row, in index order; OpenMP only spreads independent
 * segments / rows over cores, which changes no summation order.
 *
 * Parity pins (see tests/test_oracle_*.py): brute-force sums of Eq. 2/6, the gamma=lambda=1
 * telescoped closed form, a hand-derived 3-token example, scipy's IIR filter, exhaustive mask
 * enumeration, scipy logsumexp, finite differences and float64 autograd of Eq. 1 / Eq. 4-5,
 * torch's float64 softmax entropy.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* bf16 is the upper half of an IEEE binary32: widening is a 16-bit shift. */
static double widen_bf16(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* dtype: 0 = bf16 (uint16 storage), 1 = fp32, 2 = double (logits the oracle formed itself from
 * hidden states and the LM-head weight) */
static double logit_at(const void *logits, int dtype, int64_t ld, int64_t row, int64_t v)
{
    if (dtype == 0)
        return widen_bf16(((const uint16_t *)logits)[row * ld + v]);
    if (dtype == 2)
        return ((const double *)logits)[row * ld + v];
    return (double)((const float *)logits)[row * ld + v];
}

/* ------------------------------------------------------------------------------------------
 * EGAE advantages (Eq. 6 with the TD residual of Eq. 3) and Monte-Carlo returns (R_t in the
 * text after Eq. 5), one response segment [seg_begin[i], seg_end[i]) at a time.
 *
 * Eq. 6 is  A_t = delta_t + (gamma*lambda) delta_{t+1} + ... + (gamma*lambda)^{l-t-1} delta_{l-1},
 * i.e. the backward recurrence A_t = delta_t + gamma*lambda*A_{t+1} with A_l = 0, and
 * delta_t = r_t + gamma*V(s_{t+1}) - V(s_t)  (Eq. 3).
 * The state after the last token has no value: it is 0 for a finished response (terminal
 * state) and, for a truncated one, Section 3.1 sets V(s_l) = V(s_{l-1}); an explicit bootstrap
 * value may override that.
 * R_t = sum_i gamma^i r_{t+i}, i.e. R_t = r_t + gamma*R_{t+1}, R_l = 0.
 * Positions outside every segment get 0.
 * ---------------------------------------------------------------------------------------- */
void oracle_egae(const float *rewards, const float *values,
                 const int32_t *seg_begin, const int32_t *seg_end,
                 const uint8_t *truncated, const float *bootstrap /* may be NULL */,
                 int32_t B, int64_t N, double gamma, double lambda,
                 double *advantages, double *returns /* may be NULL */)
{
    for (int64_t p = 0; p < N; ++p) advantages[p] = 0.0;
    if (returns)
        for (int64_t p = 0; p < N; ++p) returns[p] = 0.0;

#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t i = 0; i < B; ++i) {
        const int64_t b = seg_begin[i], e = seg_end[i];
        if (e <= b) continue;
        double v_next;
        if (truncated[i])
            v_next = bootstrap ? (double)bootstrap[i] : (double)values[e - 1];
        else
            v_next = 0.0;
        double A = 0.0, G = 0.0;
        for (int64_t t = e - 1; t >= b; --t) {
            const double r = (double)rewards[t], v = (double)values[t];
            const double delta = r + gamma * v_next - v;
            A = delta + gamma * lambda * A;
            advantages[t] = A;
            v_next = v;
            if (returns) {
                G = r + gamma * G;
                returns[t] = G;
            }
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Token filtering (Section 3.2).  Sequence i occupies packed positions
 * [seq_begin[i], seq_begin[i+1]) laid out  prompt | earlier-window response | this-window
 * response.  Policy tokens: the response tokens generated in the current step, finished or
 * not, minus the latest tokens of an unfinished sequence (Section 3.2 allows leaving some of
 * them out; how many is a parameter: tail_drop for every unfinished sequence, or
 * tail_drop_seq[i] for sequence i when that array is given; a negative count means none).
 * Value tokens: every generated token of a finished sequence.  Prompt tokens enter neither
 * set.  Optional byte masks AND with the predicates.  Lists are in ascending position order.
 * ---------------------------------------------------------------------------------------- */
void oracle_select_tokens(const int32_t *seq_begin, const int32_t *prompt_len,
                          const int32_t *prev_len, const int32_t *new_len,
                          const uint8_t *truncated, int32_t tail_drop,
                          const int32_t *tail_drop_seq /* [B] or NULL */,
                          const uint8_t *extra_policy_mask, const uint8_t *extra_value_mask,
                          int32_t B, int64_t N,
                          int32_t *policy_idx, int32_t *value_idx, int64_t *counts)
{
    int64_t n_pol = 0, n_val = 0;
    int32_t i = 0;
    for (int64_t p = 0; p < N; ++p) {
        while (i < B && p >= seq_begin[i + 1]) ++i;
        if (i >= B) break;
        if (p < seq_begin[i]) continue;
        const int64_t off = p - seq_begin[i];
        const int64_t resp0 = prompt_len[i];
        const int64_t new0 = (int64_t)prompt_len[i] + prev_len[i];
        const int64_t end = new0 + new_len[i];
        int64_t drop = tail_drop_seq ? tail_drop_seq[i] : tail_drop;
        if (drop < 0) drop = 0;
        int64_t pol_end = end - (truncated[i] ? drop : 0);
        int is_pol = off >= new0 && off < pol_end;
        int is_val = !truncated[i] && off >= resp0 && off < end;
        if (extra_policy_mask) is_pol = is_pol && extra_policy_mask[p] != 0;
        if (extra_value_mask) is_val = is_val && extra_value_mask[p] != 0;
        if (is_pol) policy_idx[n_pol++] = (int32_t)p;
        if (is_val) value_idx[n_val++] = (int32_t)p;
    }
    counts[0] = n_pol;
    counts[1] = n_val;
}

/* ------------------------------------------------------------------------------------------
 * log pi(a|s) of Eq. 1 from a row of logits: x_y - log sum_v exp(x_v), with the usual shift
 * by the row maximum m, summed in index order:
 *     log pi(y) = (x_y - m) - log S,    softmax_v = exp((x_v - m) - log S),    S = sum_v exp(x_v - m).
 * The maximum and log S are kept apart (never added), so that the result is also exact for
 * logits of the largest representable magnitude, where m + log S would round log S away.
 * ---------------------------------------------------------------------------------------- */
static void row_max_and_logsum(const void *logits, int dtype, int64_t ld, int64_t row, int32_t V,
                               double *row_max, double *log_sum)
{
    double m = -INFINITY;
    for (int32_t v = 0; v < V; ++v) {
        const double x = logit_at(logits, dtype, ld, row, v);
        if (x > m) m = x;
    }
    double S = 0.0;
    for (int32_t v = 0; v < V; ++v) S += exp(logit_at(logits, dtype, ld, row, v) - m);
    *row_max = m;
    *log_sum = log(S);
}

void oracle_logprob(const void *logits, int dtype, int32_t V, int64_t ld,
                    const int32_t *targets, const int32_t *rows /* NULL: identity */,
                    int64_t n, double *logp)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t j = 0; j < n; ++j) {
        const int64_t row = rows ? rows[j] : j;
        double m, log_sum;
        row_max_and_logsum(logits, dtype, ld, row, V, &m, &log_sum);
        logp[j] = (logit_at(logits, dtype, ld, row, targets[row]) - m) - log_sum;
    }
}

/* ------------------------------------------------------------------------------------------
 * Statistics of the forward-only sweep that produces the old-policy log-probs (the step of
 * Algorithm 1 that snapshots pi_theta_old): per selected row the log-prob of its target and
 * the entropy of its softmax,
 *     H = - sum_v p_v log p_v,   p_v = softmax_v,   log p_v = (x_v - m) - log S,
 * a vocabulary entry of probability 0 (x_v = -inf) contributing 0; and over the selected rows
 * the means of H and of old_logp - logp (the usual sample estimate of KL(pi_old || pi_theta)).
 * aux_idx[j] (NULL: the logits row) indexes old_logp, which may be NULL (mean_kl = 0).
 * ---------------------------------------------------------------------------------------- */
void oracle_logprob_stats(const void *logits, int dtype, int32_t V, int64_t ld,
                          const int32_t *targets, const int32_t *rows, const int32_t *aux_idx,
                          int64_t n, const float *old_logp,
                          double *logp, double *entropy, double *means /* [2] */)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t j = 0; j < n; ++j) {
        const int64_t row = rows ? rows[j] : j;
        double m, log_sum;
        row_max_and_logsum(logits, dtype, ld, row, V, &m, &log_sum);
        logp[j] = (logit_at(logits, dtype, ld, row, targets[row]) - m) - log_sum;
        double H = 0.0;
        for (int32_t v = 0; v < V; ++v) {
            const double lp = (logit_at(logits, dtype, ld, row, v) - m) - log_sum;
            const double p = exp(lp);
            if (p > 0.0) H -= p * lp;
        }
        entropy[j] = H;
    }
    double sum_h = 0.0, sum_kl = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        sum_h += entropy[j];
        if (old_logp) {
            const int64_t row = rows ? rows[j] : j;
            const int64_t a = aux_idx ? aux_idx[j] : row;
            sum_kl += (double)old_logp[a] - logp[j];
        }
    }
    means[0] = n > 0 ? sum_h / (double)n : 0.0;
    means[1] = n > 0 ? sum_kl / (double)n : 0.0;
}

/* ------------------------------------------------------------------------------------------
 * Clipped surrogate of Eq. 1 as a loss to minimise, token-level mean (Section 4.1.1), and
 * its gradient with respect to the logits.
 *   rho = exp(logp - logp_old)
 *   l_j = -min(rho*A, clip(rho, 1-eps_low, 1+eps_high)*A),   L = (1/denom) sum_j l_j
 *   dL/dlogp_j = -(A*rho/denom) when the unclipped term is the active one, else 0
 *   dlogp/dx_v = 1[v=y] - softmax_v
 * The clipped branch is active only when it is strictly the smaller one.
 * aux_idx[j] (NULL: same as the logits row) indexes old_logp and adv.
 * denom <= 0 means "number of selected rows".
 * dlogits (may be NULL) is compact [n, V].
 * clip_counts[0/1]: rows whose gradient is cut by the lower / upper edge.
 * ---------------------------------------------------------------------------------------- */
void oracle_policy_loss(const void *logits, int dtype, int32_t V, int64_t ld,
                        const int32_t *targets, const int32_t *rows, const int32_t *aux_idx,
                        int64_t n, const float *old_logp, const float *adv,
                        double eps_low, double eps_high, double denom,
                        double *logp, double *token_loss, double *loss,
                        int64_t *clip_counts, double *dlogits)
{
    const double d = denom > 0.0 ? denom : (double)n;
    uint8_t *clipped = (uint8_t *)calloc((size_t)(n > 0 ? n : 1), 1);

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t j = 0; j < n; ++j) {
        const int64_t row = rows ? rows[j] : j;
        const int64_t a = aux_idx ? aux_idx[j] : row;
        const int32_t y = targets[row];
        double m, log_sum;
        row_max_and_logsum(logits, dtype, ld, row, V, &m, &log_sum);
        const double lp = (logit_at(logits, dtype, ld, row, y) - m) - log_sum;
        const double A = (double)adv[a];
        const double rho = exp(lp - (double)old_logp[a]);
        double rc = rho;
        if (rc < 1.0 - eps_low) rc = 1.0 - eps_low;
        if (rc > 1.0 + eps_high) rc = 1.0 + eps_high;
        const double s1 = rho * A, s2 = rc * A;
        int active = 1;
        if (s2 < s1) {
            active = 0;
            clipped[j] = rho < 1.0 - eps_low ? 1 : 2;
        }
        logp[j] = lp;
        token_loss[j] = -(s2 < s1 ? s2 : s1);
        if (dlogits) {
            const double g = active ? -(A * rho) / d : 0.0; /* dL/dlogp */
            double *out = dlogits + j * (int64_t)V;
            for (int32_t v = 0; v < V; ++v) {
                const double p = exp((logit_at(logits, dtype, ld, row, v) - m) - log_sum);
                out[v] = g * ((v == y ? 1.0 : 0.0) - p);
            }
        }
    }
    double sum = 0.0;
    int64_t lo = 0, hi = 0;
    for (int64_t j = 0; j < n; ++j) {
        sum += token_loss[j];
        lo += clipped[j] == 1;
        hi += clipped[j] == 2;
    }
    *loss = n > 0 ? sum / d : 0.0;
    if (clip_counts) {
        clip_counts[0] = lo;
        clip_counts[1] = hi;
    }
    free(clipped);
}

/* ------------------------------------------------------------------------------------------
 * Clipped value regression, Eq. 4-5, mean over the value tokens, and its gradient.
 *   Vc = clip(V, Vold - xi_low, Vold + xi_high)
 *   l  = 1/2 max((V-R)^2, (Vc-R)^2);  the unclipped branch wins ties.
 *   dl/dV = (V-R) on the unclipped branch; on the clipped branch (Vc-R) if Vc == V else 0.
 * dvalues (may be NULL) is [N], zero off the value tokens.
 * ---------------------------------------------------------------------------------------- */
void oracle_value_loss(const float *values, const float *old_values, const float *returns,
                       const int32_t *value_idx, int64_t n, int64_t N,
                       double xi_low, double xi_high, double denom,
                       double *loss, double *dvalues)
{
    const double d = denom > 0.0 ? denom : (double)n;
    if (dvalues)
        for (int64_t p = 0; p < N; ++p) dvalues[p] = 0.0;
    double sum = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        const int64_t p = value_idx[j];
        const double v = (double)values[p], vo = (double)old_values[p], R = (double)returns[p];
        double vc = v;
        if (vc < vo - xi_low) vc = vo - xi_low;
        if (vc > vo + xi_high) vc = vo + xi_high;
        const double e1 = (v - R) * (v - R), e2 = (vc - R) * (vc - R);
        double g;
        if (e1 >= e2) {
            sum += 0.5 * e1;
            g = v - R;
        } else {
            sum += 0.5 * e2;
            g = (vc == v) ? (vc - R) : 0.0;
        }
        if (dvalues) dvalues[p] = g / d;
    }
    *loss = n > 0 ? sum / d : 0.0;
}

/* ------------------------------------------------------------------------------------------
 * LM-head variant: the logits are x = H * W (H [M,K], W [K,V], both bf16, row-major) and are
 * never stored by the CUDA path.  The oracle forms chosen rows of x in double by the plain
 * inner-product definition so that the routines above can be applied to them, and forms
 * chosen entries of dH = dX * W^T and dW = H^T * dX from a double dX.
 * ---------------------------------------------------------------------------------------- */
void oracle_lmhead_logits_rows(const uint16_t *hidden, const uint16_t *weight,
                               int32_t K, int32_t V, const int32_t *rows, int64_t n_rows,
                               double *x /* [n_rows, V] */)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t j = 0; j < n_rows; ++j) {
        const int64_t m = rows[j];
        double *out = x + j * (int64_t)V;
        for (int32_t v = 0; v < V; ++v) out[v] = 0.0;
        for (int32_t k = 0; k < K; ++k) {
            const double h = widen_bf16(hidden[m * (int64_t)K + k]);
            const uint16_t *w = weight + (int64_t)k * V;
            for (int32_t v = 0; v < V; ++v) out[v] += h * widen_bf16(w[v]);
        }
    }
}

/* dH[j, :] = sum_v dX[j, v] * W[:, v]   for the n_rows rows whose dX is given */
void oracle_lmhead_dhidden_rows(const double *dx /* [n_rows, V] */, const uint16_t *weight,
                                int32_t K, int32_t V, int64_t n_rows, double *dh /* [n_rows,K] */)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t j = 0; j < n_rows; ++j) {
        for (int32_t k = 0; k < K; ++k) {
            const uint16_t *w = weight + (int64_t)k * V;
            const double *g = dx + j * (int64_t)V;
            double s = 0.0;
            for (int32_t v = 0; v < V; ++v) s += g[v] * widen_bf16(w[v]);
            dh[j * (int64_t)K + k] = s;
        }
    }
}

/* dW[:, cols[c]] = sum_m H[m, :] * dX[m, cols[c]]  with dX given for ALL M rows at the chosen
 * columns only: dx_cols is [M, n_cols]. */
void oracle_lmhead_dweight_cols(const uint16_t *hidden, const double *dx_cols,
                                int64_t M, int32_t K, int64_t n_cols,
                                double *dw /* [K, n_cols] */)
{
#pragma omp parallel for schedule(static)
    for (int32_t k = 0; k < K; ++k) {
        for (int64_t c = 0; c < n_cols; ++c) {
            double s = 0.0;
            for (int64_t m = 0; m < M; ++m)
                s += widen_bf16(hidden[m * (int64_t)K + k]) * dx_cols[m * n_cols + c];
            dw[(int64_t)k * n_cols + c] = s;
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Successive batching between two training steps (Section 3.2, the batching figure; the batch
 * collection step of Algorithm 1): the batch keeps its B slots.  A slot whose sequence reached an end condition is
 * freed and takes the next queued prompt; a slot whose sequence was cut at the window keeps it,
 * and the tokens generated in this step join those of earlier windows.
 *
 * Slots are visited in ascending order; the k-th freed slot takes queued prompt k while the
 * queue lasts (M prompts), later freed slots stay empty.  The context of the next step (what is
 * known before generation) is packed slot by slot:
 *   kept slot      prompt | all generated tokens so far     (copied from `tokens`)
 *   refilled slot  the queued prompt                        (copied from `queue_tokens`)
 *   empty slot     nothing
 * slot_source[i] = -1 kept, k >= 0 refilled with prompt k, -2 empty.
 * counts: [0] freed slots, [1] refilled slots, [2] context tokens of the next step.
 * next_tokens has room for `capacity` tokens; tokens beyond it are not written.
 * ---------------------------------------------------------------------------------------- */
void oracle_advance_batch(const int32_t *seq_begin, const int32_t *prompt_len,
                          const int32_t *prev_len, const int32_t *new_len,
                          const uint8_t *truncated, const int32_t *tokens,
                          const int32_t *queue_begin, const int32_t *queue_tokens,
                          int32_t B, int32_t M,
                          int32_t *next_prompt_len, int32_t *next_prev_len,
                          int32_t *next_seq_begin, int32_t *next_tokens, int64_t capacity,
                          int32_t *free_slots, int32_t *slot_source, int64_t *counts)
{
    int64_t n_free = 0, n_refilled = 0, pos = 0;
    for (int32_t i = 0; i < B; ++i) {
        next_seq_begin[i] = (int32_t)pos;
        if (truncated[i]) {                       /* unfinished: stays, this window joins the past */
            next_prompt_len[i] = prompt_len[i];
            next_prev_len[i] = prev_len[i] + new_len[i];
            slot_source[i] = -1;
            const int64_t len = (int64_t)prompt_len[i] + prev_len[i] + new_len[i];
            for (int64_t o = 0; o < len; ++o, ++pos)
                if (pos < capacity) next_tokens[pos] = tokens[seq_begin[i] + o];
        } else {                                  /* finished: the slot is freed */
            free_slots[n_free] = i;
            next_prev_len[i] = 0;
            if (n_free < M) {
                const int32_t k = (int32_t)n_free;
                const int32_t len = queue_begin[k + 1] - queue_begin[k];
                next_prompt_len[i] = len;
                slot_source[i] = k;
                for (int32_t o = 0; o < len; ++o, ++pos)
                    if (pos < capacity) next_tokens[pos] = queue_tokens[queue_begin[k] + o];
                ++n_refilled;
            } else {
                next_prompt_len[i] = 0;
                slot_source[i] = -2;
            }
            ++n_free;
        }
    }
    next_seq_begin[B] = (int32_t)pos;
    counts[0] = n_free;
    counts[1] = n_refilled;
    counts[2] = pos;
}

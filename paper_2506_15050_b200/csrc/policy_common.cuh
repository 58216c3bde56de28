// Pieces shared by the policy-loss kernels: argument block, row bookkeeping and the per-row scalar
// part of the clipped surrogate (Eq. 1 of the paper).
#pragma once

#include "common.cuh"

namespace tppo {

struct PolicyArgs {
    const void* logits;
    int64_t R;
    int32_t V;
    int64_t ld;
    const int32_t* targets;
    const int32_t* rows;
    const int32_t* n_sel;
    int64_t n_max;
    const int32_t* aux_idx;
    const float* old_logp;
    const float* adv;
    int64_t aux_len;
    float eps_low, eps_high, denom;
    float* logp;
    float* token_loss;
    float* loss;
    int32_t* stats;      // [4]: n, clipped low, clipped high, status bits
    void* dlogits;
    int32_t mode;        // TPPO_DLOGITS_*
    float* row_loss;     // workspace [n_max]: per-row loss term, 0 for skipped rows
    uint8_t* row_clip;   // workspace [n_max]: 0 none, 1 lower edge, 2 upper edge
    uint8_t* row_flag;   // workspace [R]: 1 = row is selected (FULL mode with a row list)
    struct RowRec* rec;  // workspace [n_max]: per-entry scalars gathered ahead of the vocabulary sweep
    // Two kernels may share one call's rows: part 0 = this launch takes all n rows; part 1 = the
    // first n - n_side of them; part 2 = the last n_side, with n_side = n * side_share_256 / 256.
    int32_t part;
    int32_t side_share_256;
};

// Everything the vocabulary sweep needs to know about the j-th selected entry, gathered once by a
// small kernel so that the sweep reads one 16-byte record per row instead of chasing indices.
struct __align__(16) RowRec {
    int32_t row;        // logits row, or -1 when the row index is out of range
    int32_t y;          // target id, or -1 when the entry is to be skipped (bad row, aux or target)
    float adv;          // adv[aux]
    float old_logp;     // old_logp[aux]
};
__device__ __forceinline__ RowRec load_rec(const RowRec* p) {
    const int4 v = __ldg(reinterpret_cast<const int4*>(p));
    RowRec r;
    r.row = v.x; r.y = v.y; r.adv = __int_as_float(v.z); r.old_logp = __int_as_float(v.w);
    return r;
}

__device__ __forceinline__ int64_t policy_n(const PolicyArgs& a) {
    int64_t n = a.n_max;
    if (a.n_sel) { const int64_t c = *a.n_sel; n = c < 0 ? 0 : (c < n ? c : n); }
    return n;
}
// Selected entries [lo, hi) that this launch works on.
__device__ __forceinline__ void policy_part(const PolicyArgs& a, int64_t n, int64_t& lo, int64_t& hi) {
    const int64_t n_side = a.part == 0 ? 0 : (n * a.side_share_256) >> 8;
    lo = a.part == 2 ? n - n_side : 0;
    hi = a.part == 1 ? n - n_side : n;
}
__device__ __forceinline__ float policy_inv_denom(const PolicyArgs& a, int64_t n) {
    return a.denom > 0.f ? 1.f / a.denom : 1.f / float(n > 0 ? n : 1);
}

// Row bookkeeping for the j-th selected entry.  Returns false (and raises the status bit) when
// the row, its auxiliary index or its target id is out of range; such an entry contributes
// nothing to the loss and gets a zero gradient.
struct RowMeta {
    int64_t row;
    int64_t aux;
    int32_t y;
    bool row_ok;   // the logits row exists (it can be read and, in FULL mode, written)
    bool ok;       // row, aux and target all valid
};
__device__ __forceinline__ RowMeta policy_row_meta(const PolicyArgs& a, int64_t j) {
    RowMeta m;
    m.row = a.rows ? int64_t(__ldg(a.rows + j)) : j;
    m.row_ok = m.row >= 0 && m.row < a.R;
    m.aux = 0;
    m.y = 0;
    m.ok = false;
    if (m.row_ok) {
        m.aux = a.aux_idx ? int64_t(__ldg(a.aux_idx + j)) : m.row;
        m.y = __ldg(a.targets + m.row);
        m.ok = m.aux >= 0 && m.aux < a.aux_len && m.y >= 0 && m.y < a.V;
    }
    return m;
}
__device__ __forceinline__ int policy_bad_bits(const RowMeta& m, const PolicyArgs& a) {
    if (!m.row_ok) return TPPO_DEV_BAD_INDEX;
    int bits = 0;
    if (m.aux < 0 || m.aux >= a.aux_len) bits |= TPPO_DEV_BAD_INDEX;
    if (m.y < 0 || m.y >= a.V) bits |= TPPO_DEV_BAD_TARGET;
    return bits;
}

// Scalar part of Eq. 1 for one token, written as a loss to minimise:
//   rho = exp(logp - logp_old);  l = -min(rho*A, clip(rho, 1-eps_low, 1+eps_high)*A)
// and the factor c with  dl/dx_v * (1/denom) = c * (softmax_v - 1[v == y]);  c = 0 when the
// clipped term is strictly the smaller one.
struct RowLoss {
    float logp, loss, coef;
    int clip;
};
// x_y_rel = x_y - max_v x_v and log_sum = log sum_v exp(x_v - max) are passed separately so that
// the log-prob keeps full precision when the logits are large.
__device__ __forceinline__ RowLoss ppo_row(float x_y_rel, float log_sum, float old_lp, float A,
                                           float eps_low, float eps_high, float inv_denom) {
    RowLoss r;
    r.logp = x_y_rel - log_sum;
    const float rho = expf(r.logp - old_lp);
    const float lo = 1.f - eps_low, hi = 1.f + eps_high;
    const float rc = fminf(fmaxf(rho, lo), hi);
    const float s1 = rho * A, s2 = rc * A;
    const bool clipped = s2 < s1;
    r.loss = -(clipped ? s2 : s1);
    r.coef = clipped ? 0.f : A * rho * inv_denom;
    r.clip = clipped ? (rho < lo ? 1 : 2) : 0;
    return r;
}

}  // namespace tppo

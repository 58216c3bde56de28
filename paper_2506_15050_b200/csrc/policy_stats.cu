// Forward-only statistics of the sweep that produces the old-policy log-probs (the step of
// Algorithm 1 that snapshots pi_theta_old): per selected row the log-prob of its target and the
// entropy of its softmax, and over the rows the means of the entropy and of old_logp - logp.
// One thread block per row, ONE read of the row: the running maximum m, S = sum exp(x - m) and
// T = sum exp(x - m) (x - m) are updated together, so that
//     log p_y = (x_y - m) - log S,      H = -sum p log p = log S - T / S.
#include "policy_common.cuh"

namespace tppo {

int launch_policy_prepare(const PolicyArgs& a, cudaStream_t s);
size_t policy_workspace_bytes(int64_t R, int64_t n_max);

namespace {

constexpr int kStatThreads = 512;
constexpr int kStatDeep = 4;          // 16-byte loads in flight per thread

struct RowStat {
    float m, s, t;
};
// The statistics when the reference point moves from m to m_new >= m: S scales by c = exp(m - m_new),
// T becomes c (T + (m - m_new) S).  A vanishing c drops the old terms altogether (their probability
// is 0, and 0 * log 0 counts as 0), which also keeps 0 * inf out of the arithmetic.
__device__ __forceinline__ void stat_rebase(RowStat& a, float m_new) {
    const float d = a.m - m_new;
    const float c = ex2(d * kLog2e);
    a.t = c > 0.f ? c * fmaf(d, a.s, a.t) : 0.f;
    a.s = a.s * c;
    a.m = m_new;
}
__device__ __forceinline__ void stat_add(RowStat& a, float x) {      // x <= a.m
    const float d = x - a.m;
    const float e = ex2(d * kLog2e);
    a.s += e;
    a.t += e > 0.f ? e * d : 0.f;
}
__device__ __forceinline__ RowStat stat_merge(RowStat a, RowStat b) {
    const float m = fmaxf(a.m, b.m);
    stat_rebase(a, m);
    stat_rebase(b, m);
    return RowStat{m, a.s + b.s, a.t + b.t};
}
template <int N>
__device__ __forceinline__ void stat_update(RowStat& a, const float (&x)[N]) {
    float mx = x[0];
#pragma unroll
    for (int k = 1; k < N; ++k) mx = fmaxf(mx, x[k]);
    if (mx > a.m) stat_rebase(a, mx);
#pragma unroll
    for (int k = 0; k < N; ++k) stat_add(a, x[k]);
}

__device__ __forceinline__ float widen(uint16_t h) { return __uint_as_float(uint32_t(h) << 16); }
__device__ __forceinline__ float widen(float f) { return f; }
__device__ __forceinline__ void widen8(uint4 w, float (&x)[8]) {
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
}

struct StatArgs {
    PolicyArgs p;          // logits, rows, records, logp; row_loss receives the entropy of each row
    float* entropy;        // [n_max] or null
    float* means;          // [2]
};

// T = uint16_t (bf16 bits) or float.  VEC: rows start on 16-byte boundaries.
template <typename T, bool VEC>
__global__ void __launch_bounds__(kStatThreads) policy_stats_kernel(const StatArgs sa) {
    const PolicyArgs& a = sa.p;
    __shared__ RowStat s_part[kStatThreads / 32];
    const int64_t n = policy_n(a);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T* logits = static_cast<const T*>(a.logits);
    constexpr int kPer = 16 / sizeof(T);        // elements per 16-byte unit

    for (int64_t j = blockIdx.x; j < n; j += gridDim.x) {
        const RowRec rec = load_rec(a.rec + j);
        float logp = 0.f, H = 0.f;
        uint8_t skipped = 1;
        if (rec.y >= 0) {       // (uniform over the block)
            const T* x_row = logits + int64_t(rec.row) * a.ld;
            RowStat st{-kFltMax, 0.f, 0.f};
            int v0 = 0;
            if (VEC) {
                const int nu = a.V / kPer;
                int u = tid;
                for (; u + (kStatDeep - 1) * kStatThreads < nu; u += kStatDeep * kStatThreads) {
                    uint4 raw[kStatDeep];
#pragma unroll
                    for (int d = 0; d < kStatDeep; ++d)
                        raw[d] = *reinterpret_cast<const uint4*>(x_row + int64_t(u + d * kStatThreads) * kPer);
#pragma unroll
                    for (int d = 0; d < kStatDeep; ++d) {
                        if (sizeof(T) == 2) {
                            float x[8];
                            widen8(raw[d], x);
                            stat_update<8>(st, x);
                        } else {
                            const float x[4] = {__uint_as_float(raw[d].x), __uint_as_float(raw[d].y),
                                                __uint_as_float(raw[d].z), __uint_as_float(raw[d].w)};
                            stat_update<4>(st, x);
                        }
                    }
                }
                for (; u < nu; u += kStatThreads) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(x_row + int64_t(u) * kPer);
                    if (sizeof(T) == 2) {
                        float x[8];
                        widen8(raw, x);
                        stat_update<8>(st, x);
                    } else {
                        const float x[4] = {__uint_as_float(raw.x), __uint_as_float(raw.y),
                                            __uint_as_float(raw.z), __uint_as_float(raw.w)};
                        stat_update<4>(st, x);
                    }
                }
                v0 = nu * kPer;
            }
            for (int v = v0 + tid; v < a.V; v += kStatThreads) {
                const float x[1] = {widen(x_row[v])};
                stat_update<1>(st, x);
            }
            // warp, then block (fixed order)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                RowStat other{__shfl_xor_sync(0xffffffffu, st.m, o), __shfl_xor_sync(0xffffffffu, st.s, o),
                              __shfl_xor_sync(0xffffffffu, st.t, o)};
                // both lanes of a pair must end with the same bits: merge in a fixed operand order
                st = (lane & o) ? stat_merge(other, st) : stat_merge(st, other);
            }
            if (lane == 0) s_part[warp] = st;
            __syncthreads();
            if (tid == 0) {
                RowStat tot = s_part[0];
                for (int w = 1; w < kStatThreads / 32; ++w) tot = stat_merge(tot, s_part[w]);
                // not a positive finite sum: the row held a NaN or +inf logit, or nothing but -inf
                const bool finite = tot.s > 0.f && tot.s <= kFltMax && tot.m <= kFltMax && fabsf(tot.t) <= kFltMax;
                if (finite) {
                    const float log_s = logf(tot.s);
                    logp = (widen(x_row[rec.y]) - tot.m) - log_s;
                    H = log_s - tot.t / tot.s;
                    skipped = 0;
                } else {
                    atomicOr(a.stats + 3, TPPO_DEV_NONFINITE);
                }
            }
        }
        if (tid == 0) {
            a.logp[j] = logp;
            if (sa.entropy) sa.entropy[j] = H;
            a.row_loss[j] = H;
            a.row_clip[j] = skipped;     // 1: the row takes no part in the means' sums
        }
        __syncthreads();                 // s_part is reused by the next row
    }
}

// Fixed-order sums over the rows: mean entropy and mean (old_logp - logp).  Both divide by n.
__global__ void __launch_bounds__(1024) policy_stats_finish_kernel(const StatArgs sa) {
    const PolicyArgs& a = sa.p;
    __shared__ double s_h[32], s_k[32];
    const int64_t n = policy_n(a);
    double h = 0.0, k = 0.0;
    for (int64_t j = threadIdx.x; j < n; j += blockDim.x) {
        if (a.row_clip[j]) continue;
        h += double(a.row_loss[j]);
        if (a.old_logp) k += double(load_rec(a.rec + j).old_logp) - double(a.logp[j]);
    }
    h = warp_sum(h);
    k = warp_sum(k);
    if ((threadIdx.x & 31) == 0) { s_h[threadIdx.x >> 5] = h; s_k[threadIdx.x >> 5] = k; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double th = 0.0, tk = 0.0;
        for (int w = 0; w < int(blockDim.x >> 5); ++w) { th += s_h[w]; tk += s_k[w]; }
        sa.means[0] = n > 0 ? float(th / double(n)) : 0.f;
        sa.means[1] = n > 0 ? float(tk / double(n)) : 0.f;
        a.stats[0] = int32_t(n);
    }
}

}  // namespace
}  // namespace tppo

using namespace tppo;

TPPO_API int tppo_policy_logprob_stats(const void* logits, int32_t logits_dtype, int64_t R, int32_t V,
                                       int64_t ld, const int32_t* targets, const int32_t* rows,
                                       const int32_t* n_sel, int64_t n_max, const int32_t* aux_idx,
                                       const float* old_logp, int64_t aux_len, float* logp,
                                       float* entropy, float* means, int32_t* stats, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    if (logits_dtype != TPPO_BF16 && logits_dtype != TPPO_F32) return TPPO_ERR_INVALID_ARG;
    if (R < 0 || V <= 0 || ld < V || n_max < 0 || aux_len < 0 || R >= (int64_t(1) << 31))
        return TPPO_ERR_INVALID_ARG;
    if (!means || !stats) return TPPO_ERR_INVALID_ARG;
    if (!rows && n_max > R) return TPPO_ERR_INVALID_ARG;
    if (n_max > 0 && (!logits || !targets || !logp)) return TPPO_ERR_INVALID_ARG;
    const size_t esz = logits_dtype == TPPO_BF16 ? 2 : 4;
    if (!aligned(logits, esz)) return TPPO_ERR_INVALID_ARG;
    const size_t need = policy_workspace_bytes(R, n_max);
    if (!workspace || workspace_bytes < need || !aligned(workspace, kWsAlign)) return TPPO_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    StatArgs sa{};
    PolicyArgs& a = sa.p;
    a.logits = logits; a.R = R; a.V = V; a.ld = ld; a.targets = targets; a.rows = rows;
    a.n_sel = n_sel; a.n_max = n_max; a.aux_idx = aux_idx; a.old_logp = old_logp; a.adv = nullptr;
    // without old log-probs nothing is read through the index map: any index is then in range
    a.aux_len = old_logp ? aux_len : (int64_t(1) << 62);
    a.eps_low = 0.f; a.eps_high = 0.f; a.denom = 0.f; a.logp = logp; a.token_loss = nullptr;
    a.loss = nullptr; a.stats = stats; a.dlogits = nullptr; a.mode = TPPO_DLOGITS_NONE;
    char* w = static_cast<char*>(workspace);
    a.row_loss = reinterpret_cast<float*>(w);
    w += align_up(size_t(n_max > 0 ? n_max : 1) * sizeof(float), kWsAlign);
    a.row_clip = reinterpret_cast<uint8_t*>(w);
    w += align_up(size_t(n_max > 0 ? n_max : 1), kWsAlign);
    a.row_flag = reinterpret_cast<uint8_t*>(w);
    w += align_up(size_t(R > 0 ? R : 1), kWsAlign);
    a.rec = reinterpret_cast<RowRec*>(w);
    a.part = 0; a.side_share_256 = 0;
    sa.entropy = entropy;
    sa.means = means;

    TPPO_CUDA_CHECK(cudaMemsetAsync(stats, 0, 4 * sizeof(int32_t), s));
    if (n_max > 0) {
        const int rc = launch_policy_prepare(a, s);
        if (rc != TPPO_OK) return rc;
        int64_t blocks = n_max < kNumSms * 3 ? n_max : kNumSms * 3;
        const bool vec = aligned(logits, 16) && (ld * esz) % 16 == 0;
        if (logits_dtype == TPPO_BF16) {
            if (vec) policy_stats_kernel<uint16_t, true><<<unsigned(blocks), kStatThreads, 0, s>>>(sa);
            else policy_stats_kernel<uint16_t, false><<<unsigned(blocks), kStatThreads, 0, s>>>(sa);
        } else {
            if (vec) policy_stats_kernel<float, true><<<unsigned(blocks), kStatThreads, 0, s>>>(sa);
            else policy_stats_kernel<float, false><<<unsigned(blocks), kStatThreads, 0, s>>>(sa);
        }
        TPPO_CUDA_CHECK(cudaGetLastError());
    }
    policy_stats_finish_kernel<<<1, 1024, 0, s>>>(sa);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

// tppo_policy_loss_fwd_bwd: argument checks, workspace carving, kernel choice, and the small helper
// kernels (row marking, zero fill of rows that are not selected, fixed-order final reduction).
#include "policy_common.cuh"

namespace tppo {

// ---- helper kernels -----------------------------------------------------------------------
// Gathers the per-entry scalars (row, target, advantage, old log-prob) into 16-byte records, checks
// every index once, and in FULL mode marks the selected rows.
__global__ void policy_prepare_kernel(const PolicyArgs a) {
    const int64_t n = policy_n(a);
    int bad = 0;
    for (int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; j < n;
         j += int64_t(gridDim.x) * blockDim.x) {
        const RowMeta m = policy_row_meta(a, j);
        RowRec r;
        r.row = m.row_ok ? int32_t(m.row) : -1;
        r.y = m.ok ? m.y : -1;
        r.adv = (m.ok && a.adv) ? __ldg(a.adv + m.aux) : 0.f;              // absent when only the
        r.old_logp = (m.ok && a.old_logp) ? __ldg(a.old_logp + m.aux) : 0.f; // row statistics are wanted
        a.rec[j] = r;
        if (!m.ok) bad |= policy_bad_bits(m, a);
        if (m.row_ok && a.rows && a.mode == TPPO_DLOGITS_FULL) a.row_flag[m.row] = 1;
    }
    if (bad) atomicOr(a.stats + 3, bad);
}

// FULL mode: rows of dlogits that are not selected get zeros in their V columns.
template <typename T>
__global__ void __launch_bounds__(256) policy_zero_rows_kernel(const PolicyArgs a) {
    const int64_t n = policy_n(a);
    T* base = static_cast<T*>(a.dlogits);
    const bool vec = (reinterpret_cast<uintptr_t>(base) % 16 == 0) && ((a.ld * sizeof(T)) % 16 == 0);
    constexpr int kPer = 16 / sizeof(T);
    for (int64_t r = blockIdx.x; r < a.R; r += gridDim.x) {
        const bool selected = a.rows ? (a.row_flag[r] != 0) : (r < n);
        if (selected) continue;
        T* row = base + r * a.ld;
        if (vec) {
            const int nv = a.V / kPer;
            uint4* row4 = reinterpret_cast<uint4*>(row);
            for (int u = threadIdx.x; u < nv; u += blockDim.x) row4[u] = make_uint4(0, 0, 0, 0);
            for (int v = nv * kPer + threadIdx.x; v < a.V; v += blockDim.x) row[v] = T(0);
        } else {
            for (int v = threadIdx.x; v < a.V; v += blockDim.x) row[v] = T(0);
        }
    }
}

// Fixed-order reduction of the per-row terms: one block, strided per-thread sums in fp64, a fixed
// shuffle tree, then the warps in order.  Identical from run to run.
__global__ void __launch_bounds__(1024) policy_finish_kernel(const PolicyArgs a) {
    __shared__ double s_sum[32];
    __shared__ int s_lo[32], s_hi[32];
    const int64_t n = policy_n(a);
    double acc = 0.0;
    int lo = 0, hi = 0;
    // sixteen rows per trip (a whole 16384-row micro-batch in one), loads first, so that their
    // latencies overlap; the order of the adds is fixed
    constexpr int kPerTrip = 16;
    const int64_t step = blockDim.x;
    for (int64_t j = threadIdx.x; j < n; j += kPerTrip * step) {
        float l[kPerTrip];
        uint8_t c[kPerTrip];
#pragma unroll
        for (int u = 0; u < kPerTrip; ++u) {
            const int64_t q = j + u * step;
            l[u] = q < n ? a.row_loss[q] : 0.f;
            c[u] = q < n ? a.row_clip[q] : uint8_t(0);
        }
#pragma unroll
        for (int u = 0; u < kPerTrip; ++u) {
            acc += double(l[u]);
            lo += c[u] == 1;
            hi += c[u] == 2;
        }
    }
    acc = warp_sum(acc);
    lo = __reduce_add_sync(0xffffffffu, lo);
    hi = __reduce_add_sync(0xffffffffu, hi);
    if ((threadIdx.x & 31) == 0) {
        s_sum[threadIdx.x >> 5] = acc;
        s_lo[threadIdx.x >> 5] = lo;
        s_hi[threadIdx.x >> 5] = hi;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        int tl = 0, th = 0;
        for (int w = 0; w < int(blockDim.x >> 5); ++w) { t += s_sum[w]; tl += s_lo[w]; th += s_hi[w]; }
        const double d = a.denom > 0.f ? double(a.denom) : double(n > 0 ? n : 1);
        *a.loss = n > 0 ? float(t / d) : 0.f;
        a.stats[0] = int32_t(n);
        a.stats[1] = tl;
        a.stats[2] = th;
    }
}

// Host launchers of the two helper kernels for other translation units (the LM-head variant).
int launch_policy_prepare(const PolicyArgs& a, cudaStream_t s) {
    if (a.n_max <= 0) return TPPO_OK;
    const int pb = int((a.n_max + 255) / 256 < 1184 ? (a.n_max + 255) / 256 : 1184);
    policy_prepare_kernel<<<pb, 256, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}
int launch_policy_finish(const PolicyArgs& a, cudaStream_t s) {
    policy_finish_kernel<<<1, 1024, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

int launch_policy_two_pass(const PolicyArgs& a, int dtype, cudaStream_t s, int variant, int side_sms);
int launch_policy_cluster(const PolicyArgs& a, cudaStream_t s, int variant, int* idle_sms);
bool policy_cluster_supported(const PolicyArgs& a, int dtype);

constexpr int kSideShare256 = 22;       // 8.6 % of the rows: both launches then end together at V = 152064
constexpr int64_t kSideMinRows = 2048;  // below this the split is not worth a second launch

size_t policy_workspace_bytes(int64_t R, int64_t n_max) {
    const size_t n = size_t(n_max > 0 ? n_max : 1);
    return align_up(n * sizeof(float), kWsAlign) + align_up(n, kWsAlign) +
           align_up(size_t(R > 0 ? R : 1), kWsAlign) + align_up(n * sizeof(RowRec), kWsAlign);
}
}  // namespace tppo

using namespace tppo;

TPPO_API int tppo_policy_loss_fwd_bwd(const void* logits, int32_t logits_dtype, int64_t R, int32_t V,
                                      int64_t ld, const int32_t* targets, const int32_t* rows,
                                      const int32_t* n_sel, int64_t n_max, const int32_t* aux_idx,
                                      const float* old_logp, const float* adv, int64_t aux_len,
                                      float eps_low, float eps_high, float denom, float* logp,
                                      float* token_loss, float* loss, int32_t* stats, void* dlogits,
                                      int32_t dlogits_mode, int32_t kernel_hint, void* workspace,
                                      size_t workspace_bytes, void* stream) {
    if (logits_dtype != TPPO_BF16 && logits_dtype != TPPO_F32) return TPPO_ERR_INVALID_ARG;
    if (R < 0 || V <= 0 || ld < V || n_max < 0 || aux_len < 0 || R >= (int64_t(1) << 31))
        return TPPO_ERR_INVALID_ARG;
    if (!loss || !stats) return TPPO_ERR_INVALID_ARG;
    if (!rows && n_max > R) return TPPO_ERR_INVALID_ARG;
    if (n_max > 0 && (!logits || !targets || !old_logp || !adv)) return TPPO_ERR_INVALID_ARG;
    if (!(eps_low >= 0.f) || !(eps_high >= 0.f)) return TPPO_ERR_INVALID_ARG;
    if (dlogits_mode < TPPO_DLOGITS_NONE || dlogits_mode > TPPO_DLOGITS_COMPACT)
        return TPPO_ERR_INVALID_ARG;
    if (dlogits_mode != TPPO_DLOGITS_NONE && !dlogits && (R > 0 || n_max > 0))
        return TPPO_ERR_INVALID_ARG;
    const size_t esz = logits_dtype == TPPO_BF16 ? 2 : 4;
    if (!aligned(logits, esz) || (dlogits && !aligned(dlogits, esz))) return TPPO_ERR_INVALID_ARG;
    const size_t need = policy_workspace_bytes(R, n_max);
    if (!workspace || workspace_bytes < need || !aligned(workspace, kWsAlign))
        return TPPO_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    PolicyArgs a;
    a.logits = logits; a.R = R; a.V = V; a.ld = ld; a.targets = targets; a.rows = rows;
    a.n_sel = n_sel; a.n_max = n_max; a.aux_idx = aux_idx; a.old_logp = old_logp; a.adv = adv;
    a.aux_len = aux_len; a.eps_low = eps_low; a.eps_high = eps_high; a.denom = denom;
    a.logp = logp; a.token_loss = token_loss; a.loss = loss; a.stats = stats;
    a.dlogits = dlogits; a.mode = dlogits_mode;
    char* w = static_cast<char*>(workspace);
    a.row_loss = reinterpret_cast<float*>(w);
    w += align_up(size_t(n_max > 0 ? n_max : 1) * sizeof(float), kWsAlign);
    a.row_clip = reinterpret_cast<uint8_t*>(w);
    w += align_up(size_t(n_max > 0 ? n_max : 1), kWsAlign);
    a.row_flag = reinterpret_cast<uint8_t*>(w);
    w += align_up(size_t(R > 0 ? R : 1), kWsAlign);
    a.rec = reinterpret_cast<RowRec*>(w);
    a.part = 0;
    a.side_share_256 = 0;

    const int base_hint = kernel_hint & 0xff;
    const bool can_cluster = policy_cluster_supported(a, logits_dtype);
    if (base_hint == TPPO_POLICY_CLUSTER_SMEM && !can_cluster) return TPPO_ERR_UNSUPPORTED;
    if (base_hint != TPPO_POLICY_AUTO && base_hint != TPPO_POLICY_TWO_PASS &&
        base_hint != TPPO_POLICY_CLUSTER_SMEM)
        return TPPO_ERR_INVALID_ARG;

    TPPO_CUDA_CHECK(cudaMemsetAsync(stats, 0, 4 * sizeof(int32_t), s));
    const bool fill_rows = dlogits_mode == TPPO_DLOGITS_FULL && R > 0;
    if (fill_rows && rows) TPPO_CUDA_CHECK(cudaMemsetAsync(a.row_flag, 0, size_t(R), s));
    if (n_max > 0) {
        const int pb = int((n_max + 255) / 256 < 1184 ? (n_max + 255) / 256 : 1184);
        policy_prepare_kernel<<<pb, 256, 0, s>>>(a);
        // The cluster kernel wins when a gradient is written; a forward-only sweep reads each row
        // once in either kernel and the plain one keeps more rows in flight.
        const bool use_cluster = base_hint == TPPO_POLICY_CLUSTER_SMEM ||
                                 (base_hint == TPPO_POLICY_AUTO && can_cluster &&
                                  dlogits_mode != TPPO_DLOGITS_NONE);
        int rc = TPPO_ERR_UNSUPPORTED;
        if (use_cluster) {
            // The clusters cannot cover every SM (33 clusters of 4 on 148 SMs).  With enough rows the
            // tail of the row list goes to the plain kernel, launched as a programmatic dependent so
            // that it runs beside the cluster kernel on the SMs that one leaves idle.  Share of the
            // rows for it: bits 16-23 of the hint in 1/256 (255 = none), default kSideShare256.
            const int share_hint = (kernel_hint >> 16) & 0xff;
            const int share = share_hint == 255 ? 0 : (share_hint ? share_hint : kSideShare256);
            PolicyArgs front = a;
            front.part = 1;
            front.side_share_256 = n_max >= kSideMinRows ? share : 0;
            int idle_sms = 0;
            rc = launch_policy_cluster(front, s, (kernel_hint >> 8) & 0xff, &idle_sms);
            if (rc == TPPO_OK && front.side_share_256 > 0) {
                if (idle_sms >= 2) {
                    PolicyArgs tail = front;
                    tail.part = 2;
                    rc = launch_policy_two_pass(tail, logits_dtype, s, 0, idle_sms);
                } else {     // no room beside the clusters: the same rows, after them
                    PolicyArgs tail = front;
                    tail.part = 2;
                    rc = launch_policy_two_pass(tail, logits_dtype, s, 0, 0);
                }
            }
        }
        if (!use_cluster || (rc == TPPO_ERR_UNSUPPORTED && base_hint == TPPO_POLICY_AUTO))
            rc = launch_policy_two_pass(a, logits_dtype, s, (kernel_hint >> 8) & 0xff, 0);
        if (rc != TPPO_OK) return rc;
    }
    if (fill_rows) {
        const int zb = int(R < 1184 ? R : 1184);
        if (logits_dtype == TPPO_BF16) policy_zero_rows_kernel<uint16_t><<<zb, 256, 0, s>>>(a);
        else policy_zero_rows_kernel<float><<<zb, 256, 0, s>>>(a);
    }
    policy_finish_kernel<<<1, 1024, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

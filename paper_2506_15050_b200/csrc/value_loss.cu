// Clipped value regression on the value tokens, forward and backward (Eq. 4-5 of the paper;
// the value update of Algorithm 1).
//
// Two kernels, both gathers over the index list (16 bytes read per value token).  With a gradient
// (dvalues given) the call must write all N entries of dvalues, zero off the value tokens: every
// block then owns a range of positions, fills it with zeros itself and scatters the gradients of
// exactly the tokens that lie in it (found by a search in the ascending list), so that no separate
// clear of dvalues is needed.  (A dense sweep over the positions, which reads values / old values /
// returns with aligned 16-byte loads wherever a position is marked, was built and measured: 74 us
// against 59 us for gather + clear on 17.5 M positions at 25 % density -- 25 instructions per
// POSITION for Eq. 4-5 instead of per token, and a chain of dependent tile steps per block.)
//
// The mean is reduced in a fixed order (per-thread partials in fp64, a fixed shuffle tree,
// per-block partials summed by the last block to finish), so results are run-to-run identical.
#include "common.cuh"

namespace tppo {

constexpr int kValThreads = 256;
constexpr int kValMaxBlocks = kNumSms * 8;

struct ValueArgs {
    const float* values;
    const float* old_values;
    const float* returns;
    const int32_t* value_idx;
    const int32_t* n_sel;
    int64_t n_max;
    int64_t N;
    float xi_low, xi_high, denom;
    float* loss;
    float* dvalues;
    int32_t* stats;       // [2]: n, status bits
    double* partial;      // [gridDim.x]
    uint32_t* done;       // [1] blocks finished
    uint32_t* ws_status;  // [1] status bits gathered during the call
    int32_t vec_ok;       // dvalues is 16-byte aligned
};

__device__ __forceinline__ int64_t value_n(const ValueArgs& a) {
    int64_t n = a.n_max;
    if (a.n_sel) { const int64_t c = *a.n_sel; n = c < 0 ? 0 : (c < n ? c : n); }
    return n;
}

// One token of Eq. 4-5.  Returns the loss term (already halved) and the gradient before the division
// by the number of tokens.  A token whose value, old value or return is not finite contributes
// nothing and sets `nonfinite`.
__device__ __forceinline__ float value_token(float v, float vo, float R, float xi_low, float xi_high,
                                             float& g, bool& nonfinite) {
    const float probe = fmaf(v, 0.f, fmaf(vo, 0.f, R * 0.f));     // NaN iff any of the three is not finite
    if (probe != probe) { nonfinite = true; g = 0.f; return 0.f; }
    const float vc = fminf(fmaxf(v, vo - xi_low), vo + xi_high);
    const float e1 = (v - R) * (v - R), e2 = (vc - R) * (vc - R);
    if (e1 >= e2) { g = v - R; return 0.5f * e1; }
    g = (vc == v) ? (vc - R) : 0.f;
    return 0.5f * e2;
}

// Block-wide sum of the per-thread partials in a fixed order, then the hand-over to the last block:
// every block stores its partial, the last one to finish adds them (strided per thread, fixed
// tree) and writes the loss, the count and the status bits.
__device__ __forceinline__ void value_finish(const ValueArgs& a, double acc, int bad, int64_t n,
                                             double* s_red, bool* s_last) {
    if (bad) {
        atomicOr(a.ws_status, uint32_t(bad));
        __threadfence();      // performed before the block counts itself as finished
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < kValThreads / 32; ++w) t += s_red[w];
        a.partial[blockIdx.x] = t;
        __threadfence();
        *s_last = atomicAdd(a.done, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (*s_last) {
        __threadfence();
        double t = 0.0;
        for (unsigned b = threadIdx.x; b < gridDim.x; b += kValThreads)
            t += reinterpret_cast<volatile double*>(a.partial)[b];
        t = warp_sum(t);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = t;
        __syncthreads();
        if (threadIdx.x == 0) {
            double tot = 0.0;
            for (int w = 0; w < kValThreads / 32; ++w) tot += s_red[w];
            const double d = a.denom > 0.f ? double(a.denom) : double(n > 0 ? n : 1);
            *a.loss = n > 0 ? float(tot / d) : 0.f;
            a.stats[0] = int32_t(n);
            a.stats[1] = int32_t(*reinterpret_cast<volatile uint32_t*>(a.ws_status));
        }
    }
}

// ---- without a gradient: gather over the index list ------------------------------------------------
__global__ void __launch_bounds__(kValThreads) value_loss_gather_kernel(const ValueArgs a) {
    __shared__ double s_red[kValThreads / 32];
    __shared__ bool s_last;
    const int64_t n = value_n(a);
    double acc = 0.0;
    int bad = 0;
    bool nonfinite = false;
    // Four independent tokens per thread and trip, so that the index load and the three gathers of
    // one token overlap with those of the others.
    constexpr int kUnroll = 4;
    const int64_t stride = int64_t(gridDim.x) * kValThreads;
    for (int64_t j0 = int64_t(blockIdx.x) * kValThreads + threadIdx.x; j0 < n; j0 += stride * kUnroll) {
        int64_t p[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t j = j0 + u * stride;
            p[u] = j < n ? (a.value_idx ? int64_t(__ldg(a.value_idx + j)) : j) : -1;
            ok[u] = p[u] >= 0 && p[u] < a.N;
            if (j < n && !ok[u]) bad = TPPO_DEV_BAD_INDEX;
        }
        float v[kUnroll], vo[kUnroll], R[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t q = ok[u] ? p[u] : 0;
            v[u] = ok[u] ? __ldg(a.values + q) : 0.f;
            vo[u] = ok[u] ? __ldg(a.old_values + q) : 0.f;
            R[u] = ok[u] ? __ldg(a.returns + q) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (!ok[u]) continue;
            float g;
            acc += double(value_token(v[u], vo[u], R[u], a.xi_low, a.xi_high, g, nonfinite));
        }
    }
    if (nonfinite) bad |= TPPO_DEV_NONFINITE;
    value_finish(a, acc, bad, n, s_red, &s_last);
}

// ---- with a gradient: every block owns a range of positions ---------------------------------------------
// Number of entries of the ascending list idx[0..n) that are < key (whole warp, 32 probes a round).
__device__ __forceinline__ int64_t value_lower_bound(const int32_t* __restrict__ idx, int64_t n,
                                                     int64_t key, int lane) {
    int64_t lo = 0, hi = n;
    while (hi > lo) {
        const int64_t step = (hi - lo + 31) >> 5;
        const int64_t q = lo + lane * step;
        const bool lt = q < hi && int64_t(__ldg(idx + q)) < key;
        const uint32_t m = __ballot_sync(0xffffffffu, lt);
        const int c = __ffs(int(~m)) - 1;            // leading run of probes that are < key
        if (c < 0) { lo = min(lo + 31 * step + 1, hi); continue; }
        const int64_t new_hi = min(lo + c * step, hi);
        if (c > 0) lo = lo + (c - 1) * step + 1;
        hi = new_hi;
    }
    return lo;
}

// dvalues must come out complete: the gradient on the value tokens, zero everywhere else.  Block b
// owns the positions [b N/G, (b+1) N/G): it fills them with zeros (coalesced 16-byte stores), finds
// the part of the ascending index list that falls inside them (two warp-wide searches, which run
// while the other warps are still filling), and after one barrier gathers and scatters exactly those
// tokens.  Filling and scattering of a position are thus done by the same block, in that order:
// no separate clear of dvalues, no ordering between blocks.
constexpr int kValGradBlocksPerSm = 5;
__global__ void __launch_bounds__(kValThreads, kValGradBlocksPerSm) value_loss_grad_kernel(const ValueArgs a) {
    __shared__ double s_red[kValThreads / 32];
    __shared__ bool s_last;
    __shared__ int64_t s_range[2];

    const int64_t n = value_n(a);
    const double d = a.denom > 0.f ? double(a.denom) : double(n > 0 ? n : 1);
    const float inv_d = float(1.0 / d);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double acc = 0.0;
    int bad = 0;
    bool nonfinite = false;

    // this block's positions, on 4-position boundaries
    const int64_t quads = (a.N + 3) >> 2;
    const int64_t p0 = (quads * blockIdx.x / gridDim.x) << 2;
    const int64_t p1 = min(a.N, (quads * (blockIdx.x + 1) / gridDim.x) << 2);

    // The scheme relies on a strictly ascending list with entries in [0, N) (the order the token
    // filter writes): every adjacent pair is checked once, each block taking a strided share.
    if (a.value_idx) {
        const bool vec = (reinterpret_cast<uintptr_t>(a.value_idx) & 15) == 0;
        for (int64_t q = (int64_t(blockIdx.x) * kValThreads + tid) * 4; q < n;
             q += int64_t(gridDim.x) * kValThreads * 4) {
            int32_t e[5];
            if (vec && q + 4 <= n) {
                const int4 x = __ldg(reinterpret_cast<const int4*>(a.value_idx + q));
                e[0] = x.x; e[1] = x.y; e[2] = x.z; e[3] = x.w;
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) e[k] = q + k < n ? __ldg(a.value_idx + q + k) : INT32_MAX;
            }
            e[4] = q + 4 < n ? __ldg(a.value_idx + q + 4) : INT32_MAX;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (q + k < n && (e[k] < 0 || e[k] >= a.N)) bad = TPPO_DEV_BAD_INDEX;
                if (q + k + 1 < n && e[k + 1] <= e[k]) bad = TPPO_DEV_BAD_INDEX;
            }
        }
    }
    // the entries of the list inside [p0, p1): searched by the first two warps ...
    if (a.value_idx) {
        if (warp < 2) {
            const int64_t c = value_lower_bound(a.value_idx, n, warp == 0 ? p0 : p1, lane);
            if (lane == 0) s_range[warp] = c;
        }
    } else if (tid == 0) {       // no list: positions 0 .. n-1 are the tokens
        s_range[0] = min(p0, n);
        s_range[1] = min(p1, n);
    }
    // ... while everybody fills the block's positions with zeros
    if (a.vec_ok) {
        float4* z = reinterpret_cast<float4*>(a.dvalues + p0);
        const int64_t nq = (p1 - p0) >> 2;
        for (int64_t k = tid; k < nq; k += kValThreads) z[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int64_t p = p0 + (nq << 2) + tid; p < p1; p += kValThreads) a.dvalues[p] = 0.f;
    } else {
        for (int64_t p = p0 + tid; p < p1; p += kValThreads) a.dvalues[p] = 0.f;
    }
    __syncthreads();
    const int64_t j0 = s_range[0], j1 = s_range[1];

    // Four independent tokens per thread and trip, so that the index load and the three gathers of
    // one token overlap with those of the others.
    constexpr int kUnroll = 4;
    for (int64_t jb = j0 + tid; jb < j1; jb += kValThreads * kUnroll) {
        int64_t p[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t j = jb + u * kValThreads;
            p[u] = j < j1 ? (a.value_idx ? int64_t(__ldg(a.value_idx + j)) : j) : -1;
            // (an entry outside this block's positions can only come from a list that is not ascending,
            // which the check above reports; it is skipped so that no other block's zeros are touched)
            ok[u] = p[u] >= p0 && p[u] < p1;
        }
        float v[kUnroll], vo[kUnroll], R[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t q = ok[u] ? p[u] : 0;
            v[u] = ok[u] ? __ldg(a.values + q) : 0.f;
            vo[u] = ok[u] ? __ldg(a.old_values + q) : 0.f;
            R[u] = ok[u] ? __ldg(a.returns + q) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (!ok[u]) continue;
            float g;
            acc += double(value_token(v[u], vo[u], R[u], a.xi_low, a.xi_high, g, nonfinite));
            a.dvalues[p[u]] = g * inv_d;
        }
    }
    if (nonfinite) bad |= TPPO_DEV_NONFINITE;
    value_finish(a, acc, bad, n, s_red, &s_last);
}

size_t value_workspace_bytes() {
    return align_up(2 * sizeof(uint32_t), kWsAlign) + align_up(sizeof(double) * kValMaxBlocks, kWsAlign);
}

}  // namespace tppo

using namespace tppo;

TPPO_API int tppo_value_loss(const float* values, const float* old_values, const float* returns,
                             int64_t N, const int32_t* value_idx, const int32_t* n_sel,
                             int64_t n_max, float xi_low, float xi_high, float denom, float* loss,
                             float* dvalues, int32_t* stats, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (N < 0 || n_max < 0 || N >= (int64_t(1) << 31) || !loss || !stats)
        return TPPO_ERR_INVALID_ARG;
    if (n_max > 0 && (!values || !old_values || !returns)) return TPPO_ERR_INVALID_ARG;
    if (!value_idx && n_max > N) return TPPO_ERR_INVALID_ARG;
    if (!(xi_low >= 0.f) || !(xi_high >= 0.f)) return TPPO_ERR_INVALID_ARG;
    const size_t need = value_workspace_bytes();
    if (!workspace || workspace_bytes < need || !aligned(workspace, kWsAlign))
        return TPPO_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // one clear: the finished-blocks counter and the status word the blocks raise bits in; the loss,
    // the count and the status bits are all written by the last block to finish
    TPPO_CUDA_CHECK(cudaMemsetAsync(workspace, 0, 2 * sizeof(uint32_t), s));
    ValueArgs a;
    a.values = values; a.old_values = old_values; a.returns = returns; a.value_idx = value_idx;
    a.n_sel = n_sel; a.n_max = n_max; a.N = N; a.xi_low = xi_low; a.xi_high = xi_high;
    a.denom = denom; a.loss = loss; a.dvalues = dvalues; a.stats = stats;
    a.done = static_cast<uint32_t*>(workspace);
    a.ws_status = a.done + 1;
    a.partial = reinterpret_cast<double*>(static_cast<char*>(workspace) +
                                          align_up(2 * sizeof(uint32_t), kWsAlign));
    a.vec_ok = aligned(dvalues, 16);
    if (dvalues && N > 0) {
        // one block per 16384 positions, at most one wave of resident blocks
        int64_t blocks = (N + 16383) / 16384;
        if (blocks > kNumSms * kValGradBlocksPerSm) blocks = kNumSms * kValGradBlocksPerSm;
        value_loss_grad_kernel<<<unsigned(blocks), kValThreads, 0, s>>>(a);
    } else {
        int64_t blocks = (n_max + kValThreads - 1) / kValThreads;
        if (blocks < 1) blocks = 1;
        if (blocks > kValMaxBlocks) blocks = kValMaxBlocks;
        value_loss_gather_kernel<<<unsigned(blocks), kValThreads, 0, s>>>(a);
    }
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

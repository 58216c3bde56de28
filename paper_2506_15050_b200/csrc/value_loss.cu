// Clipped value regression on the value tokens, forward and backward (Eq. 4-5 of the paper;
// the value update of Algorithm 1).
//
// Two kernels.  With a gradient (dvalues given) the call must write all N entries of dvalues, zero
// off the value tokens, so the kernel sweeps the packed POSITIONS in order: a block owns a contiguous
// range of positions, walks it tile by tile, marks in shared memory which positions of the tile the
// ascending index list names, and then reads values / old values / returns and writes dvalues with
// aligned 16-byte accesses -- zeros where nothing is marked.  No separate zero fill, no scattered
// 4-byte stores, and at the densities of a training batch (a large part of all positions are value
// tokens) every 32-byte sector is fetched once by a coalesced load instead of by a gather.  Without a
// gradient the call is a plain gather over the index list (16 bytes per value token).
//
// The mean is reduced in a fixed order (per-thread partials in fp64, a fixed shuffle tree,
// per-block partials summed by the last block to finish), so results are run-to-run identical.
#include "common.cuh"

namespace tppo {

constexpr int kValThreads = 256;
constexpr int kValMaxBlocks = kNumSms * 8;
// sweep: a tile's index window is 16 entries per thread starting at a 4-entry boundary at or below
// the cursor, so it always covers every entry a tile of kValTile positions can own
constexpr int kValWinPerThread = 16;
constexpr int kValWindow = kValThreads * kValWinPerThread;      // 4096 index entries
constexpr int kValTile = kValWindow - 64;                       // 4032 positions (a multiple of 4)
constexpr int kValGroups = kValTile / 4;                        // float4 groups per tile

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
    int32_t vec_ok;       // values, old_values, returns, dvalues are 16-byte aligned
    int32_t tiles_per_block;
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

// ---- with a gradient: sweep over the positions ---------------------------------------------------------
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

__global__ void __launch_bounds__(kValThreads) value_loss_sweep_kernel(const ValueArgs a) {
    __shared__ __align__(16) uint8_t s_flag[kValTile + 64];
    __shared__ double s_red[kValThreads / 32];
    __shared__ bool s_last;
    __shared__ int64_t s_cursor;

    const int64_t n = value_n(a);
    const double d = a.denom > 0.f ? double(a.denom) : double(n > 0 ? n : 1);
    const float inv_d = float(1.0 / d);
    const int tid = threadIdx.x, lane = tid & 31;
    const int64_t num_tiles = (a.N + kValTile - 1) / kValTile;
    const int64_t tile_first = int64_t(blockIdx.x) * a.tiles_per_block;
    const int64_t tile_end = min(num_tiles, tile_first + a.tiles_per_block);

    double acc = 0.0;
    int bad = 0;
    bool nonfinite = false;
    // The sweep relies on a strictly ascending list with entries in [0, N) (the order the token
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
    // entries of the list that lie before this block's first position
    if (a.value_idx && tile_first < tile_end) {
        if (tid < 32) {
            const int64_t c = value_lower_bound(a.value_idx, n, tile_first * kValTile, lane);
            if (lane == 0) s_cursor = c;
        }
    } else if (tid == 0) {
        s_cursor = 0;
    }
    __syncthreads();

    for (int64_t tile = tile_first; tile < tile_end; ++tile) {
        const int64_t t0 = tile * kValTile;
        const int64_t t1 = min(t0 + kValTile, a.N);
        const int64_t cursor = s_cursor;
        // ---- which positions of the tile are value tokens ---------------------------------------------
        for (int k = tid * 16; k < kValTile; k += kValThreads * 16)
            *reinterpret_cast<uint4*>(s_flag + k) = make_uint4(0, 0, 0, 0);
        __syncthreads();            // flags cleared; every thread has read the cursor
        if (a.value_idx) {
            // the window starts at a 4-entry boundary (aligned 16-byte loads); entries before the
            // cursor lie before the tile and are ignored by the range test like any other
            const int64_t w0 = (cursor & ~int64_t(3)) + int64_t(tid) * kValWinPerThread;
            int32_t e[kValWinPerThread + 1];
            if (w0 + kValWinPerThread < n && (reinterpret_cast<uintptr_t>(a.value_idx) & 15) == 0) {
#pragma unroll
                for (int q = 0; q < kValWinPerThread / 4; ++q) {
                    const int4 x = __ldg(reinterpret_cast<const int4*>(a.value_idx + w0) + q);
                    e[4 * q] = x.x; e[4 * q + 1] = x.y; e[4 * q + 2] = x.z; e[4 * q + 3] = x.w;
                }
                e[kValWinPerThread] = __ldg(a.value_idx + w0 + kValWinPerThread);
            } else {
#pragma unroll
                for (int q = 0; q <= kValWinPerThread; ++q)
                    e[q] = w0 + q < n ? __ldg(a.value_idx + w0 + q) : INT32_MAX;
            }
#pragma unroll
            for (int q = 0; q < kValWinPerThread; ++q) {
                const int64_t p = e[q];
                if (w0 + q < n) {
                    if (p >= t0 && p < t1) s_flag[p - t0] = 1;
                    // the first entry at or beyond the tile's end is where the next tile starts
                    if (p < t1 && (w0 + q + 1 >= n || int64_t(e[q + 1]) >= t1)) s_cursor = w0 + q + 1;
                }
            }
        }
        __syncthreads();
        // ---- the tile's positions, four at a time -------------------------------------------------------
        for (int gq = tid; gq < kValGroups; gq += kValThreads) {
            const int64_t p = t0 + 4 * gq;
            if (p >= t1) break;
            uint32_t f = *reinterpret_cast<const uint32_t*>(s_flag + 4 * gq);
            if (!a.value_idx) {       // no list: positions 0 .. n-1
                f = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) f |= (p + e < n ? 1u : 0u) << (8 * e);
            }
            float g[4] = {0.f, 0.f, 0.f, 0.f};
            const bool whole = p + 4 <= t1 && a.vec_ok;
            if (f) {
                float v[4], vo[4], R[4];
                if (whole) {
                    const float4 v4 = __ldg(reinterpret_cast<const float4*>(a.values + p));
                    const float4 o4 = __ldg(reinterpret_cast<const float4*>(a.old_values + p));
                    const float4 r4 = __ldg(reinterpret_cast<const float4*>(a.returns + p));
                    v[0] = v4.x; v[1] = v4.y; v[2] = v4.z; v[3] = v4.w;
                    vo[0] = o4.x; vo[1] = o4.y; vo[2] = o4.z; vo[3] = o4.w;
                    R[0] = r4.x; R[1] = r4.y; R[2] = r4.z; R[3] = r4.w;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const bool in = p + e < t1 && ((f >> (8 * e)) & 0xffu);
                        v[e] = in ? __ldg(a.values + p + e) : 0.f;
                        vo[e] = in ? __ldg(a.old_values + p + e) : 0.f;
                        R[e] = in ? __ldg(a.returns + p + e) : 0.f;
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if ((f >> (8 * e)) & 0xffu) {
                        float ge;
                        acc += double(value_token(v[e], vo[e], R[e], a.xi_low, a.xi_high, ge, nonfinite));
                        g[e] = ge * inv_d;
                    }
                }
            }
            if (whole) {
                *reinterpret_cast<float4*>(a.dvalues + p) = make_float4(g[0], g[1], g[2], g[3]);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (p + e < t1) a.dvalues[p + e] = g[e];
            }
        }
        // (the next turn's first barrier separates these reads of the flags from their clearing)
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
    a.vec_ok = aligned(values, 16) && aligned(old_values, 16) && aligned(returns, 16) &&
               aligned(dvalues, 16);
    a.tiles_per_block = 1;
    if (dvalues && N > 0) {
        const int64_t tiles = (N + kValTile - 1) / kValTile;
        int64_t blocks = tiles < kValMaxBlocks ? tiles : kValMaxBlocks;
        a.tiles_per_block = int32_t((tiles + blocks - 1) / blocks);
        blocks = (tiles + a.tiles_per_block - 1) / a.tiles_per_block;
        value_loss_sweep_kernel<<<unsigned(blocks), kValThreads, 0, s>>>(a);
    } else {
        int64_t blocks = (n_max + kValThreads - 1) / kValThreads;
        if (blocks < 1) blocks = 1;
        if (blocks > kValMaxBlocks) blocks = kValMaxBlocks;
        value_loss_gather_kernel<<<unsigned(blocks), kValThreads, 0, s>>>(a);
    }
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

// Clipped value regression on the value tokens, forward and backward (Eq. 4-5 of the paper;
// the value update of Algorithm 1).
//
// A gather over value_idx: 3 fp32 reads + 1 index read + 1 gradient write per value token.  dvalues is
// zero off the value tokens: a first kernel fills it with 16-byte stores (and clears the two words
// the blocks count in), the loss kernel is its programmatic dependent and scatters the tokens'
// entries once that kernel has ended.  Measured on 17.5 M positions at 25 % density: 53.5 us per call
// in this form with four blocks per SM and four tokens per trip, 49-50 us with eight blocks and two tokens; 55.8 us with two memsets in front of a plain launch; 61 us when the dependent kernel
// starts its gathers beside the fill, holds the gradients of its first 8192 tokens per block in
// shared memory and scatters them after the fill has ended (the fill and the gathers then share the
// DRAM and neither runs at its own rate); 74 us for a dense sweep over the positions that writes
// dvalues whole (it evaluates Eq. 4-5 per position instead of per token and walks its tiles in a
// dependent chain); 63-76 us for blocks that own a range of positions, zero-fill it themselves and
// scatter only the tokens inside it (found by a search in the ascending list: the fill and the
// gather of a block are serialised by its barrier, and the search is pure latency on top).
//
// The mean is reduced in a fixed order (per-thread partials in fp64, a fixed shuffle tree,
// per-block partials summed by the last block to finish), so results are run-to-run identical.
#include "common.cuh"

namespace tppo {

constexpr int kValThreads = 256;
constexpr int kValBlocksPerSm = 8;      // 2048 resident threads per SM at 32 registers
constexpr int kValMaxBlocks = kNumSms * kValBlocksPerSm;

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

// Zero-fills dvalues and clears the two words of the workspace the blocks count in.  The loss
// kernel is its programmatic dependent and runs beside it.
__global__ void __launch_bounds__(512) value_clear_kernel(float* dvalues, int64_t N, uint32_t* ws) {
    asm volatile("griddepcontrol.launch_dependents;");
    if (blockIdx.x == 0 && threadIdx.x < 2) ws[threadIdx.x] = 0u;
    if (!dvalues || N <= 0) return;
    // head up to the first 16-byte boundary, 16-byte stores, tail
    const int64_t head = min(N, int64_t((16 - (reinterpret_cast<uintptr_t>(dvalues) & 15)) & 15) / 4);
    const int64_t n4 = (N - head) / 4;
    const int64_t tid = int64_t(blockIdx.x) * blockDim.x + threadIdx.x, nthr = int64_t(gridDim.x) * blockDim.x;
    if (tid < head) dvalues[tid] = 0.f;
    float4* d4 = reinterpret_cast<float4*>(dvalues + head);
    for (int64_t i = tid; i < n4; i += nthr) d4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int64_t done = head + 4 * n4;
    if (tid < N - done) dvalues[done + tid] = 0.f;
}

// Launched as the programmatic dependent of the clearing kernel: its blocks are resident and have
// their arguments when that kernel ends, and start the moment it does.
__global__ void __launch_bounds__(kValThreads, kValBlocksPerSm) value_loss_kernel(const ValueArgs a) {
    __shared__ double s_red[kValThreads / 32];
    __shared__ bool s_last;
    const int64_t n = value_n(a);
    const double d = a.denom > 0.f ? double(a.denom) : double(n > 0 ? n : 1);
    const float inv_d = float(1.0 / d);
    double acc = 0.0;
    int bad = 0;
    bool nonfinite = false;
    // Two independent tokens per thread and trip, so that the index load and the three gathers of
    // one token overlap with those of the other, and eight blocks per SM: measured at 17.5 M
    // positions, call us: four blocks x four tokens 52.7, five x four 50.3, six x four 51.8, four x
    // eight 51.4, eight x four 51.1, eight x three 50.5, eight x two 49.1-50.3.  The indices of a trip
    // are loaded one trip ahead (those of the first trip before the wait for the clearing kernel,
    // which writes nothing this kernel reads before it), so that a trip's gathers start at once:
    // 50.8 -> 48.3-49.3 us.  (Indices two trips ahead plus an L2 prefetch of the next trip's three
    // gathers: 49.5-50.2, dropped.)
    constexpr int kUnroll = 2;
    const int64_t stride = int64_t(gridDim.x) * kValThreads;
    auto load_indices = [&](int64_t j0, int32_t (&p)[kUnroll]) {       // (N < 2^31 is checked by the host)
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t j = j0 + u * stride;
            p[u] = j < n ? (a.value_idx ? __ldg(a.value_idx + j) : int32_t(j)) : -1;
        }
    };
    int64_t j0 = int64_t(blockIdx.x) * kValThreads + threadIdx.x;
    int32_t p_next[kUnroll];
    load_indices(j0, p_next);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (; j0 < n; j0 += stride * kUnroll) {
        int32_t p[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            p[u] = p_next[u];
            ok[u] = p[u] >= 0 && p[u] < a.N;
            if (j0 + u * stride < n && !ok[u]) bad = TPPO_DEV_BAD_INDEX;
        }
        load_indices(j0 + stride * kUnroll, p_next);
        float v[kUnroll], vo[kUnroll], R[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int32_t q = ok[u] ? p[u] : 0;
            v[u] = ok[u] ? __ldg(a.values + q) : 0.f;
            vo[u] = ok[u] ? __ldg(a.old_values + q) : 0.f;
            R[u] = ok[u] ? __ldg(a.returns + q) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (!ok[u]) continue;
            float g;
            acc += double(value_token(v[u], vo[u], R[u], a.xi_low, a.xi_high, g, nonfinite));
            if (a.dvalues) a.dvalues[p[u]] = g * inv_d;
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
    ValueArgs a;
    a.values = values; a.old_values = old_values; a.returns = returns; a.value_idx = value_idx;
    a.n_sel = n_sel; a.n_max = n_max; a.N = N; a.xi_low = xi_low; a.xi_high = xi_high;
    a.denom = denom; a.loss = loss; a.dvalues = dvalues; a.stats = stats;
    a.done = static_cast<uint32_t*>(workspace);
    a.ws_status = a.done + 1;
    a.partial = reinterpret_cast<double*>(static_cast<char*>(workspace) +
                                          align_up(2 * sizeof(uint32_t), kWsAlign));
    // dvalues is zero off the value tokens: one kernel clears it (and the finished-blocks counter and
    // the status word the blocks raise bits in); the loss kernel starts beside it
    value_clear_kernel<<<kNumSms * 2, 512, 0, s>>>(dvalues, N, a.done);
    TPPO_CUDA_CHECK(cudaGetLastError());
    int64_t blocks = (n_max + kValThreads - 1) / kValThreads;
    if (blocks < 1) blocks = 1;
    if (blocks > kValMaxBlocks) blocks = kValMaxBlocks;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(blocks));
    cfg.blockDim = dim3(kValThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    TPPO_CUDA_CHECK(cudaLaunchKernelEx(&cfg, value_loss_kernel, a));
    return TPPO_OK;
}

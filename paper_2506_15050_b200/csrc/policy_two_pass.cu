// General-shape policy-loss kernel: one thread block per selected row, the row is read twice from
// global memory (the second read usually hits L2).  Serves fp32 logits, vocabulary sizes and row
// strides that the shared-memory-resident kernel cannot take, and small problems.
//   pass 1: per-thread online max / sum-of-exponentials, block combine  -> log-sum-exp
//   scalar: Eq. 1 ratio, clip, loss term, gradient factor
//   pass 2: gradient factor * (softmax - onehot) written in the logits' element type
#include "policy_common.cuh"

namespace tppo {

constexpr int kTwoPassThreads = 512;

template <int DT> struct ElemT;
template <> struct ElemT<TPPO_BF16> { using type = uint16_t; };
template <> struct ElemT<TPPO_F32> { using type = float; };

__device__ __forceinline__ float load_elem(const uint16_t* p) { return __uint_as_float(uint32_t(*p) << 16); }
__device__ __forceinline__ float load_elem(const float* p) { return *p; }
__device__ __forceinline__ void store_elem(uint16_t* p, float v) {
    *p = uint16_t(pack_bf16x2(v, 0.f) & 0xffffu);
}
__device__ __forceinline__ void store_elem(float* p, float v) { *p = v; }

// The same in two steps, so that several loads can be issued before the first is used.
template <typename T> struct RawUnit;
template <> struct RawUnit<uint16_t> { uint4 w; };
template <> struct RawUnit<float> { float4 a, b; };
__device__ __forceinline__ RawUnit<uint16_t> load_raw(const uint16_t* p) {
    return RawUnit<uint16_t>{*reinterpret_cast<const uint4*>(p)};
}
__device__ __forceinline__ RawUnit<float> load_raw(const float* p) {
    return RawUnit<float>{*reinterpret_cast<const float4*>(p), *reinterpret_cast<const float4*>(p + 4)};
}
__device__ __forceinline__ void widen8(const RawUnit<uint16_t>& r, float (&x)[8]) {
    x[0] = bf16_lo(r.w.x); x[1] = bf16_hi(r.w.x); x[2] = bf16_lo(r.w.y); x[3] = bf16_hi(r.w.y);
    x[4] = bf16_lo(r.w.z); x[5] = bf16_hi(r.w.z); x[6] = bf16_lo(r.w.w); x[7] = bf16_hi(r.w.w);
}
__device__ __forceinline__ void widen8(const RawUnit<float>& r, float (&x)[8]) {
    x[0] = r.a.x; x[1] = r.a.y; x[2] = r.a.z; x[3] = r.a.w; x[4] = r.b.x; x[5] = r.b.y; x[6] = r.b.z; x[7] = r.b.w;
}

// 8 consecutive elements from a 16-byte aligned address
__device__ __forceinline__ void load8(const uint16_t* p, float (&x)[8]) {
    const uint4 w = *reinterpret_cast<const uint4*>(p);
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
}
__device__ __forceinline__ void load8(const float* p, float (&x)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void store8(uint16_t* p, const float (&g)[8]) {
    uint4 w;
    w.x = pack_bf16x2(g[0], g[1]); w.y = pack_bf16x2(g[2], g[3]);
    w.z = pack_bf16x2(g[4], g[5]); w.w = pack_bf16x2(g[6], g[7]);
    *reinterpret_cast<uint4*>(p) = w;
}
__device__ __forceinline__ void store8(float* p, const float (&g)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(g[0], g[1], g[2], g[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(g[4], g[5], g[6], g[7]);
}

// running (max, sum of 2^((x - max)*log2e)) update with n new values; the difference is formed
// before the scaling so that logits of any finite magnitude stay in range
template <int N>
__device__ __forceinline__ void online_update(float& m, float& s, const float (&x)[N]) {
    float mx = x[0];
#pragma unroll
    for (int k = 1; k < N; ++k) mx = fmaxf(mx, x[k]);
    const float m_new = fmaxf(m, mx);
    float acc = s * ex2((m - m_new) * kLog2e);
#pragma unroll
    for (int k = 0; k < N; ++k) acc += ex2((x[k] - m_new) * kLog2e);
    m = m_new;
    s = acc;
}

template <int DT, bool VEC>
__global__ void __launch_bounds__(kTwoPassThreads) policy_two_pass_kernel(const PolicyArgs a) {
    using T = typename ElemT<DT>::type;
    __shared__ float s_m[kTwoPassThreads / 32], s_s[kTwoPassThreads / 32];
    __shared__ float s_max, s_logsum, s_coef;

    const int64_t n = policy_n(a);
    const float inv_denom = policy_inv_denom(a, n);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T* logits = static_cast<const T*>(a.logits);
    T* dl = static_cast<T*>(a.dlogits);

    int64_t part_lo, part_hi;
    policy_part(a, n, part_lo, part_hi);
    for (int64_t j = part_lo + blockIdx.x; j < part_hi; j += gridDim.x) {
        const RowRec rec = load_rec(a.rec + j);
        const bool row_ok = rec.row >= 0, rec_ok = rec.y >= 0;
        const T* x_row = logits + int64_t(row_ok ? rec.row : 0) * a.ld;
        T* g_row = nullptr;
        if (a.mode == TPPO_DLOGITS_FULL && row_ok) g_row = dl + int64_t(rec.row) * a.ld;
        if (a.mode == TPPO_DLOGITS_COMPACT) g_row = dl + j * int64_t(a.V);

        float coef = 0.f, row_max = 0.f, log_sum = 0.f;
        if (rec_ok) {
            // ---- pass 1 -------------------------------------------------------------------
            float m = -kFltMax, s = 0.f;      // most negative finite: no inf - inf on masked (-inf) logits
            if (VEC) {
                const int nu = a.V >> 3;
                // four independent 16-byte loads per thread and trip: a single load in flight per
                // thread leaves the sweep bound by memory latency
                constexpr int kDeep = 4;
                int u = tid;
                for (; u + (kDeep - 1) * kTwoPassThreads < nu; u += kDeep * kTwoPassThreads) {
                    RawUnit<T> raw[kDeep];
#pragma unroll
                    for (int d = 0; d < kDeep; ++d) raw[d] = load_raw(x_row + (int64_t(u + d * kTwoPassThreads) << 3));
#pragma unroll
                    for (int d = 0; d < kDeep; ++d) {
                        float x[8];
                        widen8(raw[d], x);
                        online_update<8>(m, s, x);
                    }
                }
                for (; u < nu; u += kTwoPassThreads) {
                    float x[8];
                    load8(x_row + (int64_t(u) << 3), x);
                    online_update<8>(m, s, x);
                }
                for (int v = (nu << 3) + tid; v < a.V; v += kTwoPassThreads) {
                    float x[1] = {load_elem(x_row + v)};
                    online_update<1>(m, s, x);
                }
            } else {
                for (int v = tid; v < a.V; v += kTwoPassThreads) {
                    float x[1] = {load_elem(x_row + v)};
                    online_update<1>(m, s, x);
                }
            }
            const float wm = warp_max(m);
            s = warp_sum(s * ex2((m - wm) * kLog2e));
            if (lane == 0) { s_m[warp] = wm; s_s[warp] = s; }
            __syncthreads();
            if (tid == 0) {
                float M = s_m[0];
                for (int w = 1; w < kTwoPassThreads / 32; ++w) M = fmaxf(M, s_m[w]);
                float S = 0.f;
                for (int w = 0; w < kTwoPassThreads / 32; ++w) S += s_s[w] * ex2((s_m[w] - M) * kLog2e);
                // not a positive finite sum: the row held a NaN or +inf logit, or nothing but -inf;
                // it contributes nothing and raises the status bit
                const bool row_finite = S > 0.f && S <= kFltMax && M <= kFltMax;
                const float log_s = row_finite ? logf(S) : 0.f;
                RowLoss rl;
                rl.logp = 0.f; rl.loss = 0.f; rl.coef = 0.f; rl.clip = 0;
                if (row_finite)
                    rl = ppo_row(load_elem(x_row + rec.y) - M, log_s, rec.old_logp, rec.adv,
                                 a.eps_low, a.eps_high, inv_denom);
                else
                    atomicOr(a.stats + 3, TPPO_DEV_NONFINITE);
                if (a.logp) a.logp[j] = rl.logp;
                if (a.token_loss) a.token_loss[j] = rl.loss;
                a.row_loss[j] = rl.loss;
                a.row_clip[j] = uint8_t(rl.clip);
                s_max = M;
                s_logsum = log_s;
                s_coef = rl.coef;
            }
            __syncthreads();
            coef = s_coef;
            row_max = s_max;
            log_sum = s_logsum;
        } else if (tid == 0) {
            if (a.logp) a.logp[j] = 0.f;
            if (a.token_loss) a.token_loss[j] = 0.f;
            a.row_loss[j] = 0.f;
            a.row_clip[j] = 0;
        }

        // ---- pass 2 -----------------------------------------------------------------------
        if (g_row) {
            const float off = log_sum * kLog2e;   // exponent of softmax_v = (x_v - max)*log2e - off
            if (coef == 0.f) {   // clipped, zero advantage or invalid entry: the gradient row is zero
                if (VEC) {
                    const int nu = a.V >> 3;
                    const float z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                    for (int u = tid; u < nu; u += kTwoPassThreads) store8(g_row + (int64_t(u) << 3), z);
                    for (int v = (nu << 3) + tid; v < a.V; v += kTwoPassThreads) store_elem(g_row + v, 0.f);
                } else {
                    for (int v = tid; v < a.V; v += kTwoPassThreads) store_elem(g_row + v, 0.f);
                }
            } else if (VEC) {
                const int nu = a.V >> 3;
                const int yu = rec.y >> 3, yk = rec.y & 7;
                constexpr int kDeep = 4;
                int u = tid;
                for (; u + (kDeep - 1) * kTwoPassThreads < nu; u += kDeep * kTwoPassThreads) {
                    RawUnit<T> raw[kDeep];
#pragma unroll
                    for (int d = 0; d < kDeep; ++d) raw[d] = load_raw(x_row + (int64_t(u + d * kTwoPassThreads) << 3));
#pragma unroll
                    for (int d = 0; d < kDeep; ++d) {
                        const int ud = u + d * kTwoPassThreads;
                        float x[8], g[8];
                        widen8(raw[d], x);
#pragma unroll
                        for (int k = 0; k < 8; ++k) g[k] = coef * ex2(fmaf(x[k] - row_max, kLog2e, -off));
                        if (ud == yu) {
#pragma unroll
                            for (int k = 0; k < 8; ++k) if (k == yk) g[k] -= coef;
                        }
                        store8(g_row + (int64_t(ud) << 3), g);
                    }
                }
                for (; u < nu; u += kTwoPassThreads) {
                    float x[8], g[8];
                    load8(x_row + (int64_t(u) << 3), x);
#pragma unroll
                    for (int k = 0; k < 8; ++k) g[k] = coef * ex2(fmaf(x[k] - row_max, kLog2e, -off));
                    if (u == yu) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) if (k == yk) g[k] -= coef;
                    }
                    store8(g_row + (int64_t(u) << 3), g);
                }
                for (int v = (nu << 3) + tid; v < a.V; v += kTwoPassThreads) {
                    float g = coef * ex2(fmaf(load_elem(x_row + v) - row_max, kLog2e, -off));
                    if (v == rec.y) g -= coef;
                    store_elem(g_row + v, g);
                }
            } else {
                for (int v = tid; v < a.V; v += kTwoPassThreads) {
                    float g = coef * ex2(fmaf(load_elem(x_row + v) - row_max, kLog2e, -off));
                    if (v == rec.y) g -= coef;
                    store_elem(g_row + v, g);
                }
            }
        }
        __syncthreads();   // the shared row scalars are reused by the next row
    }
    // Launched beside the cluster kernel (as its programmatic dependent) this grid must not be
    // complete before that one is: whatever follows in the stream waits for this grid only.
    if (a.part == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// variant: blocks per SM (0 = default 3).  side_sms > 0: launch as a programmatic dependent of the
// kernel before it in the stream, sized for that many SMs (the ones the cluster kernel leaves idle).
int launch_policy_two_pass(const PolicyArgs& a, int dtype, cudaStream_t s, int variant, int side_sms) {
    const int per_sm = (variant & 15) ? (variant & 15) : 3;
    int64_t blocks = a.n_max < 1 ? 1 : a.n_max;
    const int sms = side_sms > 0 ? side_sms : kNumSms;
    if (blocks > sms * per_sm) blocks = sms * per_sm;
    const size_t esz = dtype == TPPO_BF16 ? 2 : 4;
    bool vec = aligned(a.logits, 16) && (a.ld * esz) % 16 == 0;
    if (a.mode == TPPO_DLOGITS_FULL) vec = vec && aligned(a.dlogits, 16);
    if (a.mode == TPPO_DLOGITS_COMPACT)
        vec = vec && aligned(a.dlogits, 16) && (int64_t(a.V) * esz) % 16 == 0;
    void (*kern)(const PolicyArgs) = nullptr;
    if (dtype == TPPO_BF16) kern = vec ? policy_two_pass_kernel<TPPO_BF16, true> : policy_two_pass_kernel<TPPO_BF16, false>;
    else kern = vec ? policy_two_pass_kernel<TPPO_F32, true> : policy_two_pass_kernel<TPPO_F32, false>;
    cudaLaunchConfig_t lc = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.gridDim = dim3(unsigned(blocks), 1, 1);
    lc.blockDim = dim3(kTwoPassThreads, 1, 1);
    lc.dynamicSmemBytes = 0;
    lc.stream = s;
    lc.attrs = attr;
    lc.numAttrs = side_sms > 0 ? 1 : 0;
    return cudaLaunchKernelEx(&lc, kern, a) == cudaSuccess ? TPPO_OK : TPPO_ERR_CUDA;
}

}  // namespace tppo

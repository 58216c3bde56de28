// EGAE advantages and Monte-Carlo returns (Section 3.1, Eq. 6 with the TD residual of Eq. 3; R_t
// after Eq. 5) as ONE segmented reverse scan over the packed token arrays.
//
// Both recurrences are affine in the value at the next position,
//     A_t = delta_t + (gamma*lambda) * A_{t+1},      R_t = r_t + gamma * R_{t+1},
// so every position carries a map x -> a*x + b, with a = 0 on the last token of a segment and
// outside every segment.  Maps compose associatively; a tile composes its positions right to
// left, publishes the composite, and obtains the value entering from its right-hand neighbour by
// decoupled look-back over the tiles behind it.  A composite whose `a` has become 0 (a segment
// ended inside the range) ends the look-back early.  State is fp64, rounded once on store.
#include "common.cuh"

namespace tppo {

constexpr int kScanThreads = 256;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;  // 2048 positions
constexpr uint32_t kScanSpinLimit = 1u << 22;

struct Affine2 {  // x -> (aA*xA + bA, aR*xR + bR)
    double aA, bA, aR, bR;
};
__device__ __forceinline__ Affine2 identity2() { return Affine2{1.0, 0.0, 1.0, 0.0}; }
// (f o g)(x) = f(g(x))
__device__ __forceinline__ Affine2 compose(const Affine2& f, const Affine2& g) {
    return Affine2{f.aA * g.aA, fma(f.aA, g.bA, f.bA), f.aR * g.aR, fma(f.aR, g.bR, f.bR)};
}
__device__ __forceinline__ Affine2 shfl_down(const Affine2& f, int d) {
    return Affine2{__shfl_down_sync(0xffffffffu, f.aA, d), __shfl_down_sync(0xffffffffu, f.bA, d),
                   __shfl_down_sync(0xffffffffu, f.aR, d), __shfl_down_sync(0xffffffffu, f.bR, d)};
}

struct TileState {     // one per tile, 64 bytes
    double agg[4];     // composite of the tile (valid when flag >= 1)
    double inc[2];     // A and R at the tile's first position (valid when flag == 2)
    int flag;
    int pad[3];
};

struct EgaeArgs {
    const float* rewards;
    const float* values;
    const int32_t* seg_begin;
    const int32_t* seg_end;
    const uint8_t* truncated;
    const float* bootstrap;
    int32_t B;
    int32_t N;
    int32_t num_tiles;
    double gamma;
    double gl;  // gamma * lambda
    float* adv;
    float* ret;
    int32_t* status;
    TileState* state;
    uint32_t* ticket;
};

// number of entries of arr[0..n) that are <= key
__device__ __forceinline__ int seg_count_le(const int32_t* __restrict__ arr, int n, int32_t key) {
    int lo = 0, hi = n;
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (__ldg(arr + mid) <= key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(kScanThreads) egae_scan_kernel(const EgaeArgs a) {
    __shared__ uint32_t s_ticket;
    __shared__ Affine2 s_warp[kScanWarps];
    __shared__ double s_carry[kScanWarps][2];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_ticket = atomicAdd(a.ticket, 1u);
    __syncthreads();
    if (s_ticket >= uint32_t(a.num_tiles)) return;
    // Tickets go to tiles from the END of the arrays backwards, so the tiles this one looks back
    // at (those to its right) already hold earlier tickets and are running or done.
    const int tile = a.num_tiles - 1 - int(s_ticket);
    const int64_t base = int64_t(tile) * kScanTile + int64_t(threadIdx.x) * kScanItems;

    // ---- per-position maps, right to left -------------------------------------------------
    double delta[kScanItems], rew[kScanItems];
    uint32_t cont = 0;  // bit k: position k continues into position k+1 (same segment)
    Affine2 f = identity2();
    {
        const int64_t p_last = min(base + kScanItems, int64_t(a.N)) - 1;
        int i = (p_last >= base) ? seg_count_le(a.seg_begin, a.B, int32_t(p_last)) - 1 : -1;
        bool bad = false;
#pragma unroll
        for (int k = kScanItems - 1; k >= 0; --k) {
            const int64_t p = base + k;
            delta[k] = 0.0;
            rew[k] = 0.0;
            if (p >= a.N) continue;   // past the end: the identity map
            while (i >= 0 && int32_t(p) < __ldg(a.seg_begin + i)) --i;
            bool inside = false;
            int64_t e = 0;
            if (i >= 0) {
                const int64_t b = __ldg(a.seg_begin + i);
                e = __ldg(a.seg_end + i);
                if (b < 0 || e > a.N || e < b) { bad = true; e = b; }
                inside = p < e;
            }
            double aA = 0.0, aR = 0.0;
            if (inside) {
                const double r = double(__ldg(a.rewards + p));
                const double v = double(__ldg(a.values + p));
                double v_next;
                if (p + 1 < e) {
                    v_next = double(__ldg(a.values + p + 1));
                    aA = a.gl;
                    aR = a.gamma;
                    cont |= 1u << k;
                } else if (__ldg(a.truncated + i)) {
                    v_next = a.bootstrap ? double(__ldg(a.bootstrap + i)) : v;
                } else {
                    v_next = 0.0;
                }
                delta[k] = fma(a.gamma, v_next, r) - v;
                rew[k] = r;
            }
            f = compose(Affine2{aA, delta[k], aR, rew[k]}, f);
        }
        if (bad) atomicOr(a.status, TPPO_DEV_BAD_SEGMENT);
    }

    // ---- inclusive suffix composition inside the warp: S_l = f_l o f_{l+1} o ... o f_31 -------
    Affine2 S = f;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const Affine2 o = shfl_down(S, d);
        if (lane + d < 32) S = compose(S, o);
    }
    Affine2 excl = shfl_down(S, 1);   // composite of the lanes to the right
    if (lane == 31) excl = identity2();
    if (lane == 0) s_warp[warp] = S;
    __syncthreads();

    // ---- tile composite, look-back, per-warp carries --------------------------------------
    if (threadIdx.x == 0) {
        Affine2 right[kScanWarps];      // right[w]: composite of warps w+1 .. last
        Affine2 acc = identity2();
        for (int w = kScanWarps - 1; w >= 0; --w) {
            right[w] = acc;
            acc = compose(s_warp[w], acc);
        }
        const Affine2 tile_f = acc;
        TileState* st = a.state;
        if (tile + 1 < a.num_tiles) {
            st[tile].agg[0] = tile_f.aA; st[tile].agg[1] = tile_f.bA;
            st[tile].agg[2] = tile_f.aR; st[tile].agg[3] = tile_f.bR;
            __threadfence();
            *reinterpret_cast<volatile int*>(&st[tile].flag) = 1;
        }
        // value entering from the right: look back over tiles tile+1, tile+2, ...
        Affine2 F = identity2();
        double xA = 0.0, xR = 0.0;
        bool timed_out = false;
        for (int j = tile + 1;; ++j) {
            if (j >= a.num_tiles) { xA = F.bA; xR = F.bR; break; }   // nothing beyond the end
            volatile int* fl = reinterpret_cast<volatile int*>(&st[j].flag);
            int flag = *fl;
            uint32_t spins = 0;
            while (flag == 0) {
                if (++spins > kScanSpinLimit) { timed_out = true; break; }
                __nanosleep(20);
                flag = *fl;
            }
            if (timed_out) break;
            __threadfence();
            const volatile double* pd = reinterpret_cast<const volatile double*>(&st[j]);
            if (flag == 2) {
                xA = fma(F.aA, pd[4], F.bA);
                xR = fma(F.aR, pd[5], F.bR);
                break;
            }
            F = compose(F, Affine2{pd[0], pd[1], pd[2], pd[3]});
            if (F.aA == 0.0 && F.aR == 0.0) { xA = F.bA; xR = F.bR; break; }  // a segment ended
        }
        if (timed_out) { atomicOr(a.status, TPPO_DEV_WAIT_TIMEOUT); xA = 0.0; xR = 0.0; }
        st[tile].inc[0] = fma(tile_f.aA, xA, tile_f.bA);
        st[tile].inc[1] = fma(tile_f.aR, xR, tile_f.bR);
        __threadfence();
        *reinterpret_cast<volatile int*>(&st[tile].flag) = 2;
        for (int w = 0; w < kScanWarps; ++w) {
            s_carry[w][0] = fma(right[w].aA, xA, right[w].bA);
            s_carry[w][1] = fma(right[w].aR, xR, right[w].bR);
        }
    }
    __syncthreads();

    // ---- replay the thread's positions with the true incoming values ------------------------
    double A = fma(excl.aA, s_carry[warp][0], excl.bA);
    double G = fma(excl.aR, s_carry[warp][1], excl.bR);
#pragma unroll
    for (int k = kScanItems - 1; k >= 0; --k) {
        const int64_t p = base + k;
        if (p >= a.N) continue;
        const bool c = (cont >> k) & 1u;
        A = c ? fma(a.gl, A, delta[k]) : delta[k];
        G = c ? fma(a.gamma, G, rew[k]) : rew[k];
        a.adv[p] = float(A);
        if (a.ret) a.ret[p] = float(G);
    }
}

size_t egae_workspace_bytes(int64_t N) {
    const int64_t tiles = (N + kScanTile - 1) / kScanTile;
    return align_up(sizeof(uint32_t), kWsAlign) +
           align_up(size_t(tiles > 0 ? tiles : 1) * sizeof(TileState), kWsAlign);
}

}  // namespace tppo

using namespace tppo;

TPPO_API int tppo_egae(const float* rewards, const float* values, const int32_t* seg_begin,
                       const int32_t* seg_end, const uint8_t* truncated, const float* bootstrap,
                       int32_t B, int64_t N, float gamma, float lambda, float* advantages,
                       float* returns, int32_t* status, void* workspace, size_t workspace_bytes,
                       void* stream) {
    if (B < 0 || N < 0 || N >= (int64_t(1) << 31) || !status) return TPPO_ERR_INVALID_ARG;
    if (N > 0 && (!rewards || !values || !advantages)) return TPPO_ERR_INVALID_ARG;
    if (B > 0 && (!seg_begin || !seg_end || !truncated)) return TPPO_ERR_INVALID_ARG;
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f))
        return TPPO_ERR_INVALID_ARG;
    const size_t need = egae_workspace_bytes(N);
    if (!workspace || workspace_bytes < need || !aligned(workspace, kWsAlign))
        return TPPO_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TPPO_CUDA_CHECK(cudaMemsetAsync(status, 0, sizeof(int32_t), s));
    if (N == 0) return TPPO_OK;
    TPPO_CUDA_CHECK(cudaMemsetAsync(workspace, 0, need, s));
    EgaeArgs a;
    a.rewards = rewards; a.values = values; a.seg_begin = seg_begin; a.seg_end = seg_end;
    a.truncated = truncated; a.bootstrap = bootstrap; a.B = B; a.N = int32_t(N);
    a.num_tiles = int32_t((N + kScanTile - 1) / kScanTile);
    a.gamma = double(gamma);
    a.gl = double(gamma) * double(lambda);
    a.adv = advantages; a.ret = returns; a.status = status;
    a.ticket = static_cast<uint32_t*>(workspace);
    a.state = reinterpret_cast<TileState*>(static_cast<char*>(workspace) +
                                           align_up(sizeof(uint32_t), kWsAlign));
    egae_scan_kernel<<<a.num_tiles, kScanThreads, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

// ---- allocation-free variant ------------------------------------------------------------------
// For callers that can neither allocate device memory nor lend a workspace (a plug-in inside a
// runtime that owns the whole device's memory pool; a latency-critical section that must avoid
// cudaMalloc's device-wide synchronisation).  The tile descriptors and the ticket counter live in
// this fixed device array; each GPU that loads the library keeps it until the process ends.
namespace tppo {
constexpr int64_t kStaticMaxTokens = TPPO_EGAE_STATIC_MAX_TOKENS;
constexpr size_t kStaticTiles = size_t((kStaticMaxTokens + kScanTile - 1) / kScanTile);
constexpr size_t kStaticScratchBytes = 256 + kStaticTiles * sizeof(TileState);
static_assert(sizeof(TileState) == 64, "tile descriptor is 64 bytes");
}  // namespace tppo

static __device__ __align__(256) unsigned char g_egae_static_scratch[tppo::kStaticScratchBytes];

namespace tppo {
constexpr int kMaxDevices = 64;
// Device address of g_egae_static_scratch per device ordinal.  In host code the array's name is
// only a handle for the runtime, never a device address: the address comes from
// cudaGetSymbolAddress, asked once per device with that device current.
static void* g_static_scratch_addr[kMaxDevices] = {};

static int static_scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TPPO_ERR_CUDA;
    void* p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_egae_static_scratch) != cudaSuccess || !p) return TPPO_ERR_CUDA;
        __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);   // same value from any thread
    }
    *out = p;
    return TPPO_OK;
}
}  // namespace tppo

TPPO_API int tppo_egae_static(const float* rewards, const float* values, const int32_t* seg_begin,
                              const int32_t* seg_end, const uint8_t* truncated,
                              const float* bootstrap, int32_t B, int64_t N, float gamma,
                              float lambda, float* advantages, float* returns, int32_t* status,
                              void* stream) {
    if (B < 0 || N < 0 || !status) return TPPO_ERR_INVALID_ARG;
    if (N > kStaticMaxTokens) return TPPO_ERR_TOO_LARGE;
    if (N > 0 && (!rewards || !values || !advantages)) return TPPO_ERR_INVALID_ARG;
    if (B > 0 && (!seg_begin || !seg_end || !truncated)) return TPPO_ERR_INVALID_ARG;
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f))
        return TPPO_ERR_INVALID_ARG;
    void* scratch = nullptr;
    const int rc = static_scratch_for_current_device(&scratch);
    if (rc != TPPO_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TPPO_CUDA_CHECK(cudaMemsetAsync(status, 0, sizeof(int32_t), s));
    if (N == 0) return TPPO_OK;
    EgaeArgs a;
    a.rewards = rewards; a.values = values; a.seg_begin = seg_begin; a.seg_end = seg_end;
    a.truncated = truncated; a.bootstrap = bootstrap; a.B = B; a.N = int32_t(N);
    a.num_tiles = int32_t((N + kScanTile - 1) / kScanTile);
    a.gamma = double(gamma);
    a.gl = double(gamma) * double(lambda);
    a.adv = advantages; a.ret = returns; a.status = status;
    a.ticket = static_cast<uint32_t*>(scratch);
    a.state = reinterpret_cast<TileState*>(static_cast<char*>(scratch) + 256);
    // the array still holds the previous call's flags and ticket: clear the part this call uses
    TPPO_CUDA_CHECK(cudaMemsetAsync(scratch, 0, 256 + size_t(a.num_tiles) * sizeof(TileState), s));
    egae_scan_kernel<<<a.num_tiles, kScanThreads, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

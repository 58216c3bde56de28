// Token filter + stream compaction (Section 3.2 of the paper): one pass over the packed token
// positions, warp-ballot ranks inside a warp, shared-memory prefix across the warps of a tile,
// and a decoupled look-back chain across tiles, so that every selected position is written once
// in ascending order.  Integer work throughout: the result is bit-exact and run-to-run identical.
#include "common.cuh"

namespace tppo {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelItems = 16;                                  // positions per lane
constexpr int kSelTile = kSelThreads * kSelItems;              // 4096 positions per tile
constexpr uint32_t kSelSpinLimit = 1u << 22;

// tile state word: [63:62] flag (1 = tile total, 2 = inclusive prefix), [61:31] policy count,
// [30:0] value count.  One 64-bit store publishes flag and payload together.
__device__ __forceinline__ uint64_t sel_pack(uint32_t flag, uint32_t pol, uint32_t val) {
    return (uint64_t(flag) << 62) | (uint64_t(pol) << 31) | uint64_t(val);
}
__device__ __forceinline__ uint32_t sel_flag(uint64_t s) { return uint32_t(s >> 62); }
__device__ __forceinline__ uint32_t sel_pol(uint64_t s) { return uint32_t(s >> 31) & 0x7fffffffu; }
__device__ __forceinline__ uint32_t sel_val(uint64_t s) { return uint32_t(s) & 0x7fffffffu; }

// Number of entries of the ascending array arr[0..n) that are <= key, found by a whole warp: each
// round probes 32 evenly spaced entries (one load per lane) and narrows the range 32-fold.  Every
// lane returns the same count; an array that is not ascending still yields an in-range answer.
__device__ __forceinline__ int warp_count_le(const int32_t* __restrict__ arr, int n, int32_t key,
                                             int lane) {
    int lo = 0, hi = n;       // the answer lies in [lo, hi]
    while (lo < hi) {
        const int span = hi - lo;
        const int step = (span + 31) >> 5;
        const int idx = lo + lane * step;
        const bool le = idx < hi && __ldg(arr + idx) <= key;
        const uint32_t m = __ballot_sync(0xffffffffu, le);
        const int c = __ffs(int(~m)) - 1;          // leading run of probes that are <= key
        if (c < 0) { lo = min(lo + 31 * step + 1, hi); continue; }
        const int new_hi = min(lo + c * step, hi);
        if (c > 0) lo = lo + (c - 1) * step + 1;
        hi = new_hi;
    }
    return lo;
}

struct SelectArgs {
    const int32_t* seq_begin;
    const int32_t* prompt_len;
    const int32_t* prev_len;
    const int32_t* new_len;
    const uint8_t* truncated;
    const uint8_t* pol_mask;
    const uint8_t* val_mask;
    int32_t tail_drop;
    int32_t B;
    int32_t N;
    int32_t num_tiles;
    int32_t mask_vec_ok;        // both masks (where given) are 16-byte aligned
    int32_t* policy_idx;
    int32_t* value_idx;
    int32_t* counts;            // [4]
    unsigned long long* state;  // [num_tiles]
    uint32_t* ticket;           // [1]
};

// Position ranges of one sequence: policy tokens [pol_lo, pol_hi), value tokens [val_lo, val_hi),
// and the first position of the next sequence.
struct SeqBounds {
    int64_t next, pol_lo, pol_hi, val_lo, val_hi;
};
__device__ __forceinline__ SeqBounds seq_bounds(const SelectArgs& a, int i) {
    SeqBounds s;
    if (i < 0 || i >= a.B) {        // before the first or after the last sequence: nothing selected
        s.next = i < 0 ? int64_t(__ldg(a.seq_begin)) : (int64_t(1) << 40);
        s.pol_lo = s.pol_hi = s.val_lo = s.val_hi = 0;
        return s;
    }
    const int64_t begin = __ldg(a.seq_begin + i);
    s.next = __ldg(a.seq_begin + i + 1);
    const int64_t resp0 = begin + __ldg(a.prompt_len + i);
    const int64_t new0 = resp0 + __ldg(a.prev_len + i);
    const int64_t end = new0 + __ldg(a.new_len + i);
    const bool trunc = __ldg(a.truncated + i) != 0;
    s.pol_lo = new0;
    s.pol_hi = end - (trunc ? a.tail_drop : 0);
    s.val_lo = resp0;
    s.val_hi = trunc ? resp0 : end;
    return s;
}

__global__ void __launch_bounds__(kSelThreads) select_tokens_kernel(const SelectArgs a) {
    __shared__ __align__(16) uint8_t s_pm[kSelTile];
    __shared__ __align__(16) uint8_t s_vm[kSelTile];
    __shared__ uint32_t s_tile;
    __shared__ int s_seq0;
    __shared__ uint32_t s_warp_pol[kSelWarps], s_warp_val[kSelWarps];
    __shared__ uint32_t s_base_pol, s_base_val;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // Tiles are handed out in launch order, so every tile this one waits for is already running.
    if (threadIdx.x == 0) s_tile = atomicAdd(a.ticket, 1u);
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= uint32_t(a.num_tiles)) return;
    const int64_t t0 = int64_t(tile) * kSelTile;
    const int n_tile = int(min(int64_t(kSelTile), int64_t(a.N) - t0));

    // ---- stage the optional byte masks (one 16-byte load per thread and mask) ------------------
    {
        const int l = threadIdx.x * 16;
        if (a.mask_vec_ok && l + 16 <= n_tile) {
            if (a.pol_mask)
                reinterpret_cast<uint4*>(s_pm)[threadIdx.x] =
                    __ldg(reinterpret_cast<const uint4*>(a.pol_mask + t0) + threadIdx.x);
            if (a.val_mask)
                reinterpret_cast<uint4*>(s_vm)[threadIdx.x] =
                    __ldg(reinterpret_cast<const uint4*>(a.val_mask + t0) + threadIdx.x);
        } else {
            for (int k = l; k < min(l + 16, n_tile); ++k) {
                if (a.pol_mask) s_pm[k] = __ldg(a.pol_mask + t0 + k);
                if (a.val_mask) s_vm[k] = __ldg(a.val_mask + t0 + k);
            }
        }
    }
    // sequence that holds the tile's first position (-1: before the first sequence)
    if (warp == 0) {
        const int c = warp_count_le(a.seq_begin, a.B + 1, int32_t(t0), lane);
        if (lane == 0) s_seq0 = c - 1;
    }
    __syncthreads();

    // ---- phase 1: predicates, kept as one bit per item in two 16-bit lane masks ------------
    const int warp_l0 = warp * (32 * kSelItems);
    uint32_t pol_bits = 0, val_bits = 0;
    {
        int i = s_seq0;
        SeqBounds sb = seq_bounds(a, i);
#pragma unroll 4
        for (int j = 0; j < kSelItems; ++j) {
            const int l = warp_l0 + lane + j * 32;
            if (l >= n_tile) break;
            const int64_t p = t0 + l;
            while (i < a.B && p >= sb.next) sb = seq_bounds(a, ++i);
            bool is_pol = p >= sb.pol_lo && p < sb.pol_hi;
            bool is_val = p >= sb.val_lo && p < sb.val_hi;
            if (is_pol && a.pol_mask) is_pol = s_pm[l] != 0;
            if (is_val && a.val_mask) is_val = s_vm[l] != 0;
            pol_bits |= uint32_t(is_pol) << j;
            val_bits |= uint32_t(is_val) << j;
        }
    }
    uint32_t warp_pol = 0, warp_val = 0;
#pragma unroll
    for (int j = 0; j < kSelItems; ++j) {
        warp_pol += __popc(__ballot_sync(0xffffffffu, (pol_bits >> j) & 1u));
        warp_val += __popc(__ballot_sync(0xffffffffu, (val_bits >> j) & 1u));
    }
    if (lane == 0) { s_warp_pol[warp] = warp_pol; s_warp_val[warp] = warp_val; }
    __syncthreads();

    // ---- tile total -> publish -> warp-wide look-back over earlier tiles ----------------------
    if (warp == 0) {
        uint32_t tp = 0, tv = 0;
        for (int w = 0; w < kSelWarps; ++w) { tp += s_warp_pol[w]; tv += s_warp_val[w]; }
        volatile unsigned long long* st = a.state;
        if (lane == 0 && tile > 0) st[tile] = sel_pack(1, tp, tv);
        uint32_t ep = 0, ev = 0;
        bool timed_out = false;
        // 32 predecessors per round: lane l looks at tile j0 - l; positions before tile 0 count as
        // an inclusive prefix of zero.  The nearest inclusive prefix ends the walk.
        for (int64_t j0 = int64_t(tile) - 1; j0 >= 0; j0 -= 32) {
            const int64_t j = j0 - lane;
            uint64_t s = j >= 0 ? st[j] : sel_pack(2, 0, 0);
            uint32_t spins = 0;
            while (!__all_sync(0xffffffffu, sel_flag(s) != 0)) {
                if (++spins > kSelSpinLimit) { timed_out = true; break; }
                __nanosleep(20);
                if (sel_flag(s) == 0) s = st[j];
            }
            if (timed_out) break;
            const uint32_t m2 = __ballot_sync(0xffffffffu, sel_flag(s) == 2);
            const int first2 = m2 ? __ffs(int(m2)) - 1 : 32;
            const bool use = lane <= first2;
            ep += __reduce_add_sync(0xffffffffu, use ? sel_pol(s) : 0u);
            ev += __reduce_add_sync(0xffffffffu, use ? sel_val(s) : 0u);
            if (m2) break;
        }
        if (lane == 0) {
            if (timed_out) atomicOr(a.counts + 2, TPPO_DEV_WAIT_TIMEOUT);
            st[tile] = sel_pack(2, ep + tp, ev + tv);
            s_base_pol = ep;
            s_base_val = ev;
            if (tile == uint32_t(a.num_tiles) - 1) {
                a.counts[0] = int32_t(ep + tp);
                a.counts[1] = int32_t(ev + tv);
            }
        }
    }
    __syncthreads();

    // ---- phase 2: scatter --------------------------------------------------------------------
    uint32_t off_pol = s_base_pol, off_val = s_base_val;
    for (int w = 0; w < warp; ++w) { off_pol += s_warp_pol[w]; off_val += s_warp_val[w]; }
    const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
    for (int j = 0; j < kSelItems; ++j) {
        const int32_t p = int32_t(t0 + warp_l0 + lane + j * 32);
        const uint32_t bp = __ballot_sync(0xffffffffu, (pol_bits >> j) & 1u);
        const uint32_t bv = __ballot_sync(0xffffffffu, (val_bits >> j) & 1u);
        if ((pol_bits >> j) & 1u) a.policy_idx[off_pol + __popc(bp & lt)] = p;
        if ((val_bits >> j) & 1u) a.value_idx[off_val + __popc(bv & lt)] = p;
        off_pol += __popc(bp);
        off_val += __popc(bv);
    }
}

size_t select_workspace_bytes(int64_t N) {
    const int64_t tiles = (N + kSelTile - 1) / kSelTile;
    return align_up(sizeof(uint32_t), kWsAlign) + align_up(size_t(tiles > 0 ? tiles : 1) * 8, kWsAlign);
}

}  // namespace tppo

using namespace tppo;

TPPO_API int tppo_select_tokens(const int32_t* seq_begin, const int32_t* prompt_len,
                                const int32_t* prev_len, const int32_t* new_len,
                                const uint8_t* truncated, int32_t tail_drop,
                                const uint8_t* extra_policy_mask, const uint8_t* extra_value_mask,
                                int32_t B, int64_t N, int32_t* policy_idx, int32_t* value_idx,
                                int32_t* counts, void* workspace, size_t workspace_bytes,
                                void* stream) {
    if (B < 0 || N < 0 || N >= (int64_t(1) << 31) || tail_drop < 0 || !counts)
        return TPPO_ERR_INVALID_ARG;
    if (B > 0 && (!seq_begin || !prompt_len || !prev_len || !new_len || !truncated))
        return TPPO_ERR_INVALID_ARG;
    if (N > 0 && (!policy_idx || !value_idx)) return TPPO_ERR_INVALID_ARG;
    const size_t need = select_workspace_bytes(N);
    if (!workspace || workspace_bytes < need || !aligned(workspace, kWsAlign))
        return TPPO_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TPPO_CUDA_CHECK(cudaMemsetAsync(counts, 0, 4 * sizeof(int32_t), s));
    if (N == 0 || B == 0) return TPPO_OK;
    TPPO_CUDA_CHECK(cudaMemsetAsync(workspace, 0, need, s));
    SelectArgs a;
    a.seq_begin = seq_begin; a.prompt_len = prompt_len; a.prev_len = prev_len; a.new_len = new_len;
    a.truncated = truncated; a.pol_mask = extra_policy_mask; a.val_mask = extra_value_mask;
    a.tail_drop = tail_drop; a.B = B; a.N = int32_t(N);
    a.mask_vec_ok = (!extra_policy_mask || aligned(extra_policy_mask, 16)) &&
                    (!extra_value_mask || aligned(extra_value_mask, 16));
    a.num_tiles = int32_t((N + kSelTile - 1) / kSelTile);
    a.policy_idx = policy_idx; a.value_idx = value_idx; a.counts = counts;
    a.ticket = static_cast<uint32_t*>(workspace);
    a.state = reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) +
                                                    align_up(sizeof(uint32_t), kWsAlign));
    select_tokens_kernel<<<a.num_tiles, kSelThreads, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

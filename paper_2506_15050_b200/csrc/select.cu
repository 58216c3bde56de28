// Token filter + stream compaction (Section 3.2 of the paper): one pass over the packed token
// positions.  A thread turns its 32 consecutive positions into two 32-bit words by interval
// arithmetic on the sequences that overlap them, ranks come from popcounts and a warp / tile
// prefix, a decoupled look-back chain links the tiles, and every selected position is written once
// in ascending order.  Integer work throughout: the result is bit-exact and run-to-run identical.
#include <algorithm>
#include "common.cuh"
#include "ptx.cuh"

namespace tppo {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelItems = 32;                                  // positions per thread
constexpr int kSelTile = kSelThreads * kSelItems;              // 8192 positions per tile
constexpr uint32_t kSelSpinLimit = 1u << 22;
// Tile order.  0 (default): block b takes tile b; thread blocks are dispatched in index order, so the
// tiles a tile waits for (smaller indices) are running or done, and should that ever not hold the
// bounded wait gives up with TPPO_DEV_WAIT_TIMEOUT instead of hanging.  1: tiles are drawn from an
// atomic ticket counter, which needs no assumption about dispatch order (measured 6 us slower at
// 17.5 M positions: an L2 round trip at the head of every tile's chain of latencies).
#ifndef TPPO_SEL_TICKET
#define TPPO_SEL_TICKET 0
#endif

// tile state word: [63:62] flag (1 = tile total, 2 = inclusive prefix), [61:31] policy count,
// [30:0] value count.  One 64-bit store publishes flag and payload together.
__device__ __forceinline__ uint64_t sel_pack(uint32_t flag, uint32_t pol, uint32_t val) {
    return (uint64_t(flag) << 62) | (uint64_t(pol) << 31) | uint64_t(val);
}
__device__ __forceinline__ uint32_t sel_flag(uint64_t s) { return uint32_t(s >> 62); }
__device__ __forceinline__ uint32_t sel_pol(uint64_t s) { return uint32_t(s >> 31) & 0x7fffffffu; }
__device__ __forceinline__ uint32_t sel_val(uint64_t s) { return uint32_t(s) & 0x7fffffffu; }

struct SelectArgs {
    const int32_t* seq_begin;
    const int32_t* prompt_len;
    const int32_t* prev_len;
    const int32_t* new_len;
    const uint8_t* truncated;
    const uint8_t* pol_mask;
    const uint8_t* val_mask;
    int32_t tail_drop;
    const int32_t* tail_drop_seq;   // [B] or null: per-sequence count, overrides tail_drop
    int32_t B;
    int32_t N;
    int32_t num_tiles;
    int32_t mask_vec_ok;        // both masks (where given) are 16-byte aligned
    int32_t* policy_idx;
    int32_t* value_idx;
    int32_t* counts;            // [4]
    unsigned long long* state;  // [num_tiles]
    const int2* window;         // [num_tiles]: (seq0, seq1) of every tile, found by the clearing kernel
    uint32_t* ticket;           // head of the workspace, cleared to zero together with the tile states
    uint32_t spin_limit;        // polls a look-back round may take before it gives up
    int32_t no_publish;         // test hook: tiles keep their totals to themselves
    int32_t out_vec_ok;         // policy_idx and value_idx are 16-byte aligned
};

constexpr int kSeqCap = 640;   // sequence starts of one tile kept in shared memory

// 16 mask bytes -> 16 bits (bit k set iff byte k is non-zero).
__device__ __forceinline__ uint32_t nonzero_bytes4(uint32_t w) {
    // high bit of each byte set iff the byte is non-zero, then the four high bits gathered
    const uint32_t t = (w | ((w & 0x7f7f7f7fu) + 0x7f7f7f7fu)) & 0x80808080u;
    return ((t >> 7) * 0x00204081u >> 21) & 0xfu;
}
__device__ __forceinline__ uint32_t nonzero_bytes16(uint4 v) {
    return nonzero_bytes4(v.x) | (nonzero_bytes4(v.y) << 4) | (nonzero_bytes4(v.z) << 8) |
           (nonzero_bytes4(v.w) << 12);
}
// Bits [lo - p0, hi - p0) of a 32-bit word, for the positions of [lo, hi) that fall in [p0, p0+32).
__device__ __forceinline__ uint32_t range_bits32(int64_t lo, int64_t hi, int64_t p0) {
    const int64_t a = min(max(lo - p0, int64_t(0)), int64_t(32));
    const int64_t b = min(max(hi - p0, int64_t(0)), int64_t(32));
    if (b <= a) return 0u;                                       // then a < 32
    const uint32_t upto_b = b >= 32 ? 0xffffffffu : ((1u << int(b)) - 1u);
    return upto_b & ~((1u << int(a)) - 1u);
}

// One of the tile's two lists from shared memory (16-bit offsets inside the tile) to its place in
// the output array: 16-byte stores of four indices where the destination allows, single stores at
// the ragged ends.
__device__ __forceinline__ void sel_copy_out(int32_t* __restrict__ out, uint32_t base, int n,
                                             const uint16_t* __restrict__ src, int32_t t0, bool vec) {
    int32_t* dst = out + base;
    if (!vec) {
        for (int k = threadIdx.x; k < n; k += kSelThreads) dst[k] = t0 + int32_t(src[k]);
        return;
    }
    const int head = min(n, int((4u - (base & 3u)) & 3u));       // entries before the first 16-byte boundary
    const int groups = (n - head) >> 2;
    if (int(threadIdx.x) < head) dst[threadIdx.x] = t0 + int32_t(src[threadIdx.x]);
    for (int g = threadIdx.x; g < groups; g += kSelThreads) {
        const int k = head + 4 * g;
        int4 v;
        v.x = t0 + int32_t(src[k]);
        v.y = t0 + int32_t(src[k + 1]);
        v.z = t0 + int32_t(src[k + 2]);
        v.w = t0 + int32_t(src[k + 3]);
        *reinterpret_cast<int4*>(dst + k) = v;
    }
    const int tail0 = head + 4 * groups;
    if (int(threadIdx.x) < n - tail0) dst[tail0 + threadIdx.x] = t0 + int32_t(src[tail0 + threadIdx.x]);
}

// Each thread owns 32 consecutive positions.  Its policy / value bits come from interval
// arithmetic on the few sequences that overlap those positions (usually one) and from one 16-byte
// loads per byte mask, not from a test per position; selected positions are first compacted inside
// the tile in shared memory and then copied out with coalesced stores.
// (Six blocks per SM is what the two 16 KB lists allow; the bound keeps the kernel at 40 registers so
// that six are resident: 39.0 us against 40.3 us with 48 registers and five, at 17.5 M positions.)
__global__ void __launch_bounds__(kSelThreads, 6) select_tokens_kernel(const SelectArgs a) {
    // the tile's two compacted lists, as 16-bit offsets inside the tile (halves the shared memory)
    __shared__ uint16_t s_out_pol[kSelTile];
    __shared__ uint16_t s_out_val[kSelTile];
    __shared__ int32_t s_sb[kSeqCap + 1];
    __shared__ uint32_t s_tile;
    __shared__ uint32_t s_warp_cnt[kSelWarps];      // policy count | value count << 16
    __shared__ uint32_t s_base_pol, s_base_val, s_tot_pol, s_tot_val;
    int bad = 0;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // A tile only waits for tiles with smaller indices.
#if TPPO_SEL_TICKET
    asm volatile("griddepcontrol.wait;" ::: "memory");       // the counter is cleared by the kernel before
    if (threadIdx.x == 0) s_tile = atomicAdd(a.ticket, 1u);
#else
    if (threadIdx.x == 0) s_tile = blockIdx.x;
#endif
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= uint32_t(a.num_tiles)) return;
    const int64_t t0 = int64_t(tile) * kSelTile;
    const int n_tile = int(min(int64_t(kSelTile), int64_t(a.N) - t0));
    const int l0 = threadIdx.x * kSelItems;
    const int64_t p0 = t0 + l0;
    const int n_mine = max(0, min(kSelItems, n_tile - l0));    // positions this thread really owns

    // ---- the byte masks of this thread's positions, as bits (issued first: longest latency) ----
    uint32_t pm_bits = 0xffffffffu, vm_bits = 0xffffffffu;
    if (n_mine == kSelItems && a.mask_vec_ok) {
        if (a.pol_mask) {
            const uint4* m = reinterpret_cast<const uint4*>(a.pol_mask + p0);
            pm_bits = nonzero_bytes16(__ldg(m)) | (nonzero_bytes16(__ldg(m + 1)) << 16);
        }
        if (a.val_mask) {
            const uint4* m = reinterpret_cast<const uint4*>(a.val_mask + p0);
            vm_bits = nonzero_bytes16(__ldg(m)) | (nonzero_bytes16(__ldg(m + 1)) << 16);
        }
    } else {
        if (a.pol_mask) {
            pm_bits = 0;
            for (int k = 0; k < n_mine; ++k) pm_bits |= uint32_t(__ldg(a.pol_mask + p0 + k) != 0) << k;
        }
        if (a.val_mask) {
            vm_bits = 0;
            for (int k = 0; k < n_mine; ++k) vm_bits |= uint32_t(__ldg(a.val_mask + p0 + k) != 0) << k;
        }
    }
    // ... and ask for the mask bytes of a tile that a later block will take to be brought into L2
#ifndef TPPO_SEL_PREFETCH_TILES
#define TPPO_SEL_PREFETCH_TILES (2 * kNumSms)
#endif
    if (threadIdx.x == 64 && TPPO_SEL_PREFETCH_TILES > 0 && a.mask_vec_ok) {
        const int64_t q0 = (int64_t(tile) + TPPO_SEL_PREFETCH_TILES) * kSelTile;
        if (q0 + kSelTile <= a.N) {
            if (a.pol_mask) ptx::bulk_prefetch_l2(a.pol_mask + q0, kSelTile);
            if (a.val_mask) ptx::bulk_prefetch_l2(a.val_mask + q0, kSelTile);
        }
    }
    const uint32_t own_bits = n_mine >= kSelItems ? 0xffffffffu : ((1u << n_mine) - 1u);

    // ---- window of sequences that can touch the tile: [seq0, seq1), seq0 may be -1 -------------
    // Found for every tile by the small kernel launched just before this one (which also clears the
    // counts and the tile states and lets this kernel start at once: programmatic dependent launch).
    // Its end is awaited here; the mask loads above are in flight meanwhile.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int2 w = __ldcg(a.window + tile);
    const int seq0 = w.x, seq1 = w.y;
    const int first = max(seq0, 0);
    const int n_win = min(seq1, a.B) - first + 1;         // entries first .. min(seq1, B) inclusive
    const bool win_smem = n_win <= kSeqCap + 1;
    if (win_smem) {
        for (int j = threadIdx.x; j < n_win; j += kSelThreads) s_sb[j] = __ldg(a.seq_begin + first + j);
        __syncthreads();
    }

    // ---- policy / value bits of this thread's 32 positions --------------------------------------
    uint32_t pol_bits = 0, val_bits = 0;
    if (n_mine > 0 && seq1 > 0) {
        // last sequence of the window that begins at or before p0 (-1: none)
        int lo = 0, hi = min(seq1, a.B + 1) - first;       // entries first .. first+hi-1 are <= t_last
        const int32_t key = int32_t(p0);
        if (win_smem) {
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (s_sb[mid] <= key) lo = mid + 1; else hi = mid;
            }
        } else {
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (__ldg(a.seq_begin + first + mid) <= key) lo = mid + 1; else hi = mid;
            }
        }
        int i = first + lo - 1;                             // may be first-1 = -1 only when first == 0
        if (i < 0) i = 0;                                   // positions before sequence 0 select nothing
        const int64_t p_end = p0 + n_mine;
        for (; i < a.B; ++i) {
            const int64_t begin = win_smem ? s_sb[i - first] : __ldg(a.seq_begin + i);
            if (begin >= p_end) break;
            const int64_t next = win_smem ? s_sb[i + 1 - first] : __ldg(a.seq_begin + i + 1);
            if (next <= p0 || next <= begin) continue;      // empty, or entirely before this thread
            const int64_t resp0 = begin + __ldg(a.prompt_len + i);
            const int64_t new0 = resp0 + __ldg(a.prev_len + i);
            const int64_t end = new0 + __ldg(a.new_len + i);
            const bool trunc = __ldg(a.truncated + i) != 0;
            // how many of the latest tokens of an unfinished sequence are left out: one count for all,
            // or one per sequence (a negative count is reported and read as 0)
            int64_t drop = 0;
            if (trunc) {
                drop = a.tail_drop_seq ? __ldg(a.tail_drop_seq + i) : a.tail_drop;
                if (drop < 0) { drop = 0; bad = TPPO_DEV_BAD_INDEX; }
            }
            // a position belongs to the last sequence that begins at or before it: clip to [begin, next)
            pol_bits |= range_bits32(max(new0, begin), min(end - drop, next), p0);
            if (!trunc) val_bits |= range_bits32(max(resp0, begin), min(end, next), p0);
        }
    }
    pol_bits &= pm_bits & own_bits;
    val_bits &= vm_bits & own_bits;

    // ---- ranks inside the warp and the tile -----------------------------------------------------
    const uint32_t mine = uint32_t(__popc(pol_bits)) | (uint32_t(__popc(val_bits)) << 16);
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
    }
    if (lane == 31) s_warp_cnt[warp] = incl;
    __syncthreads();
    uint32_t before = incl - mine;                           // selected by lower lanes of this warp
    uint32_t tile_tot = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) {
        const uint32_t c = s_warp_cnt[w];
        if (w < warp) before += c;
        tile_tot += c;
    }
    // publish the tile's totals as early as possible: later tiles wait for them in their look-back
    if (threadIdx.x == 0 && tile > 0 && !a.no_publish)
        reinterpret_cast<volatile unsigned long long*>(a.state)[tile] =
            sel_pack(1, tile_tot & 0xffffu, tile_tot >> 16);
    if (bad) atomicOr(a.counts + 2, bad);
    // compact inside the tile (needs no global offset; earlier tiles finish meanwhile)
    {
        // (one loop over both lists, trip count the larger popcount instead of their sum, measured
        // slower: 43.3 against 41.0 us per call at 17.5 M tokens)
        uint32_t op = before & 0xffffu, ov = before >> 16;
        uint32_t b = pol_bits;
        while (b) { s_out_pol[op++] = uint16_t(l0 + __ffs(int(b)) - 1); b &= b - 1; }
        b = val_bits;
        while (b) { s_out_val[ov++] = uint16_t(l0 + __ffs(int(b)) - 1); b &= b - 1; }
    }

    // ---- tile total -> publish -> warp-wide look-back over earlier tiles ----------------------
    if (warp == 0) {
        const uint32_t tp = tile_tot & 0xffffu, tv = tile_tot >> 16;
        volatile unsigned long long* st = a.state;
        uint32_t ep = 0, ev = 0;
        bool timed_out = false;
        // 32 predecessors per round: lane l looks at tile j0 - l; positions before tile 0 count as
        // an inclusive prefix of zero.  The nearest inclusive prefix ends the walk.
        for (int64_t j0 = int64_t(tile) - 1; j0 >= 0; j0 -= 32) {
            const int64_t j = j0 - lane;
            uint64_t s = j >= 0 ? st[j] : sel_pack(2, 0, 0);
            uint32_t spins = 0;
            while (!__all_sync(0xffffffffu, sel_flag(s) != 0)) {
                if (++spins > a.spin_limit) { timed_out = true; break; }
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
            if (!a.no_publish) st[tile] = sel_pack(2, ep + tp, ev + tv);
            s_base_pol = ep;
            s_base_val = ev;
            s_tot_pol = tp;
            s_tot_val = tv;
            if (tile == uint32_t(a.num_tiles) - 1) {
                a.counts[0] = int32_t(ep + tp);
                a.counts[1] = int32_t(ev + tv);
            }
        }
    }
    __syncthreads();

    // ---- copy the tile's two lists out, coalesced ----------------------------------------------
    sel_copy_out(a.policy_idx, s_base_pol, int(s_tot_pol), s_out_pol, int32_t(t0), a.out_vec_ok != 0);
    sel_copy_out(a.value_idx, s_base_val, int(s_tot_val), s_out_val, int32_t(t0), a.out_vec_ok != 0);
}

// Launched just before the selection kernel, which is its programmatic dependent: clears the
// counts, the ticket counter and the tile states, and one thread per tile finds the tile's window
// of sequences -- seq0 = the last sequence that begins at or before the tile's first position (-1:
// none), seq1 = the number of sequences that begin at or before its last position -- by two searches
// over the sequence starts staged in shared memory (starts that do not fit are searched in global
// memory).  A search per tile inside the selection kernel was three dependent rounds of global loads
// in every tile's life.
constexpr int kSelClearThreads = 256;
constexpr int kSelClearSmemMaxB = 24575;      // 96 KB of sequence starts
template <bool LDG>
__device__ __forceinline__ int sel_count_le(const int32_t* __restrict__ arr, int n, int32_t key) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((LDG ? __ldg(arr + mid) : arr[mid]) <= key) lo = mid + 1; else hi = mid;
    }
    return lo;
}
__global__ void __launch_bounds__(kSelClearThreads) select_clear_kernel(
        int32_t* counts, uint32_t* ticket, unsigned long long* state, int2* window, int num_tiles,
        const int32_t* seq_begin, int B, int64_t N, int in_smem) {
    extern __shared__ __align__(16) int32_t s_starts[];      // seq_begin[0..B]
    asm volatile("griddepcontrol.launch_dependents;");
    const int tile = blockIdx.x * blockDim.x + threadIdx.x;
    if (tile < 4) counts[tile] = 0;
    if (tile == 0) *ticket = 0u;
    if (in_smem) {
        for (int i = threadIdx.x; i <= B; i += kSelClearThreads) s_starts[i] = __ldg(seq_begin + i);
        __syncthreads();
    }
    if (tile >= num_tiles) return;
    const int64_t t0 = int64_t(tile) * kSelTile;
    const int64_t t_last = min(t0 + kSelTile, N) - 1;
    const int c0 = in_smem ? sel_count_le<false>(s_starts, B + 1, int32_t(t0)) : sel_count_le<true>(seq_begin, B + 1, int32_t(t0));
    const int c1 = in_smem ? sel_count_le<false>(s_starts, B + 1, int32_t(t_last))
                           : sel_count_le<true>(seq_begin, B + 1, int32_t(t_last));
    state[tile] = 0ull;
    window[tile] = make_int2(c0 - 1, c1);
}

size_t select_workspace_bytes(int64_t N) {
    const int64_t tiles = (N + kSelTile - 1) / kSelTile;
    // head (ticket counter) | tile states | tile windows
    return kWsAlign + 2 * align_up(size_t(tiles > 0 ? tiles : 1) * 8, kWsAlign);
}
uint32_t test_spin_limit(uint32_t normal);
int32_t test_no_publish();

}  // namespace tppo

using namespace tppo;

TPPO_API int tppo_select_tokens(const int32_t* seq_begin, const int32_t* prompt_len,
                                const int32_t* prev_len, const int32_t* new_len,
                                const uint8_t* truncated, int32_t tail_drop,
                                const int32_t* tail_drop_seq,
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
    if (N == 0 || B == 0) {
        TPPO_CUDA_CHECK(cudaMemsetAsync(counts, 0, 4 * sizeof(int32_t), s));
        return TPPO_OK;
    }
    // One small kernel clears the counts and the tile states, and the selection kernel starts beside
    // it, reading masks and sequence bounds until it first needs either.  (Two memsets in front of a
    // plain launch cost 6 us more at 17.5 M tokens; handing the counts over by the last tile to
    // finish, to save the clear altogether, cost 6 us for the fence and counter at every tile's end.)
    const int32_t tiles = int32_t((N + kSelTile - 1) / kSelTile);
    unsigned long long* state = reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) + kWsAlign);
    int2* window = reinterpret_cast<int2*>(static_cast<char*>(workspace) + kWsAlign +
                                           align_up(size_t(tiles) * 8, kWsAlign));
    {
        const int in_smem = B <= kSelClearSmemMaxB;
        const size_t smem = in_smem ? (size_t(B) + 1) * sizeof(int32_t) : 0;
        if (smem > 48 * 1024)       // (an attribute of the function on the current device; the call is cheap)
            TPPO_CUDA_CHECK(cudaFuncSetAttribute(select_clear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (kSelClearSmemMaxB + 1) * int(sizeof(int32_t))));
        select_clear_kernel<<<(tiles + kSelClearThreads - 1) / kSelClearThreads, kSelClearThreads, smem, s>>>(
            counts, static_cast<uint32_t*>(workspace), state, window, tiles, seq_begin, B, N, in_smem);
        TPPO_CUDA_CHECK(cudaGetLastError());
    }
    SelectArgs a;
    a.seq_begin = seq_begin; a.prompt_len = prompt_len; a.prev_len = prev_len; a.new_len = new_len;
    a.truncated = truncated; a.pol_mask = extra_policy_mask; a.val_mask = extra_value_mask;
    a.tail_drop = tail_drop; a.tail_drop_seq = tail_drop_seq; a.B = B; a.N = int32_t(N);
    a.spin_limit = test_spin_limit(kSelSpinLimit);
    a.no_publish = test_no_publish();
    a.out_vec_ok = aligned(policy_idx, 16) && aligned(value_idx, 16);
    a.mask_vec_ok = (!extra_policy_mask || aligned(extra_policy_mask, 16)) &&
                    (!extra_value_mask || aligned(extra_value_mask, 16));
    a.num_tiles = tiles;
    a.policy_idx = policy_idx; a.value_idx = value_idx; a.counts = counts;
    a.ticket = static_cast<uint32_t*>(workspace);
    a.state = state;
    a.window = window;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(a.num_tiles));
    cfg.blockDim = dim3(kSelThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    TPPO_CUDA_CHECK(cudaLaunchKernelEx(&cfg, select_tokens_kernel, a));
    return TPPO_OK;
}

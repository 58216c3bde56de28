// Successive batching between two training steps (Section 3.2 of the paper, the batching figure;
// the batch collection step of Algorithm 1): the batch keeps its B slots, a finished sequence frees
// its slot for the next queued prompt, an unfinished one stays and the tokens of this window join its earlier ones.  Two
// kernels: one CTA walks the slots (two block-wide prefix sums per 4096 slots: rank among the freed
// slots, then the packed offsets of the next step's context), then a bandwidth-bound ragged copy
// moves the kept sequences and the queued prompts into the new packed token buffer.  Integer work
// throughout: bit-exact and run-to-run identical.
#include <algorithm>
#include "common.cuh"

namespace tppo {

constexpr int kAdvSlotThreads = 1024;
constexpr int kAdvCopyThreads = 256;
constexpr int kAdvCopyItems = 32;
constexpr int kAdvCopyTile = kAdvCopyThreads * kAdvCopyItems;     // 8192 tokens per CTA

struct AdvanceArgs {
    const int32_t* seq_begin;
    const int32_t* prompt_len;
    const int32_t* prev_len;
    const int32_t* new_len;
    const uint8_t* truncated;
    const int32_t* tokens;
    const int32_t* queue_begin;
    const int32_t* queue_tokens;
    int32_t B, M;
    int64_t N, queue_total, capacity;
    int32_t* next_prompt_len;
    int32_t* next_prev_len;
    int32_t* next_seq_begin;
    int32_t* next_tokens;
    int32_t* free_slots;
    int32_t* slot_source;
    int32_t* counts;     // [4]: freed, refilled, context tokens, status bits
};

// Exclusive prefix sum over the 1024 threads of the block; `total` receives the block's sum.
template <typename T>
__device__ __forceinline__ T block_exclusive_sum(T v, T* s_warp, T& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        T w = s_warp[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const T o = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w += o;
        }
        s_warp[lane] = w;              // inclusive over warps
    }
    __syncthreads();
    const T before = warp > 0 ? s_warp[warp - 1] : T(0);
    total = s_warp[31];
    __syncthreads();                   // s_warp is reused by the next call
    return before + incl - v;
}

constexpr int kAdvSlotItems = 4;                               // consecutive slots per thread

__global__ void __launch_bounds__(kAdvSlotThreads) advance_slots_kernel(const AdvanceArgs a) {
    __shared__ long long s_scan[32];
    __shared__ int s_bad;
    if (threadIdx.x == 0) s_bad = 0;
    // the copy kernel may be scheduled now; it waits for this grid to finish before it reads
    asm volatile("griddepcontrol.launch_dependents;");
    long long free_base = 0, pos_base = 0;
    int bad = 0;
    // a thread's four slots as one 16-byte access per array where the arrays allow it (the scalar
    // form's stores, 16 bytes apart between lanes, took 4 of the walk's 9 us at 4096 slots)
    const bool vec = (a.B & 3) == 0 &&
                     ((reinterpret_cast<uintptr_t>(a.prompt_len) | reinterpret_cast<uintptr_t>(a.prev_len) |
                       reinterpret_cast<uintptr_t>(a.new_len) | reinterpret_cast<uintptr_t>(a.next_prompt_len) |
                       reinterpret_cast<uintptr_t>(a.next_prev_len) | reinterpret_cast<uintptr_t>(a.slot_source) |
                       reinterpret_cast<uintptr_t>(a.next_seq_begin)) & 15) == 0 &&
                     (reinterpret_cast<uintptr_t>(a.truncated) & 3) == 0;
    for (int c0 = 0; c0 < a.B; c0 += kAdvSlotThreads * kAdvSlotItems) {
        const int i0 = c0 + int(threadIdx.x) * kAdvSlotItems;
        bool valid[kAdvSlotItems], fin[kAdvSlotItems];
        long long p[kAdvSlotItems], q[kAdvSlotItems], n[kAdvSlotItems];
        int my_fin = 0;
        static_assert(kAdvSlotItems == 4, "one 16-byte access per array and thread");
        if (vec) {
            const bool in = i0 < a.B;       // all four or none
            const uint32_t t4 = in ? __ldg(reinterpret_cast<const uint32_t*>(a.truncated + i0)) : 0u;
            const int4 z = make_int4(0, 0, 0, 0);
            const int4 p4 = in ? __ldg(reinterpret_cast<const int4*>(a.prompt_len + i0)) : z;
            const int4 q4 = in ? __ldg(reinterpret_cast<const int4*>(a.prev_len + i0)) : z;
            const int4 n4 = in ? __ldg(reinterpret_cast<const int4*>(a.new_len + i0)) : z;
            const int pp[4] = {p4.x, p4.y, p4.z, p4.w}, qq[4] = {q4.x, q4.y, q4.z, q4.w},
                      nn[4] = {n4.x, n4.y, n4.z, n4.w};
#pragma unroll
            for (int u = 0; u < kAdvSlotItems; ++u) {
                valid[u] = in;
                fin[u] = in && ((t4 >> (8 * u)) & 0xffu) == 0;
                p[u] = pp[u]; q[u] = qq[u]; n[u] = nn[u];
                my_fin += fin[u];
            }
        } else {
#pragma unroll
            for (int u = 0; u < kAdvSlotItems; ++u) {
                const int i = i0 + u;
                valid[u] = i < a.B;
                fin[u] = valid[u] && __ldg(a.truncated + i) == 0;
                p[u] = valid[u] ? __ldg(a.prompt_len + i) : 0;
                q[u] = valid[u] ? __ldg(a.prev_len + i) : 0;
                n[u] = valid[u] ? __ldg(a.new_len + i) : 0;
                my_fin += fin[u];
            }
        }
        long long n_fin;
        long long rank = free_base + block_exclusive_sum<long long>(my_fin, s_scan, n_fin);
        long long len[kAdvSlotItems];
        int32_t pl[kAdvSlotItems], pv[kAdvSlotItems], src[kAdvSlotItems];
        long long my_len = 0;
#pragma unroll
        for (int u = 0; u < kAdvSlotItems; ++u) {
            len[u] = 0; pl[u] = 0; pv[u] = 0; src[u] = -2;
            if (!valid[u]) continue;
            if (!fin[u]) {                                    // unfinished: stays in its slot
                if (p[u] < 0 || q[u] < 0 || n[u] < 0 || q[u] + n[u] > 0x7fffffffll) bad |= TPPO_DEV_BAD_INDEX;
                pl[u] = int32_t(p[u]);
                pv[u] = int32_t(q[u] + n[u]);
                src[u] = -1;
                len[u] = p[u] + q[u] + n[u];
            } else {                                          // finished: freed, refilled while the queue lasts
                a.free_slots[rank] = i0 + u;
                if (rank < a.M) {
                    const int32_t k = int32_t(rank);
                    len[u] = (long long)__ldg(a.queue_begin + k + 1) - __ldg(a.queue_begin + k);
                    if (len[u] < 0) { bad |= TPPO_DEV_BAD_INDEX; len[u] = 0; }
                    pl[u] = int32_t(len[u]);
                    src[u] = k;
                }
                ++rank;
            }
            if (len[u] < 0) len[u] = 0;
            my_len += len[u];
        }
        long long n_tok;
        long long begin = pos_base + block_exclusive_sum<long long>(my_len, s_scan, n_tok);
        if (vec) {
            if (valid[0]) {
                int32_t nb[kAdvSlotItems];
#pragma unroll
                for (int u = 0; u < kAdvSlotItems; ++u) {
                    nb[u] = int32_t(begin < 0x7fffffffll ? begin : 0x7fffffffll);
                    begin += len[u];
                }
                *reinterpret_cast<int4*>(a.next_prompt_len + i0) = make_int4(pl[0], pl[1], pl[2], pl[3]);
                *reinterpret_cast<int4*>(a.next_prev_len + i0) = make_int4(pv[0], pv[1], pv[2], pv[3]);
                *reinterpret_cast<int4*>(a.slot_source + i0) = make_int4(src[0], src[1], src[2], src[3]);
                *reinterpret_cast<int4*>(a.next_seq_begin + i0) = make_int4(nb[0], nb[1], nb[2], nb[3]);
            }
        } else {
#pragma unroll
            for (int u = 0; u < kAdvSlotItems; ++u) {
                if (valid[u]) {
                    const int i = i0 + u;
                    a.next_prompt_len[i] = pl[u];
                    a.next_prev_len[i] = pv[u];
                    a.slot_source[i] = src[u];
                    a.next_seq_begin[i] = int32_t(begin < 0x7fffffffll ? begin : 0x7fffffffll);
                    begin += len[u];
                }
            }
        }
        free_base += n_fin;
        pos_base += n_tok;
    }
    if (pos_base > 0x7fffffffll || pos_base > a.capacity) bad |= TPPO_DEV_OVERFLOW;
    // this block writes all four counts (no clear beforehand); the copy kernel, which runs after it,
    // adds its own status bits
    __syncthreads();
    if (bad) atomicOr(&s_bad, bad);
    __syncthreads();
    if (threadIdx.x == 0) {
        bad = s_bad;
        a.next_seq_begin[a.B] = int32_t(pos_base < 0x7fffffffll ? pos_base : 0x7fffffffll);
        a.counts[0] = int32_t(free_base);
        a.counts[1] = int32_t(free_base < a.M ? free_base : a.M);
        a.counts[2] = int32_t(pos_base < 0x7fffffffll ? pos_base : 0x7fffffffll);
        a.counts[3] = bad;
    }
}

// number of entries of the ascending array arr[0..n) that are <= key (whole warp, 32-ary search)
__device__ __forceinline__ int adv_warp_count_le(const int32_t* arr, int n, int32_t key, int lane) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int span = hi - lo;
        const int step = (span + 31) >> 5;
        const int idx = lo + lane * step;
        const bool le = idx < hi && arr[idx] <= key;
        const uint32_t m = __ballot_sync(0xffffffffu, le);
        const int c = __ffs(int(~m)) - 1;
        if (c < 0) { lo = min(lo + 31 * step + 1, hi); continue; }
        const int new_hi = min(lo + c * step, hi);
        if (c > 0) lo = lo + (c - 1) * step + 1;
        hi = new_hi;
    }
    return lo;
}

// Ragged copy into the next step's packed context.  A block owns one stretch of consecutive output
// positions (an even share of the context, at least 8192).
// It finds the first slot that reaches into them (one warp-wide search), puts the slots of its range
// into a small shared-memory table -- where each begins in the output and a source pointer already
// shifted so that source = pointer[output position], null for a slot whose source range is not inside
// its array -- and then every thread moves four consecutive positions at a time: four loads (the
// source is only 4-byte aligned), one 16-byte store.  Groups that straddle two slots, and blocks
// whose range holds more slots than the table, fall back to one position at a time.
// 8 bytes of traffic per token.
constexpr int kAdvTable = 128;

struct AdvSlotRef {
    int64_t begin, next;       // output range of the slot
    const int32_t* src;        // source = src[output position]; null: nothing to read
};
__device__ __forceinline__ AdvSlotRef adv_slot_ref(const AdvanceArgs& a, int i, int& bad) {
    AdvSlotRef r;
    r.begin = a.next_seq_begin[i];
    r.next = a.next_seq_begin[i + 1];
    r.src = nullptr;
    const int32_t s = a.slot_source[i];
    const int64_t len = r.next - r.begin;
    if (len <= 0) return r;
    if (s == -1) {
        const int64_t q = a.seq_begin[i];
        if (q >= 0 && q + len <= a.N) r.src = a.tokens + q - r.begin;
    } else if (s >= 0 && s < a.M) {
        const int64_t q = a.queue_begin[s];
        if (q >= 0 && q + len <= a.queue_total) r.src = a.queue_tokens + q - r.begin;
    }
    if (!r.src) bad = TPPO_DEV_BAD_INDEX;       // positions of such a slot are written as 0
    return r;
}

__global__ void __launch_bounds__(kAdvCopyThreads, 6) advance_copy_kernel(const AdvanceArgs a) {
    __shared__ int s_slot0;
    __shared__ int32_t s_begin[kAdvTable + 1];
    __shared__ const int32_t* s_src[kAdvTable];
    // launched as a programmatic dependent of the slot walk: everything above this line (block
    // scheduling, the parameter fetch) overlaps with it; its results are read only after the wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t total = min(int64_t(a.next_seq_begin[a.B]), a.capacity);
    // The grid is sized on the host for what the output buffer can hold, at most one wave of resident
    // blocks; the context actually written is split evenly between them (one slot search and one
    // table per block, no ragged last wave), in stretches that are a multiple of four positions so
    // that the 16-byte stores stay aligned, and of at least a tile.
    int64_t per = (total + gridDim.x - 1) / gridDim.x;
    per = max((per + 3) & ~int64_t(3), int64_t(kAdvCopyTile));
    const int64_t t0 = int64_t(blockIdx.x) * per;
    if (t0 >= total) return;
    const int64_t t1 = min(t0 + per, total);
    if (threadIdx.x < 32) {
        const int c = adv_warp_count_le(a.next_seq_begin, a.B + 1, int32_t(t0), threadIdx.x);
        if (threadIdx.x == 0) s_slot0 = c - 1;      // last slot that begins at or before t0
    }
    __syncthreads();
    const int slot0 = max(s_slot0, 0);
    int bad = 0;
    for (int j = threadIdx.x; j <= kAdvTable; j += kAdvCopyThreads) {
        const int i = slot0 + j;
        if (j < kAdvTable && i < a.B) {
            const AdvSlotRef r = adv_slot_ref(a, i, bad);
            s_begin[j] = int32_t(r.begin);
            s_src[j] = r.src;
        } else {
            s_begin[j] = i <= a.B ? a.next_seq_begin[min(i, a.B)] : INT32_MAX;
            if (j < kAdvTable) s_src[j] = nullptr;
        }
    }
    __syncthreads();
    // the table serves the block when its last entry begins at or beyond the block's last position
    const bool table_ok = int64_t(s_begin[kAdvTable]) >= t1 || slot0 + kAdvTable >= a.B;
    const bool vec = (reinterpret_cast<uintptr_t>(a.next_tokens) & 15) == 0;
    if (table_ok && vec) {
        // kGroups groups of four positions per trip, all their loads issued before the first store
        const int n_slots = min(kAdvTable, a.B - slot0);          // table entries in use
        const int32_t e1 = int32_t(t1);
        int h = 0;
        constexpr int kStep = 4 * kAdvCopyThreads;
        constexpr int kGroups = 2;      // (3, 4 and 6 groups in flight measured the same: 30.2-31.1 us per call)
        for (int32_t p0 = int32_t(t0) + 4 * threadIdx.x; p0 < e1; p0 += kGroups * kStep) {
            int4 v[kGroups];
            bool whole[kGroups];
#pragma unroll
            for (int u = 0; u < kGroups; ++u) {
                const int32_t p = p0 + u * kStep;
                v[u] = make_int4(0, 0, 0, 0);
                whole[u] = false;
                if (p >= e1) continue;
                while (h + 1 < n_slots && p >= s_begin[h + 1]) ++h;
                whole[u] = p + 4 <= e1 && p + 4 <= s_begin[h + 1];      // four positions of one slot
                if (whole[u]) {
                    const int32_t* src = s_src[h];
                    if (src) {
                        v[u].x = __ldg(src + p); v[u].y = __ldg(src + p + 1);
                        v[u].z = __ldg(src + p + 2); v[u].w = __ldg(src + p + 3);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kGroups; ++u) {
                const int32_t p = p0 + u * kStep;
                if (p >= e1) continue;
                if (whole[u]) {
                    *reinterpret_cast<int4*>(a.next_tokens + p) = v[u];
                } else {        // the group straddles two slots or the end: one position at a time
                    int hh = 0;
                    for (int e = 0; e < 4 && p + e < e1; ++e) {
                        while (hh + 1 < n_slots && p + e >= s_begin[hh + 1]) ++hh;
                        const int32_t* src = s_src[hh];
                        a.next_tokens[p + e] = src ? __ldg(src + p + e) : 0;
                    }
                }
            }
        }
    } else {
        // one position at a time, each thread walking the slots forward as its positions advance
        int i = slot0;
        AdvSlotRef r = adv_slot_ref(a, i, bad);
        for (int64_t p = t0 + threadIdx.x; p < t1; p += kAdvCopyThreads) {
            while (p >= r.next && i + 1 < a.B) r = adv_slot_ref(a, ++i, bad);
            a.next_tokens[p] = (r.src && p >= r.begin && p < r.next) ? __ldg(r.src + p) : 0;
        }
    }
    if (bad) atomicOr(a.counts + 3, bad);
}

}  // namespace tppo

using namespace tppo;

TPPO_API int tppo_advance_batch(const int32_t* seq_begin, const int32_t* prompt_len,
                                const int32_t* prev_len, const int32_t* new_len,
                                const uint8_t* truncated, const int32_t* tokens, int64_t N,
                                const int32_t* queue_begin, const int32_t* queue_tokens,
                                int64_t queue_total, int32_t B, int32_t M,
                                int32_t* next_prompt_len, int32_t* next_prev_len,
                                int32_t* next_seq_begin, int32_t* next_tokens, int64_t capacity,
                                int32_t* free_slots, int32_t* slot_source, int32_t* counts,
                                void* stream) {
    if (B < 0 || M < 0 || N < 0 || queue_total < 0 || capacity < 0 || !counts || !next_seq_begin)
        return TPPO_ERR_INVALID_ARG;
    if (N >= (int64_t(1) << 31) || queue_total >= (int64_t(1) << 31) || capacity >= (int64_t(1) << 31))
        return TPPO_ERR_INVALID_ARG;
    if (B > 0 && (!seq_begin || !prompt_len || !prev_len || !new_len || !truncated ||
                  !next_prompt_len || !next_prev_len || !free_slots || !slot_source))
        return TPPO_ERR_INVALID_ARG;
    if ((N > 0 && !tokens) || (M > 0 && !queue_begin) || (queue_total > 0 && !queue_tokens) ||
        (capacity > 0 && !next_tokens))
        return TPPO_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    AdvanceArgs a;
    a.seq_begin = seq_begin; a.prompt_len = prompt_len; a.prev_len = prev_len; a.new_len = new_len;
    a.truncated = truncated; a.tokens = tokens; a.queue_begin = queue_begin;
    a.queue_tokens = queue_tokens; a.B = B; a.M = M; a.N = N; a.queue_total = queue_total;
    a.capacity = capacity; a.next_prompt_len = next_prompt_len; a.next_prev_len = next_prev_len;
    a.next_seq_begin = next_seq_begin; a.next_tokens = next_tokens; a.free_slots = free_slots;
    a.slot_source = slot_source; a.counts = counts;
    advance_slots_kernel<<<1, kAdvSlotThreads, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    if (B > 0 && capacity > 0) {
        // the number of context tokens is only known on the device: size the grid for the most the
        // output buffer can hold; CTAs past the end return at once
        int64_t upper = N + queue_total < capacity ? N + queue_total : capacity;
        int64_t tiles = (upper + kAdvCopyTile - 1) / kAdvCopyTile;
        tiles = std::min<int64_t>(tiles, int64_t(kNumSms) * 6);       // one wave of resident blocks
        if (tiles > 0) {
            // programmatic dependent launch: the copy kernel's blocks are scheduled while the slot
            // walk still runs and wait inside the kernel for its results
            cudaLaunchConfig_t lc = {};
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            lc.gridDim = dim3(unsigned(tiles), 1, 1);
            lc.blockDim = dim3(kAdvCopyThreads, 1, 1);
            lc.dynamicSmemBytes = 0;
            lc.stream = s;
            lc.attrs = attr;
            lc.numAttrs = 1;
            TPPO_CUDA_CHECK(cudaLaunchKernelEx(&lc, advance_copy_kernel, a));
        }
    }
    return TPPO_OK;
}

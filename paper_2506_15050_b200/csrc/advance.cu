// Successive batching between two training steps (Section 3.2 of the paper, the batching figure;
// the batch collection step of Algorithm 1): the batch keeps its B slots, a finished sequence frees
// its slot for the next queued prompt, an unfinished one stays and the tokens of this window join its earlier ones.  Two
// kernels: one CTA walks the slots (two block-wide prefix sums per 4096 slots: rank among the freed
// slots, then the packed offsets of the next step's context), then a bandwidth-bound ragged copy
// moves the kept sequences and the queued prompts into the new packed token buffer.  Integer work
// throughout: bit-exact and run-to-run identical.
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
    long long free_base = 0, pos_base = 0;
    int bad = 0;
    for (int c0 = 0; c0 < a.B; c0 += kAdvSlotThreads * kAdvSlotItems) {
        const int i0 = c0 + int(threadIdx.x) * kAdvSlotItems;
        bool valid[kAdvSlotItems], fin[kAdvSlotItems];
        long long p[kAdvSlotItems], q[kAdvSlotItems], n[kAdvSlotItems];
        int my_fin = 0;
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
        free_base += n_fin;
        pos_base += n_tok;
    }
    if (pos_base > 0x7fffffffll || pos_base > a.capacity) bad |= TPPO_DEV_OVERFLOW;
    if (bad) atomicOr(a.counts + 3, bad);
    if (threadIdx.x == 0) {
        a.next_seq_begin[a.B] = int32_t(pos_base < 0x7fffffffll ? pos_base : 0x7fffffffll);
        a.counts[0] = int32_t(free_base);
        a.counts[1] = int32_t(free_base < a.M ? free_base : a.M);
        a.counts[2] = int32_t(pos_base < 0x7fffffffll ? pos_base : 0x7fffffffll);
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

// Ragged copy into the next step's packed context: consecutive threads take consecutive output
// positions (coalesced stores; loads are coalesced inside a slot), each thread walks the slots
// forward as its positions advance.  8 bytes of traffic per token.
__global__ void __launch_bounds__(kAdvCopyThreads) advance_copy_kernel(const AdvanceArgs a) {
    __shared__ int s_slot0;
    const int64_t total = min(int64_t(a.next_seq_begin[a.B]), a.capacity);
    const int64_t t0 = int64_t(blockIdx.x) * kAdvCopyTile;
    if (t0 >= total) return;
    if (threadIdx.x < 32) {
        const int c = adv_warp_count_le(a.next_seq_begin, a.B + 1, int32_t(t0), threadIdx.x);
        if (threadIdx.x == 0) s_slot0 = c - 1;      // last slot that begins at or before t0
    }
    __syncthreads();
    int i = max(s_slot0, 0);
    int64_t begin = a.next_seq_begin[i], next = a.next_seq_begin[i + 1];
    int32_t src = a.slot_source[i];
    int64_t src_base = src == -1 ? int64_t(a.seq_begin[i]) : (src >= 0 ? int64_t(a.queue_begin[src]) : 0);
    int bad = 0;
    // batches of eight positions: resolve the sources, issue the eight loads, then store
    for (int j0 = 0; j0 < kAdvCopyItems; j0 += 8) {
        const int32_t* srcp[8];
        int64_t pos[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t p = t0 + threadIdx.x + int64_t(j0 + u) * kAdvCopyThreads;
            pos[u] = p;
            srcp[u] = nullptr;
            if (p >= total) continue;
            while (p >= next && i + 1 < a.B) {
                ++i;
                begin = next;
                next = a.next_seq_begin[i + 1];
                src = a.slot_source[i];
                src_base = src == -1 ? int64_t(a.seq_begin[i]) : (src >= 0 ? int64_t(a.queue_begin[src]) : 0);
            }
            const int64_t q = src_base + (p - begin);
            if (src == -1 && q >= 0 && q < a.N) srcp[u] = a.tokens + q;
            else if (src >= 0 && q >= 0 && q < a.queue_total) srcp[u] = a.queue_tokens + q;
            else bad = TPPO_DEV_BAD_INDEX;
        }
        int32_t v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = srcp[u] ? __ldg(srcp[u]) : 0;
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (pos[u] < total) a.next_tokens[pos[u]] = v[u];
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
    TPPO_CUDA_CHECK(cudaMemsetAsync(counts, 0, 4 * sizeof(int32_t), s));
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
        const int64_t tiles = (upper + kAdvCopyTile - 1) / kAdvCopyTile;
        if (tiles > 0) {
            advance_copy_kernel<<<unsigned(tiles), kAdvCopyThreads, 0, s>>>(a);
            TPPO_CUDA_CHECK(cudaGetLastError());
        }
    }
    return TPPO_OK;
}

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
// Tiles are staged in shared memory so that every global access is a coalesced 16-byte one.
#include <cstddef>

#include "common.cuh"

namespace tppo {

constexpr int kScanThreads = 128;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kScanItems = 16;
constexpr int kScanTile = kScanThreads * kScanItems;  // 2048 positions
constexpr int kSegCap = 64;                           // segments of one tile kept in shared memory
constexpr int kScanCtasPerSm = 6;
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

// One per tile, 64 bytes, three self-validating 16-byte pairs.  The array starts out as all-ones
// bytes; a pair counts as published only when neither of its two words holds that pattern, so a
// reader needs one load per pair and neither a separate flag nor a fence (each 8-byte word is
// written whole, and a pair with one word still unset is simply read again).
struct TileState {
    double aggA[2];    // (a, b) of the tile's composite for the advantage recurrence
    double aggR[2];    // (a, b) of the tile's composite for the return recurrence
    double inc[2];     // A and R at the tile's first position
    double pad[2];
};
static_assert(sizeof(TileState) == 64, "tile state is four 16-byte pairs");
constexpr unsigned long long kUnset = 0xffffffffffffffffull;
// NaNs are published with the canonical quiet pattern so that no result can look unset.
__device__ __forceinline__ double publishable(double x) {
    return x != x ? __longlong_as_double(0x7ff8000000000000ll) : x;
}
__device__ __forceinline__ void st_pair(double* p, double x, double y) {
    asm volatile("st.relaxed.gpu.global.v2.f64 [%0], {%1, %2};"
                 ::"l"(p), "d"(publishable(x)), "d"(publishable(y)) : "memory");
}
__device__ __forceinline__ bool ld_pair(const double* p, double& x, double& y) {
    asm volatile("ld.relaxed.gpu.global.v2.f64 {%0, %1}, [%2];" : "=d"(x), "=d"(y) : "l"(p) : "memory");
    return (unsigned long long)__double_as_longlong(x) != kUnset &&
           (unsigned long long)__double_as_longlong(y) != kUnset;
}

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
    int32_t vec_ok;   // rewards, values, adv, ret are all 16-byte aligned
    double gamma;
    double gl;  // gamma * lambda
    double gamma_run, gl_run;   // gamma and gamma*lambda to the power kScanItems
    float* adv;
    float* ret;
    int32_t* status;
    TileState* state;
    uint32_t* ticket;
};

// Number of entries of the ascending array arr[0..n) that are <= key, found by a whole warp: each
// round probes 32 evenly spaced entries, so 4096 entries take three rounds of one load each
// instead of twelve dependent loads.  Every lane returns the same count.  An array that is not
// ascending still yields an in-range answer.
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
        if (c < 0) { lo = min(lo + 31 * step + 1, hi); continue; }   // all 32 probes <= key
        const int new_hi = min(lo + c * step, hi);
        if (c > 0) lo = lo + (c - 1) * step + 1;
        hi = new_hi;
    }
    return lo;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                 ::"r"(uint32_t(__cvta_generic_to_shared(smem_dst))), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.wait_all;" ::: "memory");
}

// Shared-memory image of one tile: its inputs and the window of segments that can touch it.
// r and v are stored in 16-byte chunks (four positions); a thread owns four consecutive chunks,
// so chunk c sits at slot c ^ ((c >> 3) & 3): the eight lanes of a quarter warp then read eight
// different bank groups instead of two.  Aligned and sized to 16 bytes: float4 and cp.async access
// in both halves of a two-element array.
struct __align__(16) TileBuf {
    float r[kScanTile];          // rewards
    float v[kScanTile + 4];      // values (+1 look-ahead)
    int32_t seg_b[kSegCap], seg_e[kSegCap];
    float seg_boot[kSegCap];
    uint8_t seg_t[kSegCap];
    int win_lo, win_hi;          // segment indices [win_lo, win_hi) may touch the tile
};
static_assert(sizeof(TileBuf) % 16 == 0 && offsetof(TileBuf, v) % 16 == 0, "vector access alignment");
__device__ __forceinline__ int chunk_slot(int c) { return c ^ ((c >> 3) & 3); }
__device__ __forceinline__ int pos_slot(int l) { return (chunk_slot(l >> 2) << 2) | (l & 3); }

// Starts the copy of a tile's rewards and values into `buf`, by threads first, first + step, ...
// 16-byte chunks go through cp.async (the caller waits with cp_async_wait_all and a barrier); a
// ragged tail or unaligned arrays are read directly.
__device__ __forceinline__ void egae_stage_inputs(const EgaeArgs& a, TileBuf& buf, int64_t t0,
                                                  int n_tile, int first, int step) {
    if (a.vec_ok) {
        for (int u = first; u < kScanTile / 4; u += step) {
            if (4 * u + 4 <= n_tile) {
                const int s = 4 * chunk_slot(u);
                cp_async16(buf.r + s, a.rewards + t0 + 4 * u);
                cp_async16(buf.v + s, a.values + t0 + 4 * u);
            } else {
                for (int k = 4 * u; k < n_tile; ++k) {
                    buf.r[pos_slot(k)] = __ldg(a.rewards + t0 + k);
                    buf.v[pos_slot(k)] = __ldg(a.values + t0 + k);
                }
            }
        }
    } else {
        for (int k = first; k < n_tile; k += step) {
            buf.r[pos_slot(k)] = __ldg(a.rewards + t0 + k);
            buf.v[pos_slot(k)] = __ldg(a.values + t0 + k);
        }
    }
    if (first == 0)    // value of the position after the tile, if there is one
        buf.v[pos_slot(n_tile)] = (t0 + n_tile < a.N) ? __ldg(a.values + t0 + n_tile) : 0.f;
}

// Segments are ascending and disjoint, so seg_begin and seg_end are both ascending: the window of
// a tile starts after the segments that end at or before its first position and stops before those
// that begin after its last one.  Called by two whole warps (which = 0: lower end, 1: upper end).
__device__ __forceinline__ void egae_window_search(const EgaeArgs& a, TileBuf& buf, int64_t t0,
                                                   int n_tile, int which, int lane) {
    if (which == 0) {
        const int lo = warp_count_le(a.seg_end, a.B, int32_t(t0), lane);
        if (lane == 0) buf.win_lo = lo;
    } else {
        const int hi = warp_count_le(a.seg_begin, a.B, int32_t(t0 + n_tile - 1), lane);
        if (lane == 0) buf.win_hi = hi;
    }
}
// Copies the window's segments into shared memory (when they fit).  Returns true when a segment
// with bounds outside [0, N] or end < begin was seen; such a segment is treated as empty.
__device__ __forceinline__ bool egae_window_load(const EgaeArgs& a, TileBuf& buf) {
    const int win_lo = buf.win_lo, win_n = buf.win_hi - buf.win_lo;
    bool bad = false;
    if (win_n <= kSegCap) {
        for (int j = threadIdx.x; j < win_n; j += kScanThreads) {
            const int i = win_lo + j;
            int32_t b = __ldg(a.seg_begin + i), e = __ldg(a.seg_end + i);
            if (b < 0 || e > a.N || e < b) { bad = true; e = b; }
            buf.seg_b[j] = b;
            buf.seg_e[j] = e;
            buf.seg_t[j] = __ldg(a.truncated + i);
            buf.seg_boot[j] = a.bootstrap ? __ldg(a.bootstrap + i) : 0.f;
        }
    }
    return bad;
}

// Value entering a tile from its right-hand side, by a whole warp: lane i inspects tile first + i.
// A tile that has published its first-position values (or lies beyond the end, or whose composite
// has multiplier 0 because a segment ended inside it) terminates the search; the composites of the
// tiles before it are folded in order.  One round of loads usually suffices, where a single lane
// walking tile by tile would pay one L2 round trip per tile.  Returns false when the bounded wait
// ran out.  The result is valid in lane 0.
__device__ __forceinline__ bool egae_look_back(const EgaeArgs& a, int first, int lane, double& xA,
                                               double& xR) {
    Affine2 F = identity2();      // composite of the tiles folded so far (meaningful in lane 0)
    for (int base = first;; base += 32) {
        const int j = base + lane;
        const bool beyond = j >= a.num_tiles;
        const TileState* st = a.state + (beyond ? 0 : j);
        double i0 = 0.0, i1 = 0.0, pa = 1.0, pb = 0.0, qa = 1.0, qb = 0.0;
        bool got_inc = beyond, got_agg = false;
        int p = 32;
        uint32_t spins = 0;
        for (;;) {
            if (!beyond) {     // the three pairs are requested together: one round trip
                if (!got_inc) got_inc = ld_pair(st->inc, i0, i1);
                if (!got_agg) {
                    double ta, tb, ua, ub;
                    const bool ga = ld_pair(st->aggA, ta, tb);
                    const bool gr = ld_pair(st->aggR, ua, ub);
                    if (ga && gr) { got_agg = true; pa = ta; pb = tb; qa = ua; qb = ub; }
                }
            }
            const bool term = got_inc || (got_agg && pa == 0.0 && qa == 0.0);
            const uint32_t tmask = __ballot_sync(0xffffffffu, term);
            const uint32_t rmask = __ballot_sync(0xffffffffu, got_inc || got_agg);
            p = tmask ? __ffs(int(tmask)) - 1 : 32;
            const uint32_t need = p < 32 ? ((1u << p) - 1u) : 0xffffffffu;
            if ((rmask & need) == need) break;
            if (++spins > kScanSpinLimit) return false;     // uniform: decided from the ballots
            __nanosleep(20);
        }
        // lane < p: the tile's composite; lane p: the constant map to its value; beyond p: identity
        Affine2 m = identity2();
        if (lane < p) m = Affine2{pa, pb, qa, qb};
        else if (lane == p) m = got_inc ? Affine2{0.0, i0, 0.0, i1} : Affine2{0.0, pb, 0.0, qb};
        if (p > 0) {
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const Affine2 o = shfl_down(m, d);
                if (lane + d < 32) m = compose(m, o);
            }
        }
        if (p < 32) {       // m is constant in lane 0: its b is the value entering the first folded tile
            xA = fma(F.aA, m.bA, F.bA);
            xR = fma(F.aR, m.bR, F.bR);
            return true;
        }
        F = compose(F, m);
    }
}

// Persistent CTAs take tiles by ticket, from the END of the arrays backwards, so the tiles a tile
// looks back at (those to its right) hold earlier tickets and are running or done.  While a tile is
// being scanned the next ticket is drawn, the next tile's inputs stream into the other buffer
// (cp.async, issued by the warps that do not look back) and two of them find its segment window, so
// none of those latencies is exposed.  A thread owns sixteen consecutive positions: the warp scan
// and the barriers are paid once per 512 positions of a warp.
__global__ void __launch_bounds__(kScanThreads, kScanCtasPerSm) egae_scan_kernel(const EgaeArgs a) {
    __shared__ __align__(16) TileBuf s_buf[2];
    __shared__ uint32_t s_ticket[2];
    __shared__ Affine2 s_warp[kScanWarps];
    __shared__ double s_carry[kScanWarps][2];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // the ticket counter starts at all-ones like the rest of the workspace (one memset): + 1 wraps
    // the first draw to ticket 0
    if (threadIdx.x == 0) s_ticket[0] = atomicAdd(a.ticket, 1u) + 1u;
    __syncthreads();
    uint32_t ticket = s_ticket[0];
    if (ticket >= uint32_t(a.num_tiles)) return;
    bool bad = false;
    {   // first tile of this CTA: nothing to overlap with
        const int tile = a.num_tiles - 1 - int(ticket);
        const int64_t t0 = int64_t(tile) * kScanTile;
        const int n_tile = int(min(int64_t(kScanTile), int64_t(a.N) - t0));
        egae_stage_inputs(a, s_buf[0], t0, n_tile, threadIdx.x, kScanThreads);
        if (warp < 2) egae_window_search(a, s_buf[0], t0, n_tile, warp, lane);
        __syncthreads();
        bad |= egae_window_load(a, s_buf[0]);
        cp_async_wait_all();
        __syncthreads();
    }

    for (int it = 0;; ++it) {
        TileBuf& buf = s_buf[it & 1];
        TileBuf& nbuf = s_buf[(it & 1) ^ 1];
        const int tile = a.num_tiles - 1 - int(ticket);
        const int64_t t0 = int64_t(tile) * kScanTile;
        const int n_tile = int(min(int64_t(kScanTile), int64_t(a.N) - t0));
        if (threadIdx.x == 0) s_ticket[(it & 1) ^ 1] = atomicAdd(a.ticket, 1u) + 1u;   // next tile

        // ---- per-position maps, right to left -----------------------------------------------
        const int win_lo = buf.win_lo;
        const int win_n = max(buf.win_hi - win_lo, 0);
        const bool win_smem = win_n <= kSegCap;
        const int l0 = threadIdx.x * kScanItems;  // first position of this thread inside the tile
        const int swz = (threadIdx.x >> 1) & 3;   // the thread's chunks 4*tid + q sit at slot (4*tid + q) ^ swz
        double delta[kScanItems];
        uint32_t cont = 0;    // bit k: position k continues into position k+1 (same segment)
        uint32_t inside = 0;  // bit k: position k lies inside a segment
        Affine2 f = identity2();
        // index (inside the window) of the last segment that begins at or before the thread's
        // last position, or -1
        const int l_last = min(l0 + kScanItems, n_tile) - 1;
        int i = -1;
        if (l_last >= l0) {
            const int32_t key = int32_t(t0 + l_last);
            int lo = 0, hi = win_n;
            if (win_smem && win_n <= 4) {
                while (lo < win_n && buf.seg_b[lo] <= key) ++lo;
            } else if (win_smem) {
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (buf.seg_b[mid] <= key) lo = mid + 1; else hi = mid;
                }
            } else {
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (__ldg(a.seg_begin + win_lo + mid) <= key) lo = mid + 1; else hi = mid;
                }
            }
            i = lo - 1;
        }
        // The common case: all sixteen positions lie inside one segment and none of them is its
        // last token.  Then every map has the same multiplier and no per-position test is needed.
        bool fast = false;
        if (win_smem && i >= 0 && l0 + kScanItems <= n_tile)
            fast = int64_t(buf.seg_b[i]) <= t0 + l0 && t0 + l0 + kScanItems < int64_t(buf.seg_e[i]);
        if (fast) {
            double dn = double(buf.v[pos_slot(l0 + kScanItems)]);
            double bA = 0.0, bR = 0.0;
#pragma unroll
            for (int q = kScanItems / 4 - 1; q >= 0; --q) {
                const int s = 4 * ((4 * threadIdx.x + q) ^ swz);
                const float4 r4 = *reinterpret_cast<const float4*>(buf.r + s);
                const float4 v4 = *reinterpret_cast<const float4*>(buf.v + s);
                const float rr[4] = {r4.x, r4.y, r4.z, r4.w};
                const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                for (int e = 3; e >= 0; --e) {
                    const double dv = double(vv[e]), dr = double(rr[e]);
                    const double d = fma(a.gamma, dn, dr) - dv;
                    delta[4 * q + e] = d;
                    bA = fma(a.gl, bA, d);
                    bR = fma(a.gamma, bR, dr);
                    dn = dv;
                }
            }
            f = Affine2{a.gl_run, bA, a.gamma_run, bR};
            cont = 0xffffu;
            inside = 0xffffu;
        } else {
            float vnext_f = buf.v[pos_slot(min(l0 + kScanItems, n_tile))];
#pragma unroll
            for (int k = kScanItems - 1; k >= 0; --k) {
                const int l = l0 + k;
                delta[k] = 0.0;
                if (l >= n_tile) continue;   // past the end: the identity map
                const int32_t p = int32_t(t0 + l);
                const float vf = buf.v[pos_slot(l)];
                int32_t b = 0, e = 0;
                bool have = false;
                while (i >= 0) {
                    if (win_smem) {
                        b = buf.seg_b[i];
                        e = buf.seg_e[i];
                    } else {
                        b = __ldg(a.seg_begin + win_lo + i);
                        e = __ldg(a.seg_end + win_lo + i);
                        if (b < 0 || e > a.N || e < b) { bad = true; e = b; }
                    }
                    if (p >= b) { have = true; break; }
                    --i;
                }
                double aA = 0.0, aR = 0.0, dr = 0.0;
                if (have && p < e) {
                    dr = double(buf.r[pos_slot(l)]);
                    const double v = double(vf);
                    double v_next;
                    if (p + 1 < e) {
                        v_next = double(vnext_f);
                        aA = a.gl;
                        aR = a.gamma;
                        cont |= 1u << k;
                    } else {
                        const bool tr = win_smem ? (buf.seg_t[i] != 0)
                                                 : (__ldg(a.truncated + win_lo + i) != 0);
                        if (tr) {
                            v_next = a.bootstrap ? double(win_smem ? buf.seg_boot[i]
                                                                   : __ldg(a.bootstrap + win_lo + i))
                                                 : v;
                        } else {
                            v_next = 0.0;
                        }
                    }
                    delta[k] = fma(a.gamma, v_next, dr) - v;
                    inside |= 1u << k;
                }
                vnext_f = vf;
                f = compose(Affine2{aA, delta[k], aR, dr}, f);
            }
        }

        // ---- inclusive suffix composition inside the warp: S_l = f_l o f_{l+1} o ... o f_31 ---
        Affine2 S = f;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const Affine2 o = shfl_down(S, d);
            if (lane + d < 32) S = compose(S, o);
        }
        Affine2 excl = shfl_down(S, 1);   // composite of the lanes to the right
        if (lane == 31) excl = identity2();
        if (lane == 0) s_warp[warp] = S;
        __syncthreads();                                                      // (A)

        const uint32_t next_ticket = s_ticket[(it & 1) ^ 1];
        const bool has_next = next_ticket < uint32_t(a.num_tiles);
        if (warp != 0) {
            // ---- next tile: start its loads and its window search while warp 0 looks back -----
            if (has_next) {
                const int ntile = a.num_tiles - 1 - int(next_ticket);
                const int64_t nt0 = int64_t(ntile) * kScanTile;
                const int nn_tile = int(min(int64_t(kScanTile), int64_t(a.N) - nt0));
                egae_stage_inputs(a, nbuf, nt0, nn_tile, threadIdx.x - 32, kScanThreads - 32);
                if (warp <= 2) egae_window_search(a, nbuf, nt0, nn_tile, warp - 1, lane);
            }
        } else {
            // ---- tile composite, look-back, per-warp carries (warp 0) --------------------------
            // lane w < 4 holds warp w's composite; suffix-compose them, so that lane w ends with
            // W_w o ... o W_3 and lane 0 with the tile's composite
            Affine2 W = lane < kScanWarps ? s_warp[lane] : identity2();
#pragma unroll
            for (int d = 1; d < kScanWarps; d <<= 1) W = compose(W, shfl_down(W, d));
            Affine2 right = shfl_down(W, 1);            // composite of the warps to the right
            if (lane >= kScanWarps - 1) right = identity2();
            TileState* st = a.state;
            if (lane == 0 && tile + 1 < a.num_tiles) {
                st_pair(st[tile].aggA, W.aA, W.bA);
                st_pair(st[tile].aggR, W.aR, W.bR);
            }
            double xA = 0.0, xR = 0.0;
            const bool ok = egae_look_back(a, tile + 1, lane, xA, xR);
            if (lane == 0) {
                if (!ok) { atomicOr(a.status, TPPO_DEV_WAIT_TIMEOUT); xA = 0.0; xR = 0.0; }
                st_pair(st[tile].inc, fma(W.aA, xA, W.bA), fma(W.aR, xR, W.bR));
            }
            xA = __shfl_sync(0xffffffffu, xA, 0);
            xR = __shfl_sync(0xffffffffu, xR, 0);
            if (lane < kScanWarps) {
                s_carry[lane][0] = fma(right.aA, xA, right.bA);
                s_carry[lane][1] = fma(right.aR, xR, right.bR);
            }
        }
        __syncthreads();                                                      // (B)
        if (has_next) bad |= egae_window_load(a, nbuf);

        // ---- replay the thread's positions with the true incoming values, store -----------------
        double A = fma(excl.aA, s_carry[warp][0], excl.bA);
        double G = fma(excl.aR, s_carry[warp][1], excl.bR);
        const bool full = a.vec_ok && l0 + kScanItems <= n_tile;
#pragma unroll
        for (int q = kScanItems / 4 - 1; q >= 0; --q) {
            float rr[4] = {0.f, 0.f, 0.f, 0.f};
            if (l0 + 4 * q < n_tile) {       // the chunk was staged (a ragged one only in part: masked below)
                const float4 r4 = *reinterpret_cast<const float4*>(buf.r + 4 * ((4 * threadIdx.x + q) ^ swz));
                rr[0] = r4.x; rr[1] = r4.y; rr[2] = r4.z; rr[3] = r4.w;
            }
            float oa[4], og[4];
#pragma unroll
            for (int e = 3; e >= 0; --e) {
                const int k = 4 * q + e;
                const bool c = (cont >> k) & 1u;
                const double dr = ((inside >> k) & 1u) ? double(rr[e]) : 0.0;
                A = c ? fma(a.gl, A, delta[k]) : delta[k];
                G = c ? fma(a.gamma, G, dr) : dr;
                oa[e] = float(A);
                og[e] = float(G);
            }
            if (full) {
                *reinterpret_cast<float4*>(a.adv + t0 + l0 + 4 * q) = make_float4(oa[0], oa[1], oa[2], oa[3]);
                if (a.ret)
                    *reinterpret_cast<float4*>(a.ret + t0 + l0 + 4 * q) = make_float4(og[0], og[1], og[2], og[3]);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (l0 + 4 * q + e < n_tile) {
                        a.adv[t0 + l0 + 4 * q + e] = oa[e];
                        if (a.ret) a.ret[t0 + l0 + 4 * q + e] = og[e];
                    }
                }
            }
        }
        if (!has_next) break;
        cp_async_wait_all();
        __syncthreads();                                                      // (D)
        ticket = next_ticket;
    }
    if (bad) atomicOr(a.status, TPPO_DEV_BAD_SEGMENT);
}

// persistent grid: as many CTAs as can be resident, fewer when there are fewer tiles
static inline int egae_grid(int num_tiles) {
    const int resident = kNumSms * kScanCtasPerSm;
    return num_tiles < resident ? num_tiles : resident;
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
    // one memset: tile states start out unset (all-ones), the ticket counter at all-ones too
    TPPO_CUDA_CHECK(cudaMemsetAsync(workspace, 0xff, need, s));
    EgaeArgs a;
    a.rewards = rewards; a.values = values; a.seg_begin = seg_begin; a.seg_end = seg_end;
    a.truncated = truncated; a.bootstrap = bootstrap; a.B = B; a.N = int32_t(N);
    a.num_tiles = int32_t((N + kScanTile - 1) / kScanTile);
    a.gamma = double(gamma);
    a.gl = double(gamma) * double(lambda);
    a.gamma_run = 1.0; a.gl_run = 1.0;
    for (int k = 0; k < kScanItems; ++k) { a.gamma_run *= a.gamma; a.gl_run *= a.gl; }
    a.adv = advantages; a.ret = returns; a.status = status;
    a.vec_ok = aligned(rewards, 16) && aligned(values, 16) && aligned(advantages, 16) &&
               (!returns || aligned(returns, 16));
    a.ticket = static_cast<uint32_t*>(workspace);
    a.state = reinterpret_cast<TileState*>(static_cast<char*>(workspace) +
                                           align_up(sizeof(uint32_t), kWsAlign));
    egae_scan_kernel<<<egae_grid(a.num_tiles), kScanThreads, 0, s>>>(a);
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
    a.gamma_run = 1.0; a.gl_run = 1.0;
    for (int k = 0; k < kScanItems; ++k) { a.gamma_run *= a.gamma; a.gl_run *= a.gl; }
    a.adv = advantages; a.ret = returns; a.status = status;
    a.vec_ok = aligned(rewards, 16) && aligned(values, 16) && aligned(advantages, 16) &&
               (!returns || aligned(returns, 16));
    a.ticket = static_cast<uint32_t*>(scratch);
    a.state = reinterpret_cast<TileState*>(static_cast<char*>(scratch) + 256);
    // the array still holds the previous call's tile states and ticket: reset the part this call
    // uses to the all-ones pattern (tile states unset, ticket counter one draw before ticket 0)
    TPPO_CUDA_CHECK(cudaMemsetAsync(scratch, 0xff, 256 + size_t(a.num_tiles) * sizeof(TileState), s));
    egae_scan_kernel<<<egae_grid(a.num_tiles), kScanThreads, 0, s>>>(a);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

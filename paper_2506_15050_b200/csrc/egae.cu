// EGAE advantages and Monte-Carlo returns (Section 3.1, Eq. 6 with the TD residual of Eq. 3; R_t
// after Eq. 5) as ONE segmented reverse scan over the packed token arrays.
//
// The advantage recurrence A_t = delta_t + (gamma*lambda) A_{t+1} is carried as G_t = A_t + V_t,
//     G_t = r_t + gamma (1 - lambda) V_{t+1} + (gamma*lambda) G_{t+1},    R_t = r_t + gamma R_{t+1},
// (on the last token of a segment G_t = r_t + gamma V_next, with V_next the boundary value), so the
// values enter additively and successive values never cancel against each other.  Both recurrences
// are affine in the value at the next position: every position carries a map x -> a*x + b, with
// a = 0 on the last token of a segment and outside every segment.  Maps compose associatively.
//
// Precision.  A thread owns sixteen consecutive positions (its run).  The composite map of a run,
// and everything that crosses threads -- the warp scan, the tile composites, the look-back -- is
// fp64: the value that enters a run is exact to double rounding however long the segment is.  (With
// fp32 run composites, each run's rounding, small as it is, added up over the hundreds of runs of a
// long response: 2.5e-5 absolute on zero-mean dense rewards over 9000 tokens.)  The results of a run
// are then replayed from that entering value, rounded to fp32 once, sequentially in fp32 (the
// multiplier gamma*lambda split into two floats, exact to 2^-48).  The error of a result is thus the
// rounding of the entering value plus at most sixteen fp32 roundings at the magnitude of |G| or |R|
// inside its own run; nothing accumulates over the length of a segment.
//
// Tiles of 2048 positions are worked on from the END of the arrays backwards, so the tiles a
// tile looks back at (those to its right) were started earlier and are running or done.  A tile
// composes its positions right to left, publishes the composite, and obtains the value entering
// from its right-hand neighbour by decoupled look-back over the tiles behind it.  A composite whose
// `a` has become 0 (a segment ended inside the range) ends the look-back early.  The inputs of a
// whole tile arrive by two tiled TMA copies (rows of 32 positions, 128-byte swizzle: the four
// 16-byte chunks a thread owns then sit in different bank groups from its neighbours'); there is no
// per-thread staging code.
#include <algorithm>
#include <cstddef>
#include <cstring>

#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "umma.cuh"

namespace tppo {

#ifndef TPPO_SCAN_ITEMS
#define TPPO_SCAN_ITEMS 16
#endif
constexpr int kScanItems = TPPO_SCAN_ITEMS;           // consecutive positions per thread (its run): 16 or 32
constexpr int kScanTile = 2048;                       // positions per tile (4096 measured 5 % slower)
constexpr int kScanThreads = kScanTile / kScanItems;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kScanChunks = kScanItems / 4;           // 16-byte chunks of a run
constexpr int kThreadsPerRow = 32 / kScanItems;       // a row of the tile image holds 32 positions
constexpr uint32_t kRunMask = kScanItems == 32 ? 0xffffffffu : ((1u << (kScanItems & 31)) - 1u);
static_assert(kScanItems == 8 || kScanItems == 16 || kScanItems == 32, "a run is a quarter, half or whole row");
__device__ __forceinline__ uint32_t bits_below(int k) { return k >= 32 ? 0xffffffffu : ((1u << k) - 1u); }
constexpr int kSegCap = 32;                           // segments of one tile kept in shared memory
#ifndef TPPO_SCAN_CTAS
#define TPPO_SCAN_CTAS (TPPO_SCAN_ITEMS == 16 ? 8 : (TPPO_SCAN_ITEMS == 8 ? 4 : 12))
#endif
constexpr int kScanCtasPerSm = TPPO_SCAN_CTAS;   // registers resp. shared memory allow no more
constexpr int kScanBoxRows = 64;                      // rows of 32 positions per TMA box
constexpr int kScanBoxes = kScanTile / (kScanBoxRows * 32);
static_assert(kScanTile % (kScanBoxRows * 32) == 0, "a tile is a whole number of TMA boxes");
constexpr uint32_t kScanSpinLimit = 1u << 22;
// Tile order.  0 (default): block b takes tile num_tiles-1-b.  A tile only ever waits for tiles to
// its right, i.e. for blocks with smaller indices, and thread blocks are dispatched in index order, so
// those are running or done; should that ever not hold, the bounded wait gives up and the call
// reports TPPO_DEV_WAIT_TIMEOUT instead of hanging.  1: tiles are drawn from an atomic ticket
// counter instead, which needs no assumption about dispatch order (measured 1.3 us slower at
// 17.5 M tokens: one L2 round trip and one barrier more in every tile's life).
#ifndef TPPO_EGAE_TICKET
#define TPPO_EGAE_TICKET 0
#endif

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
    int32_t win[4];    // per 2048-position part of the tile: segments [win[2p], win[2p+1]) may touch it (written by the clearing kernel)
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
__device__ __forceinline__ bool pair_set(double x, double y) {
    return (unsigned long long)__double_as_longlong(x) != kUnset &&
           (unsigned long long)__double_as_longlong(y) != kUnset;
}
// The three pairs of a tile state in one go: the loads are issued back to back (one round trip to
// L2 instead of three).
__device__ __forceinline__ void ld_state(const TileState* st, double& pa, double& pb, double& qa,
                                         double& qb, double& i0, double& i1) {
    asm volatile(
        "ld.relaxed.gpu.global.v2.f64 {%0, %1}, [%6];\n\t"
        "ld.relaxed.gpu.global.v2.f64 {%2, %3}, [%6+16];\n\t"
        "ld.relaxed.gpu.global.v2.f64 {%4, %5}, [%6+32];"
        : "=d"(pa), "=d"(pb), "=d"(qa), "=d"(qb), "=d"(i0), "=d"(i1) : "l"(st) : "memory");
}
static_assert(offsetof(TileState, aggA) == 0 && offsetof(TileState, aggR) == 16 &&
              offsetof(TileState, inc) == 32, "ld_state reads the pairs by offset");

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
    int32_t tma_ok;   // the two tensor maps are valid: whole tiles arrive by TMA
    double gamma;
    double gl;  // gamma * lambda
    double gamma_run, gl_run;   // gamma and gamma*lambda to the power kScanItems
    float gamma_f;              // gamma (an fp32 input: exact)
    float gl_hi, gl_lo;         // gamma*lambda = gl_hi + gl_lo up to 2^-48
    float c1;                   // gamma * (1 - lambda)
    double c1_d;                // the same, not rounded to fp32
    float* adv;
    float* ret;
    int32_t* status;
    TileState* state;
    int32_t after_clear;   // launched as the programmatic dependent of the kernel that clears status and states
    uint32_t* ticket;      // head of the workspace, cleared to all-ones with the tile states (+1 wraps to 0)
    uint32_t spin_limit;   // polls a look-back may spend on one round of tiles before it gives up
    int32_t no_publish;    // test hook: tiles keep their states to themselves, so every look-back runs out
};
__device__ __forceinline__ void egae_raise(const EgaeArgs& a, int bits) { atomicOr(a.status, bits); }
__device__ __forceinline__ bool finite_f32(float x) { return fabsf(x) <= kFltMax; }

// Shared-memory image of one tile.  r and v are 64 rows of 32 positions (128 bytes) in the layout
// the TMA's 128-byte swizzle writes: 16-byte chunk c of row y sits at chunk c ^ (y & 7) of that row
// (the arrays are 1024-byte aligned, eight rows).  A thread owns half a row; the eight lanes of a
// quarter warp then read eight different bank groups.
constexpr int kRowPos = 32;
struct __align__(1024) TileBuf {
    float r[kScanTile];          // rewards
    float v[kScanTile];          // values
    float v_after;               // value of the position after the tile (0 beyond the arrays)
};
// The segments that can touch a tile (its window), copied next to it when they are few.
struct TileWin {
    int32_t seg_b[kSegCap], seg_e[kSegCap];
    float seg_boot[kSegCap];
    uint8_t seg_t[kSegCap];
    int win_lo, win_hi;          // segment indices [win_lo, win_hi) may touch the tile
};
static_assert(offsetof(TileBuf, v) % 1024 == 0, "swizzle atom alignment");
__device__ __forceinline__ int pos_slot(int l) {      // float index of position l
    const int y = l >> 5;
    return (y << 5) | (((((l >> 2) & 7) ^ (y & 7)) << 2)) | (l & 3);
}

// What one position contributes, for threads that touch a segment boundary or lie outside every
// segment (the others never call this).  `i` is the index, inside the window, of the last segment
// that begins at or before the positions still to come; the caller walks l downwards and `i`
// follows.  x is the additive term of the G recurrence, r the reward; cont says that the position
// continues into position l + 1 of the same segment (otherwise its map is constant).  The value of
// position l + 1 is passed in: by the time of the replay its slot may hold a result already.
struct PosTerm {
    float x, r, v;
    double xd;          // x before its rounding to fp32
    bool cont, inside;
};
__device__ __forceinline__ PosTerm egae_position(const EgaeArgs& a, const TileBuf& buf,
                                                 const TileWin& win, int64_t t0,
                                                 int n_tile, int win_lo, bool win_smem, int l,
                                                 float v_next_pos, int& i, bool& bad, bool& nonfinite) {
    PosTerm o{0.f, 0.f, 0.f, 0.0, false, false};
    if (l >= n_tile) return o;
    const int32_t p = int32_t(t0 + l);
    int32_t b = 0, e = 0;
    bool have = false;
    while (i >= 0) {
        if (win_smem) {
            b = win.seg_b[i];
            e = win.seg_e[i];
        } else {
            b = __ldg(a.seg_begin + win_lo + i);
            e = __ldg(a.seg_end + win_lo + i);
            if (b < 0 || e > a.N || e < b) { bad = true; e = b; }
        }
        if (p >= b) { have = true; break; }
        --i;
    }
    if (!have || p >= e) return o;
    o.inside = true;
    o.r = buf.r[pos_slot(l)];
    o.v = buf.v[pos_slot(l)];
    if (!finite_f32(o.r)) { o.r = 0.f; nonfinite = true; }      // read as 0 and reported
    if (!finite_f32(o.v)) { o.v = 0.f; nonfinite = true; }
    if (!finite_f32(v_next_pos)) v_next_pos = 0.f;               // (its owner reports it)
    if (p + 1 < e) {
        o.xd = fma(a.c1_d, double(v_next_pos), double(o.r));
        o.x = fmaf(a.c1, v_next_pos, o.r);
        o.cont = true;
    } else {      // last token: G = r + gamma * (0 | bootstrap value | its own value)
        const bool tr = win_smem ? (win.seg_t[i] != 0) : (__ldg(a.truncated + win_lo + i) != 0);
        float v_next = 0.f;
        if (tr) v_next = a.bootstrap ? (win_smem ? win.seg_boot[i] : __ldg(a.bootstrap + win_lo + i)) : o.v;
        if (!finite_f32(v_next)) { v_next = 0.f; nonfinite = true; }     // tr is set here
        o.xd = fma(a.gamma, double(v_next), double(o.r));
        o.x = fmaf(a.gamma_f, v_next, o.r);
    }
    return o;
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
            if (!beyond && !got_inc) {
                double ta, tb, ua, ub, j0, j1;
                ld_state(st, ta, tb, ua, ub, j0, j1);
                if (pair_set(j0, j1)) { got_inc = true; i0 = j0; i1 = j1; }
                if (!got_agg && pair_set(ta, tb) && pair_set(ua, ub)) {
                    got_agg = true; pa = ta; pb = tb; qa = ua; qb = ub;
                }
            }
            const bool term = got_inc || (got_agg && pa == 0.0 && qa == 0.0);
            const uint32_t tmask = __ballot_sync(0xffffffffu, term);
            const uint32_t rmask = __ballot_sync(0xffffffffu, got_inc || got_agg);
            p = tmask ? __ffs(int(tmask)) - 1 : 32;
            const uint32_t need = p < 32 ? ((1u << p) - 1u) : 0xffffffffu;
            if ((rmask & need) == need) break;
            if (++spins > a.spin_limit) return false;       // uniform: decided from the ballots
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

// Number of entries of an ascending array arr[0..n) that are <= key, found by a whole warp: each
// round probes 32 evenly spaced entries until at most 128 remain, which are then read in one go
// (four independent loads per lane), so 4096 entries take two dependent rounds instead of twelve
// dependent loads.  Every lane returns the same count; an array that is not ascending still yields
// an in-range answer.  Two counts at once (the two ends of a tile's segment window), the rounds of
// both searches overlapped so that their loads are in flight together.
__device__ __forceinline__ void warp_count_le2(const int32_t* __restrict__ arr1, int32_t key1,
                                               const int32_t* __restrict__ arr2, int32_t key2, int n,
                                               int lane, int& c1, int& c2) {
    int lo1 = 0, hi1 = n, lo2 = 0, hi2 = n;
    while (hi1 - lo1 > 128 || hi2 - lo2 > 128) {
        const bool go1 = hi1 - lo1 > 128, go2 = hi2 - lo2 > 128;
        const int step1 = (hi1 - lo1 + 31) >> 5, step2 = (hi2 - lo2 + 31) >> 5;
        const int idx1 = lo1 + lane * step1, idx2 = lo2 + lane * step2;
        const int32_t x1 = go1 && idx1 < hi1 ? __ldg(arr1 + idx1) : INT32_MAX;
        const int32_t x2 = go2 && idx2 < hi2 ? __ldg(arr2 + idx2) : INT32_MAX;
        const uint32_t m1 = __ballot_sync(0xffffffffu, go1 && idx1 < hi1 && x1 <= key1);
        const uint32_t m2 = __ballot_sync(0xffffffffu, go2 && idx2 < hi2 && x2 <= key2);
        if (go1) {
            const int c = __ffs(int(~m1)) - 1;      // leading run of probes that are <= key
            if (c < 0) {
                lo1 = min(lo1 + 31 * step1 + 1, hi1);
            } else {
                const int new_hi = min(lo1 + c * step1, hi1);
                if (c > 0) lo1 = lo1 + (c - 1) * step1 + 1;
                hi1 = new_hi;
            }
        }
        if (go2) {
            const int c = __ffs(int(~m2)) - 1;
            if (c < 0) {
                lo2 = min(lo2 + 31 * step2 + 1, hi2);
            } else {
                const int new_hi = min(lo2 + c * step2, hi2);
                if (c > 0) lo2 = lo2 + (c - 1) * step2 + 1;
                hi2 = new_hi;
            }
        }
    }
    bool le1[4], le2[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int i1 = lo1 + 32 * j + lane, i2 = lo2 + 32 * j + lane;
        le1[j] = i1 < hi1 && __ldg(arr1 + i1) <= key1;
        le2[j] = i2 < hi2 && __ldg(arr2 + i2) <= key2;
    }
    c1 = lo1;
    c2 = lo2;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        c1 += __popc(__ballot_sync(0xffffffffu, le1[j]));
        c2 += __popc(__ballot_sync(0xffffffffu, le2[j]));
    }
}

// The segment window of a tile, found and copied into shared memory by one warp.  Returns true when
// a segment with bounds outside [0, N] or end < begin was seen; such a segment is treated as empty.
static_assert(kSegCap == 32, "one lane per window segment");
__device__ __forceinline__ bool egae_window(const EgaeArgs& a, TileWin& win, int64_t t0, int n_tile,
                                            int lane, bool& nonfinite, const int32_t* found) {
    // segments are ascending and disjoint, so seg_begin and seg_end are both ascending: the window
    // starts after the segments that end at or before the tile's first position and stops before
    // those that begin after its last one
    int lo, hi;
    if (found) {      // found for every tile by the clearing kernel
        const int2 w = __ldcg(reinterpret_cast<const int2*>(found));
        lo = w.x; hi = w.y;
    } else {
        warp_count_le2(a.seg_end, int32_t(t0), a.seg_begin, int32_t(t0 + n_tile - 1), a.B, lane, lo, hi);
    }
    if (lane == 0) { win.win_lo = lo; win.win_hi = hi; }
    bool bad = false;
    if (hi - lo <= kSegCap && lane < hi - lo) {
        const int i = lo + lane;
        int32_t b = __ldg(a.seg_begin + i), e = __ldg(a.seg_end + i);
        if (b < 0 || e > a.N || e < b) { bad = true; e = b; }
        win.seg_b[lane] = b;
        win.seg_e[lane] = e;
        win.seg_t[lane] = __ldg(a.truncated + i);
        float boot = a.bootstrap ? __ldg(a.bootstrap + i) : 0.f;
        if (!finite_f32(boot)) { boot = 0.f; nonfinite |= win.seg_t[lane] != 0; }   // used by cut responses only
        win.seg_boot[lane] = boot;
    }
    return bad;
}

// What a thread keeps of its run between composing its maps and replaying them.
struct RunState {
    Affine2 excl;     // composite of the lanes to its right inside the warp
    int i_start;      // window index of the last segment that begins at or before its last position
    bool fast;        // its sixteen positions lie inside one segment, none of them the last token
    // Otherwise, when at most one segment ends inside the run (`masked`): which positions lie inside
    // a segment (bits 0-15), which of them continue into the next position (bits 16-31), and for the
    // one last token, its position (or -1) and the value its TD residual bootstraps from
    bool masked;
    uint32_t inside, cont;
    int k_last;
    float v_boundary;
    bool boundary_own;   // the boundary value is the last token's own value (no bootstrap array)
    float v_right;       // value of the position after the run (its slot is overwritten by the replay)
};

// The thread's sixteen positions, right to left: its composite map.  `probe` comes back NaN when a
// reward or value that the straight-line paths read was not finite (x * 0 is NaN exactly then).
__device__ __forceinline__ Affine2 egae_run_map_once(const EgaeArgs& a, const TileBuf& buf,
                                                     const TileWin& win, int64_t t0,
                                                     int n_tile, int tid, RunState& rs, bool& bad,
                                                     float& probe, bool& nonfinite) {
    float probe0 = 0.f;
    const int win_lo = win.win_lo;
    const int win_n = max(win.win_hi - win_lo, 0);
    const bool win_smem = win_n <= kSegCap;
    const int l0 = tid * kScanItems;        // first position of this thread inside the tile
    // its four chunks: row tid/2, chunks 4*(tid&1) + q, stored at chunk ^ (row & 7)
    const int row_base = (tid / kThreadsPerRow) << 5;
    const int chunk0 = (tid % kThreadsPerRow) * kScanChunks, swz = (tid / kThreadsPerRow) & 7;
    const int l_last = min(l0 + kScanItems, n_tile) - 1;
    int i_start = -1;
    if (l_last >= l0) {
        const int32_t key = int32_t(t0 + l_last);
        int lo = 0, hi = win_n;
        if (win_smem && win_n <= 4) {
            while (lo < win_n && win.seg_b[lo] <= key) ++lo;
        } else if (win_smem) {
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (win.seg_b[mid] <= key) lo = mid + 1; else hi = mid;
            }
        } else {
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (__ldg(a.seg_begin + win_lo + mid) <= key) lo = mid + 1; else hi = mid;
            }
        }
        i_start = lo - 1;
    }
    bool fast = false;
    if (win_smem && i_start >= 0 && l0 + kScanItems <= n_tile)
        fast = int64_t(win.seg_b[i_start]) <= t0 + l0 &&
               t0 + l0 + kScanItems < int64_t(win.seg_e[i_start]);
    rs.i_start = i_start;
    rs.fast = fast;
    rs.masked = false;
    float v_right = l0 + kScanItems < kScanTile ? buf.v[pos_slot(l0 + kScanItems)] : buf.v_after;
    if (!finite_f32(v_right)) v_right = 0.f;     // read as 0; the thread that owns it reports it
    rs.v_right = v_right;
    if (!fast && win_smem) {
        // The segments that overlap the run, from the right: usually one or two.  With at most one
        // segment end inside the run the per-position work stays branch-free (two bit masks and one
        // special position); runs that hold several tiny segments take the general loop below.
        const int64_t p0 = t0 + l0;
        uint32_t inside = 0, cont = 0;
        int n_last = 0;
        rs.k_last = -1;
        rs.v_boundary = 0.f;
        rs.boundary_own = false;
        for (int i = i_start; i >= 0; --i) {
            const int64_t b = win.seg_b[i], e = win.seg_e[i];
            if (e <= p0 && e > b) break;      // ascending and disjoint: the earlier ones end earlier still
            const int lo = int(max(b, p0) - p0), hi = int(min(e, p0 + kScanItems) - p0);
            if (hi <= lo) continue;
            const uint32_t m = bits_below(hi) & ~bits_below(lo);
            inside |= m;
            cont |= m;
            if (e <= p0 + kScanItems) {       // the segment's last token lies in the run
                const int k = int(e - 1 - p0);
                cont &= ~(1u << k);
                ++n_last;
                rs.k_last = k;
                rs.v_boundary = 0.f;
                rs.boundary_own = false;
                if (win.seg_t[i]) {
                    if (a.bootstrap) rs.v_boundary = win.seg_boot[i];
                    else rs.boundary_own = true;
                }
            }
        }
        rs.inside = inside;
        rs.cont = cont;
        rs.masked = n_last <= 1;
    }
    if (rs.masked) {
        const uint32_t inside = rs.inside, cont = rs.cont;
        double bG = 0.0, bR = 0.0;
        float vn = v_right;
#pragma unroll
        for (int q = kScanChunks - 1; q >= 0; --q) {
            const int s = row_base + (((chunk0 + q) ^ swz) << 2);
            const float4 r4 = *reinterpret_cast<const float4*>(buf.r + s);
            const float4 v4 = *reinterpret_cast<const float4*>(buf.v + s);
            const float rr[4] = {r4.x, r4.y, r4.z, r4.w};
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
            for (int e = 3; e >= 0; --e) {
                const int k = 4 * q + e;
                const bool in = (inside >> k) & 1u, c = (cont >> k) & 1u;
                probe0 = fmaf(rr[e], 0.f, probe0);
                probe0 = fmaf(vv[e], 0.f, probe0);
                const double rd = in ? double(rr[e]) : 0.0;
                double x = fma(a.c1_d, double(vn), rd);
                if (k == rs.k_last) x = fma(a.gamma, double(rs.boundary_own ? vv[e] : rs.v_boundary), rd);
                x = in ? x : 0.0;
                bG = c ? fma(a.gl, bG, x) : x;
                bR = c ? fma(a.gamma, bR, rd) : rd;
                vn = vv[e];
            }
        }
        probe = probe0;
        const bool whole = cont == kRunMask;
        return Affine2{whole ? a.gl_run : 0.0, double(bG), whole ? a.gamma_run : 0.0, double(bR)};
    }
    if (fast) {
        // every map has the same multiplier and no per-position test is needed
        double bG = 0.0, bR = 0.0;
        float vn = v_right;
#pragma unroll
        for (int q = kScanChunks - 1; q >= 0; --q) {
            const int s = row_base + (((chunk0 + q) ^ swz) << 2);
            const float4 r4 = *reinterpret_cast<const float4*>(buf.r + s);
            const float4 v4 = *reinterpret_cast<const float4*>(buf.v + s);
            const float rr[4] = {r4.x, r4.y, r4.z, r4.w};
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
            for (int e = 3; e >= 0; --e) {
                probe0 = fmaf(rr[e], 0.f, probe0);
                probe0 = fmaf(vv[e], 0.f, probe0);
                const double rd = double(rr[e]);
                bG = fma(a.gl, bG, fma(a.c1_d, double(vn), rd));
                bR = fma(a.gamma, bR, rd);
                vn = vv[e];
            }
        }
        probe = probe0;
        return Affine2{a.gl_run, double(bG), a.gamma_run, double(bR)};
    }
    double bG = 0.0, bR = 0.0;
    double aG = 1.0, aR = 1.0;
    int i = i_start;
    float v_next = v_right;
#pragma unroll 1
    for (int k = kScanItems - 1; k >= 0; --k) {
        const PosTerm t = egae_position(a, buf, win, t0, n_tile, win_lo, win_smem, l0 + k, v_next, i, bad, nonfinite);
        v_next = buf.v[pos_slot(l0 + k)];
        if (t.cont) {
            bG = fma(a.gl, bG, t.xd);
            bR = fma(a.gamma, bR, double(t.r));
            aG *= a.gl;
            aR *= a.gamma;
        } else {
            bG = t.xd;
            bR = t.r;
            aG = 0.0;
            aR = 0.0;
        }
    }
    probe = 0.f;       // this path tests and replaces every value it reads
    return Affine2{aG, double(bG), aR, double(bR)};
}

// The composite map of the thread's run.  When a reward or value of the run is a NaN or an infinity
// the thread overwrites it with 0 in the tile image (its own slots only: nobody else writes them,
// and a neighbour that reads the first of them as the value after ITS run replaces it on the fly
// too), reports it when the position lies inside a segment, and evaluates the run again.
__device__ __forceinline__ Affine2 egae_run_map(const EgaeArgs& a, TileBuf& buf, const TileWin& win,
                                                int64_t t0, int n_tile, int tid, RunState& rs,
                                                bool& bad, bool& nonfinite) {
    Affine2 f = identity2();
#pragma unroll 1
    for (int attempt = 0; attempt < 2; ++attempt) {
        float probe = 0.f;
        f = egae_run_map_once(a, buf, win, t0, n_tile, tid, rs, bad, probe, nonfinite);
        if (probe == probe) break;
        const uint32_t inside = rs.fast ? kRunMask : rs.inside;
#pragma unroll 1
        for (int k = 0; k < kScanItems; ++k) {
            const int sl = pos_slot(tid * kScanItems + k);
            const bool fr = finite_f32(buf.r[sl]), fv = finite_f32(buf.v[sl]);
            if (!fr) buf.r[sl] = 0.f;
            if (!fv) buf.v[sl] = 0.f;
            if ((!fr || !fv) && ((inside >> k) & 1u)) nonfinite = true;
        }
    }
    return f;
}

// Four results of one chunk: into the tile image itself (advantages over the values, returns over
// the rewards; a TMA store takes them to global memory) or straight to global memory.
__device__ __forceinline__ void egae_put4(const EgaeArgs& a, TileBuf& buf, bool in_place, int s,
                                          int64_t pos, int n_left, bool vec, const float (&oa)[4],
                                          const float (&og)[4]) {
    if (in_place) {
        *reinterpret_cast<float4*>(buf.v + s) = make_float4(oa[0], oa[1], oa[2], oa[3]);
        if (a.ret) *reinterpret_cast<float4*>(buf.r + s) = make_float4(og[0], og[1], og[2], og[3]);
    } else if (vec && n_left >= 4) {
        *reinterpret_cast<float4*>(a.adv + pos) = make_float4(oa[0], oa[1], oa[2], oa[3]);
        if (a.ret) *reinterpret_cast<float4*>(a.ret + pos) = make_float4(og[0], og[1], og[2], og[3]);
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (e < n_left) {
                a.adv[pos + e] = oa[e];
                if (a.ret) a.ret[pos + e] = og[e];
            }
        }
    }
}

// Replays the thread's positions from the values entering its run and stores the results.
__device__ __forceinline__ void egae_run_replay(const EgaeArgs& a, TileBuf& buf,
                                                const TileWin& win, int64_t t0,
                                                int n_tile, int tid, const RunState& rs, float G,
                                                float R, bool in_place, bool& bad, bool& nonfinite) {
    const int l0 = tid * kScanItems;
    if (rs.fast) {
        const int row_base = (tid / kThreadsPerRow) << 5;
        const int chunk0 = (tid % kThreadsPerRow) * kScanChunks, swz = (tid / kThreadsPerRow) & 7;
        float vn = rs.v_right;
#pragma unroll
        for (int q = kScanChunks - 1; q >= 0; --q) {
            const int s = row_base + (((chunk0 + q) ^ swz) << 2);
            const float4 r4 = *reinterpret_cast<const float4*>(buf.r + s);
            const float4 v4 = *reinterpret_cast<const float4*>(buf.v + s);
            const float rr[4] = {r4.x, r4.y, r4.z, r4.w};
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
            float oa[4], og[4];
#pragma unroll
            for (int e = 3; e >= 0; --e) {
                const float x = fmaf(a.c1, vn, rr[e]);
                G = fmaf(a.gl_hi, G, fmaf(a.gl_lo, G, x));
                R = fmaf(a.gamma_f, R, rr[e]);
                vn = vv[e];
                oa[e] = G - vn;
                og[e] = R;
            }
            egae_put4(a, buf, in_place, s, t0 + l0 + 4 * q, 4, a.vec_ok != 0, oa, og);
        }
        return;
    }
    if (rs.masked) {
        const int row_base = (tid / kThreadsPerRow) << 5;
        const int chunk0 = (tid % kThreadsPerRow) * kScanChunks, swz = (tid / kThreadsPerRow) & 7;
        const uint32_t inside = rs.inside, cont = rs.cont;
        float vn = rs.v_right;
#pragma unroll
        for (int q = kScanChunks - 1; q >= 0; --q) {
            const int s = row_base + (((chunk0 + q) ^ swz) << 2);
            const float4 r4 = *reinterpret_cast<const float4*>(buf.r + s);
            const float4 v4 = *reinterpret_cast<const float4*>(buf.v + s);
            const float rr[4] = {r4.x, r4.y, r4.z, r4.w};
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
            float oa[4], og[4];
#pragma unroll
            for (int e = 3; e >= 0; --e) {
                const int k = 4 * q + e;
                const bool in = (inside >> k) & 1u, c = (cont >> k) & 1u;
                float x = fmaf(a.c1, vn, rr[e]);
                if (k == rs.k_last) x = fmaf(a.gamma_f, rs.boundary_own ? vv[e] : rs.v_boundary, rr[e]);
                x = in ? x : 0.f;
                const float re = in ? rr[e] : 0.f;
                G = c ? fmaf(a.gl_hi, G, fmaf(a.gl_lo, G, x)) : x;
                R = c ? fmaf(a.gamma_f, R, re) : re;
                vn = vv[e];
                oa[e] = in ? G - vn : 0.f;
                og[e] = R;
            }
            egae_put4(a, buf, in_place, s, t0 + l0 + 4 * q, n_tile - (l0 + 4 * q), a.vec_ok != 0, oa, og);
        }
        return;
    }
    const int win_lo = win.win_lo;
    const bool win_smem = max(win.win_hi - win_lo, 0) <= kSegCap;
    int i = rs.i_start;
    float v_next = rs.v_right;
#pragma unroll 1
    for (int k = kScanItems - 1; k >= 0; --k) {
        const int l = l0 + k;
        const PosTerm t = egae_position(a, buf, win, t0, n_tile, win_lo, win_smem, l, v_next, i, bad, nonfinite);
        v_next = buf.v[pos_slot(l)];
        G = t.cont ? fmaf(a.gl_hi, G, fmaf(a.gl_lo, G, t.x)) : t.x;
        R = t.cont ? fmaf(a.gamma_f, R, t.r) : t.r;
        const float adv = t.inside ? G - t.v : 0.f;
        if (in_place) {
            buf.v[pos_slot(l)] = adv;
            if (a.ret) buf.r[pos_slot(l)] = R;
        } else if (l < n_tile) {
            a.adv[t0 + l] = adv;
            if (a.ret) a.ret[t0 + l] = R;
        }
    }
}

// One CTA per tile, from the END of the arrays backwards, so the tiles a tile looks back at (those
// to its right) were started earlier and are running or done.  A tile is kScanParts parts of 2048
// positions (one by default); a thread owns one run of sixteen positions in every part.  The
// latencies of a tile (copy, segment window, look-back) are covered by the other CTAs resident on
// the SM.  A whole part's results are written over its inputs in shared memory and leave by TMA stores.
//
// Measured at 17.5 M tokens against this form (81 us per call), and dropped:
//  - two parts per tile (the same 128 threads map the right part, then the left part, then one
//    publication and one look-back per 4096 positions; six tiles per SM): 95 us;
//  - resident CTAs that take tile after tile by ticket, (a) with two tile images, the look-back for
//    tile k-1 after the maps of tile k: 92 us -- the copy of tile k+1 cannot start before the replay
//    of tile k-1 has left its image, so every step waits for a copy; (b) with three images and
//    specialised warps (four compute warps, a warp that looks back and publishes, a warp that moves
//    tiles, draws tickets and fetches windows), four CTAs per SM: 82 us, and 90 us when the look-back
//    warp runs ahead of the others -- the steps of the resident CTAs lock into one another through
//    the look-back, and each step then lasts as long as the slowest neighbour's.
// In-kernel clock stamps of a debug build: a tile lives about 20 k cycles (start to first barrier 2.6 k,
// window + copy 3.9 k, maps and warp scans 3.1 k, compose + publish 0.9 k, look-back 5.8 k, carries
// 0.9 k, replay + store 2.8 k); every variant above has fewer warps per SM in the two compute phases,
// and those run at one instruction per six cycles and warp.
#ifndef TPPO_SCAN_PARTS
#define TPPO_SCAN_PARTS 1
#endif
constexpr int kScanParts = TPPO_SCAN_PARTS;
constexpr int kScan2CtasPerSm = 6;
template <int H>
__global__ void __launch_bounds__(kScanThreads, H == 1 ? kScanCtasPerSm : kScan2CtasPerSm)
egae_scan_kernel(const EgaeArgs a, const __grid_constant__ CUtensorMap map_r,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_adv,
                 const __grid_constant__ CUtensorMap map_ret) {
    constexpr int kWarpsAll = H * kScanWarps;       // "warps" of the tile, left to right: part p, warp w -> p * 4 + w
    static_assert(kWarpsAll <= 32, "one lane per warp composite");
    __shared__ TileBuf buf[H];
    __shared__ TileWin win[H];
    __shared__ __align__(8) uint64_t s_bar[H];      // the part's inputs have arrived
#if TPPO_EGAE_TICKET
    __shared__ uint32_t s_ticket;
#endif
    __shared__ Affine2 s_warp[kWarpsAll];
    __shared__ double s_carry[kWarpsAll][2];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#if TPPO_EGAE_TICKET
    if (threadIdx.x == 0) {
        // the ticket counter starts at all-ones like the rest of the workspace: + 1 wraps the first
        // draw to ticket 0
        if (a.after_clear) asm volatile("griddepcontrol.wait;" ::: "memory");
        s_ticket = atomicAdd(a.ticket, 1u) + 1u;
    }
    __syncthreads();
    const uint32_t ticket = s_ticket;
#else
    const uint32_t ticket = blockIdx.x;
#endif
    // Thread 0 initialises the copy barriers and issues the copies at once; the other threads first
    // touch a barrier after the block-wide barrier below (one barrier less in every tile's life, and
    // the copies start that much earlier).
    if (threadIdx.x == 0) {
#pragma unroll
        for (int p = 0; p < H; ++p) ptx::mbar_init(ptx::smem_addr(&s_bar[p]), 1);
        ptx::fence_mbar_init_cluster();
    }
    if (ticket >= uint32_t(a.num_tiles)) return;       // (the grid has exactly num_tiles CTAs)
    const int tile = a.num_tiles - 1 - int(ticket);
    const int64_t tile0 = int64_t(tile) * (H * kScanTile);
    bool bad = false, nonfinite = false, copy_late = false;
    int n_part[H];
    bool by_tma[H];
#pragma unroll
    for (int p = 0; p < H; ++p) {
        const int64_t left = int64_t(a.N) - (tile0 + int64_t(p) * kScanTile);
        n_part[p] = int(max(int64_t(0), min(int64_t(kScanTile), left)));
        by_tma[p] = a.tma_ok && n_part[p] == kScanTile;
    }

    // ---- inputs: TMA copies for a whole part (rightmost first), plain loads for a ragged or unaligned one
    if (threadIdx.x == 0) {
#pragma unroll
        for (int p = H - 1; p >= 0; --p) {
            if (!by_tma[p]) continue;
            const uint32_t bar = ptx::smem_addr(&s_bar[p]);
            ptx::mbar_arrive_expect_tx(bar, 2 * kScanTile * uint32_t(sizeof(float)));
#pragma unroll
            for (int bx = 0; bx < kScanBoxes; ++bx) {
                const int32_t y = int32_t((tile0 + int64_t(p) * kScanTile) / kRowPos) + bx * kScanBoxRows;
                umma::tma_load_2d(ptx::smem_addr(buf[p].r + bx * kScanBoxRows * kRowPos), &map_r, bar, 0, y);
                umma::tma_load_2d(ptx::smem_addr(buf[p].v + bx * kScanBoxRows * kRowPos), &map_v, bar, 0, y);
            }
        }
    }
    // ... and asks for the inputs of the tile that a block a quarter wave later will take to be
    // brought into L2 now, so that its copy is served from there (tppo_egae at 17.5 M tokens: none
    // 81.0 us; 37 / 74 / 148 / 222 / 296 / 444 / 592 / 888 / 1184 / 2368 tiles ahead 77.0 / 76.3 / 76.2 /
    // 75.6-76.5 / 75.6-75.9 / 76.4 / 76.5-76.8 / 77.8 / 78.1 / 83.6)
#ifndef TPPO_SCAN_PREFETCH_TILES
#define TPPO_SCAN_PREFETCH_TILES (2 * kNumSms)
#endif
    if (threadIdx.x == 32 && a.tma_ok && TPPO_SCAN_PREFETCH_TILES > 0 && tile >= TPPO_SCAN_PREFETCH_TILES) {
        const int64_t q0 = int64_t(tile - TPPO_SCAN_PREFETCH_TILES) * (H * kScanTile);
        ptx::bulk_prefetch_l2(a.rewards + q0, H * kScanTile * uint32_t(sizeof(float)));
        ptx::bulk_prefetch_l2(a.values + q0, H * kScanTile * uint32_t(sizeof(float)));
    }
#pragma unroll
    for (int p = 0; p < H; ++p) {
        const int64_t t0 = tile0 + int64_t(p) * kScanTile;
        if (!by_tma[p]) {
            for (int k = threadIdx.x; k < n_part[p]; k += kScanThreads) {
                buf[p].r[pos_slot(k)] = __ldg(a.rewards + t0 + k);
                buf[p].v[pos_slot(k)] = __ldg(a.values + t0 + k);
            }
        }
        if (threadIdx.x == kScanThreads - 1)
            buf[p].v_after = (t0 + n_part[p] < a.N) ? __ldg(a.values + t0 + n_part[p]) : 0.f;
    }
    if (warp < H) {
        // warp p fetches the segment window of part p.  With a clearing kernel in front (which lets
        // this kernel start at once: programmatic dependent launch) the windows were found there:
        // its end is awaited here
        if (a.after_clear) asm volatile("griddepcontrol.wait;" ::: "memory");
        if (n_part[warp] > 0)
            bad |= egae_window(a, win[warp], tile0 + int64_t(warp) * kScanTile, n_part[warp], lane, nonfinite,
                               a.after_clear ? a.state[tile].win + 2 * warp : nullptr);
    }
    __syncthreads();
    if (by_tma[H - 1] && !ptx::mbar_wait<false>(ptx::smem_addr(&s_bar[H - 1]), 0)) copy_late = true;

    // ---- per part, right to left: the thread's sixteen positions, right to left: its composite map;
    //      the warp's scan
    RunState rs[H];
#pragma unroll
    for (int p = H - 1; p >= 0; --p) {
        if (p < H - 1 && by_tma[p] && !ptx::mbar_wait<false>(ptx::smem_addr(&s_bar[p]), 0)) copy_late = true;
        rs[p] = RunState{};
        Affine2 S = identity2();
        if (n_part[p] > 0) {
            S = egae_run_map(a, buf[p], win[p], tile0 + int64_t(p) * kScanTile, n_part[p], threadIdx.x, rs[p],
                             bad, nonfinite);
            // inclusive suffix composition inside the warp: S_l = f_l o f_{l+1} o ... o f_31
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const Affine2 o = shfl_down(S, d);
                if (lane + d < 32) S = compose(S, o);
            }
        }
        rs[p].excl = shfl_down(S, 1);   // composite of the lanes to the right
        if (lane == 31) rs[p].excl = identity2();
        if (lane == 0) s_warp[p * kScanWarps + warp] = S;
    }
    // Everything above read inputs only (and the windows).  The status word and the tile states are
    // cleared by the kernel in front: its end is awaited here by every thread, before the first word
    // of either is touched.
    if (a.after_clear) asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();                                                      // (A)

    // ---- tile composite, look-back, per-warp carries (warp 0) ------------------------------------
    if (warp == 0) {
        // lane j < kWarpsAll holds the composite of "warp" j; suffix-compose them, so that lane j
        // ends with W_j o ... o W_last and lane 0 with the tile's composite
        Affine2 W = lane < kWarpsAll ? s_warp[lane] : identity2();
#pragma unroll
        for (int d = 1; d < kWarpsAll; d <<= 1) W = compose(W, shfl_down(W, d));
        Affine2 right = shfl_down(W, 1);            // composite of the warps to the right
        if (lane >= kWarpsAll - 1) right = identity2();
        TileState* st = a.state;
        const bool publish = lane == 0 && !a.no_publish;
        if (publish && tile + 1 < a.num_tiles) {
            st_pair(st[tile].aggA, W.aA, W.bA);
            st_pair(st[tile].aggR, W.aR, W.bR);
        }
        double xA = 0.0, xR = 0.0;
        const bool ok = egae_look_back(a, tile + 1, lane, xA, xR);
        if (lane == 0) {
            if (!ok) { egae_raise(a, TPPO_DEV_WAIT_TIMEOUT); xA = 0.0; xR = 0.0; }
            if (publish) st_pair(st[tile].inc, fma(W.aA, xA, W.bA), fma(W.aR, xR, W.bR));
        }
        xA = __shfl_sync(0xffffffffu, xA, 0);
        xR = __shfl_sync(0xffffffffu, xR, 0);
        if (lane < kWarpsAll) {
            s_carry[lane][0] = fma(right.aA, xA, right.bA);
            s_carry[lane][1] = fma(right.aR, xR, right.bR);
        }
    }
    __syncthreads();                                                      // (B)

    // ---- replay the thread's positions from the true incoming values, store -----------------------
#pragma unroll
    for (int p = H - 1; p >= 0; --p) {
        if (n_part[p] <= 0) continue;
        const double* c = s_carry[p * kScanWarps + warp];
        const float G = float(fma(rs[p].excl.aA, c[0], rs[p].excl.bA));
        const float R = float(fma(rs[p].excl.aR, c[1], rs[p].excl.bR));
        egae_run_replay(a, buf[p], win[p], tile0 + int64_t(p) * kScanTile, n_part[p], threadIdx.x, rs[p], G, R,
                        by_tma[p], bad, nonfinite);
    }
    if (bad) egae_raise(a, TPPO_DEV_BAD_SEGMENT);
    if (nonfinite) egae_raise(a, TPPO_DEV_NONFINITE);
    if (copy_late) egae_raise(a, TPPO_DEV_WAIT_TIMEOUT);
    bool any_tma = false;
#pragma unroll
    for (int p = 0; p < H; ++p) any_tma |= by_tma[p];
    if (any_tma) {
        ptx::fence_proxy_async_smem();       // the TMA stores read what was just written
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int p = 0; p < H; ++p) {
                if (!by_tma[p]) continue;
#pragma unroll
                for (int bx = 0; bx < kScanBoxes; ++bx) {
                    const int32_t y = int32_t((tile0 + int64_t(p) * kScanTile) / kRowPos) + bx * kScanBoxRows;
                    umma::tma_store_2d(&map_adv, ptx::smem_addr(buf[p].v + bx * kScanBoxRows * kRowPos), 0, y);
                    if (a.ret) umma::tma_store_2d(&map_ret, ptx::smem_addr(buf[p].r + bx * kScanBoxRows * kRowPos), 0, y);
                }
            }
            ptx::bulk_commit();
            ptx::bulk_wait_read<0>();   // shared memory must outlive the stores' reads of it
        }
    }
}

bool make_f32_rows_tensor_map(CUtensorMap* map, const void* base, uint64_t rows);
uint32_t test_spin_limit(uint32_t normal);
int32_t test_no_publish();

// Fills the constants derived from gamma and lambda and the tensor maps, then launches one CTA per
// tile.  The caller has set the pointers, sizes, state and ticket.
constexpr size_t kScanHeadBytes = 256;      // the ticket counter

// Number of entries of the ascending array arr[0..n) that are <= key.
template <bool LDG>
__device__ __forceinline__ int count_le(const int32_t* __restrict__ arr, int n, int32_t key) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((LDG ? __ldg(arr + mid) : arr[mid]) <= key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Launched just before the scan, which is its programmatic dependent and starts beside it: status
// word to 0, ticket counter to all-ones, and one thread per tile sets the tile's state to unset
// (all-ones) and finds the segment window of each of its parts, so that the scan reads a window instead of
// searching for it: the search (three dependent rounds of global loads by one warp) was the longest
// latency of a tile's first phase, longer than the copy of its inputs.  Here a block first copies the
// segment bounds into shared memory (2 x 4 x B bytes, one round of loads) and searches there; bounds
// that do not fit are searched in global memory.
constexpr int kClearThreads = 256;
constexpr int kClearSmemMaxB = 12288;       // 96 KB of segment bounds
__global__ void __launch_bounds__(kClearThreads) egae_clear_kernel(int32_t* status, uint4* head,
                                                                   TileState* state, int num_tiles,
                                                                   const int32_t* seg_begin,
                                                                   const int32_t* seg_end, int B,
                                                                   int64_t N, int in_smem, int parts) {
    extern __shared__ __align__(16) int32_t s_bounds[];      // seg_end[0..B), seg_begin[0..B)
    asm volatile("griddepcontrol.launch_dependents;");
    const int tile = blockIdx.x * blockDim.x + threadIdx.x;
    if (tile == 0) *status = 0;
    if (tile < int(kScanHeadBytes / 16)) head[tile] = make_uint4(~0u, ~0u, ~0u, ~0u);
    if (in_smem) {
        // 16-byte loads where the arrays allow it, all of a thread's loads in flight together
        const bool vec = ((reinterpret_cast<uintptr_t>(seg_end) | reinterpret_cast<uintptr_t>(seg_begin)) & 15) == 0 &&
                         (B & 3) == 0;
        if (vec) {
            const int4* e4 = reinterpret_cast<const int4*>(seg_end);
            const int4* b4 = reinterpret_cast<const int4*>(seg_begin);
            int4* se = reinterpret_cast<int4*>(s_bounds);
            int4* sb = reinterpret_cast<int4*>(s_bounds + B);
#pragma unroll 4
            for (int i = threadIdx.x; i < B / 4; i += kClearThreads) {
                se[i] = __ldg(e4 + i);
                sb[i] = __ldg(b4 + i);
            }
        } else {
            for (int i = threadIdx.x; i < B; i += kClearThreads) {
                s_bounds[i] = __ldg(seg_end + i);
                s_bounds[B + i] = __ldg(seg_begin + i);
            }
        }
        __syncthreads();
    }
    if (tile >= num_tiles) return;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    for (int p = 0; p < parts; ++p) {       // parts <= 2
        const int64_t t0 = (int64_t(tile) * parts + p) * kScanTile;
        if (t0 >= N) break;
        const int64_t t_last = min(t0 + kScanTile, N) - 1;
        w[2 * p] = uint32_t(in_smem ? count_le<false>(s_bounds, B, int32_t(t0)) : count_le<true>(seg_end, B, int32_t(t0)));
        w[2 * p + 1] = uint32_t(in_smem ? count_le<false>(s_bounds + B, B, int32_t(t_last))
                                        : count_le<true>(seg_begin, B, int32_t(t_last)));
    }
    uint4* st = reinterpret_cast<uint4*>(state + tile);
    st[0] = make_uint4(~0u, ~0u, ~0u, ~0u);
    st[1] = make_uint4(~0u, ~0u, ~0u, ~0u);
    st[2] = make_uint4(~0u, ~0u, ~0u, ~0u);
    st[3] = make_uint4(w[0], w[1], w[2], w[3]);
}



static int egae_launch(EgaeArgs& a, float gamma, float lambda, cudaStream_t s) {
    constexpr int parts = kScanParts;
    a.num_tiles = int32_t((int64_t(a.N) + parts * kScanTile - 1) / (parts * kScanTile));
    a.gamma = double(gamma);
    a.gl = double(gamma) * double(lambda);
    a.gamma_run = 1.0; a.gl_run = 1.0;
    for (int k = 0; k < kScanItems; ++k) { a.gamma_run *= a.gamma; a.gl_run *= a.gl; }
    a.gamma_f = gamma;
    a.gl_hi = float(a.gl);
    a.gl_lo = float(a.gl - double(a.gl_hi));
    a.c1_d = double(gamma) * (1.0 - double(lambda));
    a.c1 = float(a.c1_d);
    a.vec_ok = aligned(a.rewards, 16) && aligned(a.values, 16) && aligned(a.adv, 16) &&
               (!a.ret || aligned(a.ret, 16));
    CUtensorMap map_r, map_v, map_adv, map_ret;
    memset(&map_r, 0, sizeof(map_r));
    memset(&map_v, 0, sizeof(map_v));
    memset(&map_adv, 0, sizeof(map_adv));
    memset(&map_ret, 0, sizeof(map_ret));
    // whole tiles exist only from 2048 positions on; without the driver's encoder (or with
    // unaligned arrays) every tile takes the plain-load path
    a.tma_ok = a.vec_ok && a.N >= kScanTile &&
               make_f32_rows_tensor_map(&map_r, a.rewards, uint64_t(a.N) / kRowPos) &&
               make_f32_rows_tensor_map(&map_v, a.values, uint64_t(a.N) / kRowPos) &&
               make_f32_rows_tensor_map(&map_adv, a.adv, uint64_t(a.N) / kRowPos) &&
               (!a.ret || make_f32_rows_tensor_map(&map_ret, a.ret, uint64_t(a.N) / kRowPos));
    a.spin_limit = test_spin_limit(kScanSpinLimit);
    a.no_publish = test_no_publish();
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(a.num_tiles));
    cfg.blockDim = dim3(kScanThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = a.after_clear ? 1 : 0;
    TPPO_CUDA_CHECK(cudaLaunchKernelEx(&cfg, egae_scan_kernel<kScanParts>, a, map_r, map_v, map_adv, map_ret));
    return TPPO_OK;
}

size_t egae_workspace_bytes(int64_t N) {
    const int64_t tiles = (N + kScanTile - 1) / kScanTile;
    return kScanHeadBytes + align_up(size_t(tiles > 0 ? tiles : 1) * sizeof(TileState), kWsAlign);
}
static void egae_carve(EgaeArgs& a, void* ws) {
    a.ticket = static_cast<uint32_t*>(ws);
    a.state = reinterpret_cast<TileState*>(static_cast<char*>(ws) + kScanHeadBytes);
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
    if (N == 0) {
        TPPO_CUDA_CHECK(cudaMemsetAsync(status, 0, sizeof(int32_t), s));
        return TPPO_OK;
    }
    // Tile states start out unset (all-ones), the ticket counter at all-ones too, the status at 0:
    // one small kernel writes them, and the scan starts beside it as its programmatic dependent,
    // copying tiles in and composing maps until it first needs either.  (Two memsets in front of a
    // plain launch cost about 5 us more at 17.5 M tokens; letting the last tile to finish hand over
    // the status bits, to save the clear altogether, cost 9 us for the fence and counter at every
    // tile's end.)
    {
        static_assert(kScanHeadBytes / 16 <= kClearThreads, "the first block writes the head");
        constexpr int parts = kScanParts;
        const int tiles = int((N + parts * kScanTile - 1) / (parts * kScanTile));
        const int in_smem = B <= kClearSmemMaxB;
        const size_t smem = in_smem ? size_t(2) * size_t(B) * sizeof(int32_t) : 0;
        if (smem > 48 * 1024)       // (an attribute of the function on the current device; the call is cheap)
            TPPO_CUDA_CHECK(cudaFuncSetAttribute(egae_clear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 2 * kClearSmemMaxB * int(sizeof(int32_t))));
        egae_clear_kernel<<<(tiles + kClearThreads - 1) / kClearThreads, kClearThreads, smem, s>>>(
            status, static_cast<uint4*>(workspace),
            reinterpret_cast<TileState*>(static_cast<char*>(workspace) + kScanHeadBytes), tiles,
            seg_begin, seg_end, B, N, in_smem, parts);
        TPPO_CUDA_CHECK(cudaGetLastError());
    }
    EgaeArgs a{};
    a.after_clear = 1;
    a.rewards = rewards; a.values = values; a.seg_begin = seg_begin; a.seg_end = seg_end;
    a.truncated = truncated; a.bootstrap = bootstrap; a.B = B; a.N = int32_t(N);
    a.adv = advantages; a.ret = returns; a.status = status;
    egae_carve(a, workspace);
    return egae_launch(a, gamma, lambda, s);
}

// ---- allocation-free variant ------------------------------------------------------------------
// For callers that can neither allocate device memory nor lend a workspace (a plug-in inside a
// runtime that owns the whole device's memory pool; a latency-critical section that must avoid
// cudaMalloc's device-wide synchronisation).  The tile descriptors and the ticket counter live in
// this fixed device array; each GPU that loads the library keeps it until the process ends.
namespace tppo {
constexpr int64_t kStaticMaxTokens = TPPO_EGAE_STATIC_MAX_TOKENS;
constexpr size_t kStaticTiles = size_t((kStaticMaxTokens + kScanTile - 1) / kScanTile);
constexpr size_t kStaticScratchBytes = kScanHeadBytes + kStaticTiles * sizeof(TileState);
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
    EgaeArgs a{};
    a.rewards = rewards; a.values = values; a.seg_begin = seg_begin; a.seg_end = seg_end;
    a.truncated = truncated; a.bootstrap = bootstrap; a.B = B; a.N = int32_t(N);
    a.adv = advantages; a.ret = returns; a.status = status;
    egae_carve(a, scratch);
    // the array still holds the previous call's tile states and ticket: reset the part this call
    // uses to the all-ones pattern (tile states unset, ticket counter one draw before ticket 0)
    const size_t tiles = size_t((N + kScanTile - 1) / kScanTile);
    TPPO_CUDA_CHECK(cudaMemsetAsync(scratch, 0xff, kScanHeadBytes + tiles * sizeof(TileState), s));
    return egae_launch(a, gamma, lambda, s);
}

// Shared-memory-resident policy-loss kernel for bf16 logits (the throughput kernel).
//
// A thread-block cluster of C CTAs owns one selected logits row at a time; CTA c owns the c-th
// contiguous slice of the row.  Each slice is brought into shared memory once by 1-D bulk (TMA)
// copies issued by a dedicated producer warp into a ring of STAGES slice buffers, so the copies of
// the next rows are in flight while the current row is being worked on.  The 15 compute warps pull
// their 16-byte units of the slice into registers, form a thread-local maximum and the
// exponentials relative to it (one ex2 per logit, kept in registers as fp32), and reduce
// (max, sum, target logit) over the warp and -- through asynchronous distributed-shared-memory
// stores that count bytes on the receiver's mbarrier -- the cluster.  With the row's log-sum-exp known every thread evaluates
// Eq. 1 of the paper (ratio, clip, loss term, gradient factor), rescales its stored exponentials
// into  factor * (softmax - onehot),  rounds once to bf16 and stores the result: either straight
// from registers with 128-bit global stores (default; the stage buffer is then free as soon as
// the row is in registers), or over its slice in shared memory, from where the producer warp sends
// it out with bulk stores.  Each logit crosses the HBM interface exactly once in each direction.
// No multicast is used: every CTA issues plain copies of its own slice.
//
// Thirty-three clusters of four fill 132 of the 148 SMs.  On large row lists the host gives the
// last rows of the list to the plain two-pass kernel, launched as a programmatic dependent of this
// one, so that it runs on the remaining SMs at the same time (policy_loss.cu).
#include "policy_common.cuh"
#include "ptx.cuh"


namespace tppo {

constexpr int kClComputeWarps = 15;
constexpr int kClComputeThreads = kClComputeWarps * 32;      // 480
constexpr int kClThreads = kClComputeThreads + 32;           // + producer warp
constexpr int kClMaxUnits = 10;                              // 16-byte units per thread per slice
constexpr int kClMaxStages = 4;
constexpr int kClMaxCluster = 8;
constexpr int kClMaxParts = kClMaxCluster * kClComputeWarps; // warp partials a CTA receives per row
constexpr uint32_t kClCtlBytes = 4096;                       // control block ahead of the stages
constexpr uint32_t kClCopyChunk = 1u << 17;                  // bytes per bulk copy instruction
constexpr uint32_t kNegInfPair = 0xff80ff80u;                // two bf16 -inf

struct ClusterCtl {
    unsigned long long full[kClMaxStages];   // slice landed in shared memory (tx-count barrier)
    unsigned long long done[kClMaxStages];   // compute warps are finished with the stage
    unsigned long long xchg[2];              // all (max, sum) partials of the row have arrived
    float2 part[2][kClMaxParts];             // (max, sum) of every compute warp of the cluster
    float xy[2];                             // the row's target logit, sent by the thread that owns it
};
static_assert(sizeof(ClusterCtl) <= kClCtlBytes, "control block too large");

struct ClusterLaunch {
    uint32_t stages;
    uint32_t stage_stride;   // bytes between stage buffers (multiple of 128)
};

// OUT: 0 = forward only, 1 = gradient via shared memory + bulk stores, 2 = gradient straight from registers
template <int C, int OUT>
__global__ void __launch_bounds__(kClThreads, 1)
policy_cluster_kernel(const PolicyArgs a, const ClusterLaunch cfg) {
    extern __shared__ __align__(1024) uint8_t smem[];
    ClusterCtl* ctl = reinterpret_cast<ClusterCtl*>(smem);
    const uint32_t stage0 = ptx::smem_addr(smem) + kClCtlBytes;

    const uint32_t rank = ptx::cluster_ctarank();
    const int32_t cid = int32_t(ptx::cluster_id_x()), ncl = int32_t(ptx::num_clusters_x());
    // The rest of the device (the SMs that cannot host one more cluster) may work on the tail of the
    // row list at the same time: a kernel launched as a programmatic dependent of this one starts as
    // soon as every CTA here has passed this point.
    asm volatile("griddepcontrol.launch_dependents;");
    const int32_t n = int32_t(policy_n(a));
    int64_t part_lo, part_hi;
    policy_part(a, n, part_lo, part_hi);
    const int32_t n_rows = int32_t(part_hi);                        // this launch: entries [0, n_rows)
    const int32_t n_it = n_rows > cid ? (n_rows - cid + ncl - 1) / ncl : 0;   // rows j = cid + it * ncl
    const uint32_t S = cfg.stages;
    constexpr bool GRAD = OUT != 0;
    constexpr bool STAGED = OUT == 1;   // the stage buffer also stages the gradient

    // this CTA's slice of every row, in 16-byte units
    const uint32_t units_total = uint32_t(a.V) >> 3;
    const uint32_t u0 = uint32_t(uint64_t(rank) * units_total / C);
    const uint32_t u1 = uint32_t(uint64_t(rank + 1) * units_total / C);
    const uint32_t nu = u1 - u0;
    const uint32_t slice_bytes = nu * 16u;

    const int tid = threadIdx.x;
    if (tid == 0) {
        for (uint32_t s = 0; s < kClMaxStages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->done[s]), kClComputeWarps);
        }
        ptx::mbar_init(ptx::smem_addr(&ctl->xchg[0]), 1);
        ptx::mbar_init(ptx::smem_addr(&ctl->xchg[1]), 1);
        ptx::fence_mbar_init_cluster();
    }
    ptx::cluster_sync_all();   // barriers of every CTA are initialised before any remote signal

    const uint8_t* logits = static_cast<const uint8_t*>(a.logits);
    uint8_t* dl = static_cast<uint8_t*>(a.dlogits);

    if (tid >= kClComputeThreads) {
        // ===================== producer warp: all bulk copies of this CTA =====================
        if (tid == kClComputeThreads) {
            int32_t issued = 0;
            auto issue_load = [&](int32_t it) {
                const uint32_t st = uint32_t(it) % S;
                const int64_t j = int64_t(cid) + int64_t(it) * ncl;
                const int64_t r = __ldg(&a.rec[j].row);
                const uint32_t bar = ptx::smem_addr(&ctl->full[st]);
                if (r >= 0 && slice_bytes > 0) {
                    ptx::mbar_arrive_expect_tx(bar, slice_bytes);
                    const uint8_t* src = logits + (r * a.ld) * 2 + uint64_t(u0) * 16u;
                    const uint32_t dst = stage0 + st * cfg.stage_stride;
                    for (uint32_t off = 0; off < slice_bytes; off += kClCopyChunk) {
                        const uint32_t len = min(kClCopyChunk, slice_bytes - off);
                        ptx::bulk_load(dst + off, src + off, len, bar);
                    }
                } else {
                    ptx::mbar_arrive(bar);   // nothing to read: complete the phase directly
                }
                issued = it + 1;
            };
            const int32_t pro = n_it < int32_t(S) ? n_it : int32_t(S);
            for (int32_t it = 0; it < pro; ++it) issue_load(it);

            bool ok = true;
            uint32_t st = 0, ph = 0;
            for (int32_t it = 0; it < n_it; ++it) {
                ok = ptx::mbar_wait<false>(ptx::smem_addr(&ctl->done[st]), ph);
                if (!ok) break;
                if (STAGED) {
                    const int64_t j = int64_t(cid) + int64_t(it) * ncl;
                    uint8_t* dst = nullptr;
                    if (a.mode == TPPO_DLOGITS_COMPACT) {
                        dst = dl + (j * int64_t(a.V)) * 2;
                    } else {
                        const int64_t r = __ldg(&a.rec[j].row);
                        if (r >= 0) dst = dl + (r * a.ld) * 2;
                    }
                    if (dst && slice_bytes > 0) {
                        dst += uint64_t(u0) * 16u;
                        const uint32_t src = stage0 + st * cfg.stage_stride;
                        for (uint32_t off = 0; off < slice_bytes; off += kClCopyChunk) {
                            const uint32_t len = min(kClCopyChunk, slice_bytes - off);
                            ptx::bulk_store(dst + off, src + off, len);
                        }
                    }
                    ptx::bulk_commit();
                    if (S == 1) {
                        ptx::bulk_wait_read<0>();             // single buffer: drain, then refill
                        if (it + 1 < n_it) issue_load(it + 1);
                    } else if (it >= 1) {
                        ptx::bulk_wait_read<1>();             // the store of row it-1 has left smem
                        if (it - 1 + int32_t(S) < n_it) issue_load(it - 1 + int32_t(S));
                    }
                } else {
                    if (it + int32_t(S) < n_it) issue_load(it + int32_t(S));   // the row is in registers
                }
                if (++st == S) { st = 0; ph ^= 1u; }
            }
            if (!ok) {
                atomicOr(a.stats + 3, TPPO_DEV_WAIT_TIMEOUT);
                // let the copies that are still in flight into this CTA's shared memory land
                const int32_t first = issued > int32_t(S) ? issued - int32_t(S) : 0;
                for (int32_t it = first; it < issued; ++it)
                    ptx::mbar_wait<false>(ptx::smem_addr(&ctl->full[uint32_t(it) % S]), (uint32_t(it) / S) & 1u);
            }
            ptx::bulk_wait<0>();
        }
        __syncwarp();
    } else {
        // ================================ compute warps ======================================
        const int lane = tid & 31, warp = tid >> 5;
        const float inv_denom = policy_inv_denom(a, n);
        constexpr uint32_t kPartBytes = uint32_t(C) * kClComputeWarps * 8u;   // partials per row
        RowRec rec_next;
        rec_next.row = -1; rec_next.y = -1; rec_next.adv = 0.f; rec_next.old_logp = 0.f;
        if (n_it > 0) rec_next = load_rec(a.rec + cid);
        bool ok = true;
        uint32_t st = 0, ph = 0;
        for (int32_t it = 0; it < n_it; ++it) {
            const int64_t j = int64_t(cid) + int64_t(it) * ncl;
            const RowRec rec = rec_next;
            const bool row_ok = rec.row >= 0, rec_ok = rec.y >= 0;
            const uint32_t par = uint32_t(it) & 1u, xph = (uint32_t(it) >> 1) & 1u;
            if (tid == 0)   // this row's exchange: C*15 warp partials (+ the target logit)
                ptx::mbar_arrive_expect_tx(ptx::smem_addr(&ctl->xchg[par]), kPartBytes + (rec_ok ? 4u : 0u));
            if (it + 1 < n_it) rec_next = load_rec(a.rec + j + ncl);   // one row ahead, used next turn
            // (warp-uniform: a wait that runs out takes the whole warp to the exit together)
            if (!ptx::mbar_wait_warp<false>(ptx::smem_addr(&ctl->full[st]), ph)) { ok = false; break; }

            // ---- slice -> registers ------------------------------------------------------
            const uint32_t sbase = stage0 + st * cfg.stage_stride;
            uint4 xw[kClMaxUnits];
#pragma unroll
            for (int k = 0; k < kClMaxUnits; ++k) {
                const uint32_t u = uint32_t(tid) + uint32_t(k) * kClComputeThreads;
                xw[k] = (u < nu && row_ok) ? ptx::lds128(sbase + u * 16u)
                                                : make_uint4(kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair);
            }
            // the target logit, if it lies in one of this thread's units
            const int32_t yu = (rec.y >> 3) - int32_t(u0);
            const bool y_mine = rec_ok && yu >= 0 && yu < int32_t(nu) && (yu % kClComputeThreads) == tid;
            const uint32_t y_off = uint32_t(yu) * 16u + uint32_t(rec.y & 7) * 2u;   // within the slice
            const uint32_t y_addr = sbase + y_off;
            float x_y = 0.f;
            if (y_mine) x_y = __uint_as_float(uint32_t(ptx::lds_u16(y_addr)) << 16);
            if (!STAGED) {   // the stage can be refilled as soon as every warp holds its units
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->done[st]));
            }
            // ---- thread-local max (packed bf16 max, then widen) --------------------------------
            uint32_t pm = kNegInfPair;
#pragma unroll
            for (int k = 0; k < kClMaxUnits; ++k) {
                pm = ptx::max_bf16x2(pm, ptx::max_bf16x2(ptx::max_bf16x2(xw[k].x, xw[k].y),
                                                         ptx::max_bf16x2(xw[k].z, xw[k].w)));
            }
            float m_t = fmaxf(bf16_lo(pm), bf16_hi(pm));
            // a thread with no unit, or whose logits are all -inf (masked): the most negative finite
            // float keeps x - m_t free of inf - inf; every finite bf16 lies above it
            m_t = fmaxf(m_t, -kFltMax);
            // ---- exponentials relative to the thread-local max, kept in registers ---------
            // exp(x - m) = 2^((x - m) * log2 e): the difference first, so that logits of any finite
            // magnitude stay in range (m * log2 e alone overflows beyond 2.3e38)
            // (two fp32 lanes per instruction: packed ADD / MUL halve the issue slots)
            uint64_t e2[kClMaxUnits][4];
            uint64_t s2 = ptx::pack_f32x2(0.f, 0.f);
            const uint64_t k2 = ptx::pack_f32x2(kLog2e, kLog2e), o2 = ptx::pack_f32x2(-m_t, -m_t);
#pragma unroll
            for (int k = 0; k < kClMaxUnits; ++k) {
                const uint32_t w[4] = {xw[k].x, xw[k].y, xw[k].z, xw[k].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float t0, t1;
                    ptx::unpack_f32x2(ptx::mul_f32x2(ptx::add_f32x2(ptx::pack_f32x2(bf16_lo(w[q]), bf16_hi(w[q])), o2), k2), t0, t1);
                    e2[k][q] = ptx::pack_f32x2(ex2(t0), ex2(t1));
                    s2 = ptx::add_f32x2(s2, e2[k][q]);
                }
            }
            float s_t;
            {
                float sa, sb;
                ptx::unpack_f32x2(s2, sa, sb);
                s_t = sa + sb;
            }
            // ---- warp partial -> every CTA of the cluster (asynchronous remote stores that count
            //      bytes on the receiver's barrier: no fence, no second hop) ----------------------
            const float wm = warp_max(m_t);
            const float ws = warp_sum(s_t * ex2((m_t - wm) * kLog2e));
            if (lane < C) {
                const uint32_t slot = ptx::smem_addr(&ctl->part[par][rank * kClComputeWarps + warp]);
                ptx::st_async_f32x2(ptx::map_to_cta(slot, lane), wm, ws,
                                    ptx::map_to_cta(ptx::smem_addr(&ctl->xchg[par]), lane));
            }
            if (y_mine) {
#pragma unroll
                for (int c = 0; c < C; ++c)
                    ptx::st_async_f32(ptx::map_to_cta(ptx::smem_addr(&ctl->xy[par]), c), x_y,
                                      ptx::map_to_cta(ptx::smem_addr(&ctl->xchg[par]), c));
            }
            if (!ptx::mbar_wait_warp<true>(ptx::smem_addr(&ctl->xchg[par]), xph)) { ok = false; break; }
            // every warp combines the cluster's partials on its own
            float pmx = -kFltMax, psum = 0.f;
            {
                float2 p[(kClMaxParts + 31) / 32];
#pragma unroll
                for (int i = 0; i < (C * kClComputeWarps + 31) / 32; ++i) {
                    const int idx = lane + i * 32;
                    p[i] = idx < C * kClComputeWarps ? ctl->part[par][idx] : make_float2(-kFltMax, 0.f);
                    pmx = fmaxf(pmx, p[i].x);
                }
                pmx = warp_max(pmx);
#pragma unroll
                for (int i = 0; i < (C * kClComputeWarps + 31) / 32; ++i)
                    psum += p[i].y * ex2((p[i].x - pmx) * kLog2e);
                psum = warp_sum(psum);
            }
            const float Mx = pmx, Ssum = psum;
            // A row whose sum of exponentials is not a positive finite number held a NaN or +inf
            // logit, or nothing but -inf: it contributes nothing (same value in every thread of the
            // cluster, since all combine the same partials in the same order).
            const bool row_finite = Ssum > 0.f && Ssum <= kFltMax && Mx <= kFltMax;
            const bool use = rec_ok && row_finite;
            RowLoss rl;
            rl.logp = 0.f; rl.loss = 0.f; rl.coef = 0.f; rl.clip = 0;
            if (use) rl = ppo_row(ctl->xy[par] - Mx, logf(Ssum), rec.old_logp, rec.adv, a.eps_low, a.eps_high, inv_denom);
            if (rank == 0 && tid == 0) {
                if (rec_ok && !row_finite) atomicOr(a.stats + 3, TPPO_DEV_NONFINITE);
                if (a.logp) a.logp[j] = rl.logp;
                if (a.token_loss) a.token_loss[j] = rl.loss;
                a.row_loss[j] = rl.loss;
                a.row_clip[j] = uint8_t(rl.clip);
            }
            if (GRAD) {
                // ---- factor * (softmax - onehot), one rounding to bf16 ---------------------------
                const float scale = use ? rl.coef * ex2((m_t - Mx) * kLog2e) / Ssum : 0.f;   // skipped row: zeros
                uint8_t* grow = nullptr;      // this CTA's slice of the gradient row (direct stores)
                if (!STAGED) {
                    if (a.mode == TPPO_DLOGITS_COMPACT) grow = dl + (j * int64_t(a.V)) * 2 + uint64_t(u0) * 16u;
                    else if (row_ok) grow = dl + (int64_t(rec.row) * a.ld) * 2 + uint64_t(u0) * 16u;
                }
                const uint64_t sc2 = ptx::pack_f32x2(scale, scale);
                if (!row_finite) {   // rare: NaN * 0 is not 0, so clear the stored exponentials
#pragma unroll
                    for (int k = 0; k < kClMaxUnits; ++k)
#pragma unroll
                        for (int q = 0; q < 4; ++q) e2[k][q] = 0ull;
                }
#pragma unroll
                for (int k = 0; k < kClMaxUnits; ++k) {
                    const uint32_t u = uint32_t(tid) + uint32_t(k) * kClComputeThreads;
                    if (u < nu) {
                        uint4 g;
                        g.x = ptx::pack_bf16x2_from_f32x2(ptx::mul_f32x2(e2[k][0], sc2));
                        g.y = ptx::pack_bf16x2_from_f32x2(ptx::mul_f32x2(e2[k][1], sc2));
                        g.z = ptx::pack_bf16x2_from_f32x2(ptx::mul_f32x2(e2[k][2], sc2));
                        g.w = ptx::pack_bf16x2_from_f32x2(ptx::mul_f32x2(e2[k][3], sc2));
                        if (STAGED) ptx::sts128(sbase + u * 16u, g);
                        else if (grow) ptx::stg128(grow + u * 16u, g);
                    }
                }
                if (y_mine) {   // the one-hot term, applied before the single rounding
                    const float g = use ? ex2((x_y - m_t) * kLog2e) * scale - rl.coef : 0.f;
                    const uint16_t gb = uint16_t(pack_bf16x2(g, 0.f) & 0xffffu);
                    if (STAGED) ptx::sts_u16(y_addr, gb);
                    else if (grow) *reinterpret_cast<uint16_t*>(grow + y_off) = gb;   // after this thread's own 16-byte store
                }
                if (STAGED) {
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->done[st]));
                }
            }
            if (++st == S) { st = 0; ph ^= 1u; }
        }
        if (!ok && (tid & 31) == 0) atomicOr(a.stats + 3, TPPO_DEV_WAIT_TIMEOUT);
    }
    // No CTA may leave while a peer can still write into its shared memory or signal its barriers.
    __syncwarp();
    ptx::cluster_sync_all();
}

// ---- host side --------------------------------------------------------------------------------
struct ClusterPlan {
    int cluster;
    uint32_t stages, stage_stride, smem_bytes;
    int max_clusters;
};

template <int C, int OUT>
static int plan_and_launch(const PolicyArgs& a, cudaStream_t s, int forced_stages, int* idle_sms) {
    const uint32_t units_total = uint32_t(a.V) >> 3;
    const uint32_t max_units = (units_total + C - 1) / C;     // largest slice, 16-byte units
    if (max_units > uint32_t(kClMaxUnits) * kClComputeThreads || max_units == 0) return TPPO_ERR_UNSUPPORTED;
    const uint32_t stride = uint32_t(align_up(size_t(max_units) * 16u, 128));
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return TPPO_ERR_CUDA;
    int max_optin = 0;
    if (cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
        return TPPO_ERR_CUDA;
    if (uint32_t(max_optin) < kClCtlBytes + stride) return TPPO_ERR_UNSUPPORTED;
    uint32_t stages = (uint32_t(max_optin) - kClCtlBytes) / stride;
    if (stages > uint32_t(kClMaxStages)) stages = kClMaxStages;
    if (forced_stages > 0 && uint32_t(forced_stages) < stages) stages = uint32_t(forced_stages);
    const uint32_t smem_bytes = kClCtlBytes + stages * stride;

    auto kern = policy_cluster_kernel<C, OUT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_bytes)) != cudaSuccess)
        return TPPO_ERR_CUDA;
    cudaLaunchConfig_t lc = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.blockDim = dim3(kClThreads, 1, 1);
    lc.dynamicSmemBytes = smem_bytes;
    lc.stream = s;
    lc.attrs = attr;
    lc.numAttrs = 1;
    lc.gridDim = dim3(C, 1, 1);
    int max_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&max_clusters, kern, &lc) != cudaSuccess || max_clusters < 1)
        return TPPO_ERR_UNSUPPORTED;
    int64_t clusters = a.n_max < 1 ? 1 : a.n_max;
    if (clusters > max_clusters) clusters = max_clusters;
    if (idle_sms) {      // SMs that host no CTA of this launch (one CTA fills an SM)
        int n_sm = 0;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n_sm = 0;
        *idle_sms = n_sm - int(clusters) * C > 0 ? n_sm - int(clusters) * C : 0;
    }
    lc.gridDim = dim3(unsigned(clusters * C), 1, 1);
    ClusterLaunch cfg{stages, stride};
    if (cudaLaunchKernelEx(&lc, kern, a, cfg) != cudaSuccess) return TPPO_ERR_CUDA;
    return TPPO_OK;
}

// variant: bits 0-3 cluster size (0 = default 4), bits 4-6 stage cap (0 = as many as fit),
// bit 7: store the gradient straight from registers instead of staging it in shared memory for
// bulk stores (measured slower: the 128-bit global stores stall the compute warps)
int launch_policy_cluster(const PolicyArgs& a, cudaStream_t s, int variant, int* idle_sms) {
    const int c = (variant & 15) ? (variant & 15) : 4;
    const int st = (variant >> 4) & 7;
    const int out = a.mode == TPPO_DLOGITS_NONE ? 0 : ((variant & 128) ? 2 : 1);
    switch (c * 4 + out) {
        case 2 * 4 + 0: return plan_and_launch<2, 0>(a, s, st, idle_sms);
        case 2 * 4 + 1: return plan_and_launch<2, 1>(a, s, st, idle_sms);
        case 2 * 4 + 2: return plan_and_launch<2, 2>(a, s, st, idle_sms);
        case 4 * 4 + 0: return plan_and_launch<4, 0>(a, s, st, idle_sms);
        case 4 * 4 + 1: return plan_and_launch<4, 1>(a, s, st, idle_sms);
        case 4 * 4 + 2: return plan_and_launch<4, 2>(a, s, st, idle_sms);
        case 8 * 4 + 0: return plan_and_launch<8, 0>(a, s, st, idle_sms);
        case 8 * 4 + 1: return plan_and_launch<8, 1>(a, s, st, idle_sms);
        case 8 * 4 + 2: return plan_and_launch<8, 2>(a, s, st, idle_sms);
        default: return TPPO_ERR_UNSUPPORTED;
    }
}

bool policy_cluster_supported(const PolicyArgs& a, int dtype) {
    if (dtype != TPPO_BF16) return false;
    if (a.V % 8 != 0 || a.ld % 8 != 0 || !aligned(a.logits, 16)) return false;
    if (a.mode != TPPO_DLOGITS_NONE && !aligned(a.dlogits, 16)) return false;
    const uint32_t max_units = ((uint32_t(a.V) >> 3) + 3) / 4;
    return max_units <= uint32_t(kClMaxUnits) * kClComputeThreads && a.V >= 4096;
}

}  // namespace tppo

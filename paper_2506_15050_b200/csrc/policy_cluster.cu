// Shared-memory-resident policy-loss kernel for bf16 logits (the throughput kernel).
//
// A thread-block cluster of C CTAs owns one selected logits row at a time; CTA c owns the c-th
// contiguous slice of the row.  Each slice is brought into shared memory once by 1-D bulk (TMA)
// copies issued by a dedicated producer warp into a ring of STAGES slice buffers, so the copies of
// the next rows are in flight while the current row is being worked on.  The 15 compute warps pull
// their 16-byte units of the slice into registers, form a thread-local maximum and the
// exponentials relative to it (one ex2 per logit, kept in registers as fp32), and reduce
// (max, sum, target logit) over the warp, the CTA and -- through distributed shared memory and a
// cluster-scope mbarrier -- the cluster.  With the row's log-sum-exp known every thread evaluates
// Eq. 1 of the paper (ratio, clip, loss term, gradient factor), rescales its stored exponentials
// into  factor * (softmax - onehot),  rounds once to bf16 and writes the result over its slice in
// shared memory; the producer warp sends it to global memory with bulk stores and reuses the
// buffer once the store has drained.  Each logit crosses the HBM interface exactly once in each
// direction.  No multicast is used: every CTA issues plain copies of its own slice.
#include "policy_common.cuh"
#include "ptx.cuh"

namespace tppo {

constexpr int kClComputeWarps = 15;
constexpr int kClComputeThreads = kClComputeWarps * 32;      // 480
constexpr int kClThreads = kClComputeThreads + 32;           // + producer warp
constexpr int kClMaxUnits = 10;                              // 16-byte units per thread per slice
constexpr int kClMaxStages = 4;
constexpr int kClMaxCluster = 8;
constexpr uint32_t kClCtlBytes = 1024;                       // control block ahead of the stages
constexpr uint32_t kClCopyChunk = 16384;                     // bytes per bulk copy instruction
constexpr uint32_t kNegInfPair = 0xff80ff80u;                // two bf16 -inf

struct ClusterCtl {
    unsigned long long full[kClMaxStages];   // slice landed in shared memory (tx-count barrier)
    unsigned long long done[kClMaxStages];   // compute warps are finished with the stage
    unsigned long long xchg[2];              // C partials arrived from the cluster
    unsigned long long wready;               // every compute warp has published its partial
    float4 part[2][kClMaxCluster];           // (max, sum, target logit, -) of each CTA
    float2 wpart[kClComputeWarps];           // (max, sum) of each warp
    float wxy;                               // target logit if it lies in this CTA's slice
    int abort;
};
static_assert(sizeof(ClusterCtl) <= kClCtlBytes, "control block too large");

struct ClusterLaunch {
    uint32_t stages;
    uint32_t stage_stride;   // bytes between stage buffers (multiple of 128)
};

template <int C, bool GRAD>
__global__ void __launch_bounds__(kClThreads, 1)
policy_cluster_kernel(const PolicyArgs a, const ClusterLaunch cfg) {
    extern __shared__ __align__(1024) uint8_t smem[];
    ClusterCtl* ctl = reinterpret_cast<ClusterCtl*>(smem);
    const uint32_t stage0 = ptx::smem_addr(smem) + kClCtlBytes;

    const uint32_t rank = ptx::cluster_ctarank();
    const int64_t cid = ptx::cluster_id_x(), ncl = ptx::num_clusters_x();
    const int64_t n = policy_n(a);
    const int64_t n_it = n > cid ? (n - cid + ncl - 1) / ncl : 0;   // rows j = cid + it * ncl
    const uint32_t S = cfg.stages;

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
        ptx::mbar_init(ptx::smem_addr(&ctl->xchg[0]), C);
        ptx::mbar_init(ptx::smem_addr(&ctl->xchg[1]), C);
        ptx::mbar_init(ptx::smem_addr(&ctl->wready), kClComputeWarps);
        ctl->abort = 0;
        ctl->wxy = 0.f;
        ptx::fence_mbar_init_cluster();
    }
    ptx::cluster_sync_all();   // barriers of every CTA are initialised before any remote arrive

    const uint8_t* logits = static_cast<const uint8_t*>(a.logits);
    uint8_t* dl = static_cast<uint8_t*>(a.dlogits);

    if (tid >= kClComputeThreads) {
        // ===================== producer warp: all bulk copies of this CTA =====================
        if (tid == kClComputeThreads) {
            int64_t issued = 0;
            auto issue_load = [&](int64_t it) {
                const uint32_t st = uint32_t(it % S);
                const int64_t j = cid + it * ncl;
                const int64_t r = a.rows ? int64_t(__ldg(a.rows + j)) : j;
                const uint32_t bar = ptx::smem_addr(&ctl->full[st]);
                if (r >= 0 && r < a.R && slice_bytes > 0) {
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
            const int64_t pro = n_it < int64_t(S) ? n_it : int64_t(S);
            for (int64_t it = 0; it < pro; ++it) issue_load(it);

            bool ok = true;
            for (int64_t it = 0; it < n_it && ok; ++it) {
                const uint32_t st = uint32_t(it % S);
                ok = ptx::mbar_wait<false>(ptx::smem_addr(&ctl->done[st]), uint32_t(it / S) & 1u);
                if (!ok) break;
                if (GRAD) {
                    const int64_t j = cid + it * ncl;
                    uint8_t* dst = nullptr;
                    if (a.mode == TPPO_DLOGITS_COMPACT) {
                        dst = dl + (j * int64_t(a.V)) * 2;
                    } else {
                        const int64_t r = a.rows ? int64_t(__ldg(a.rows + j)) : j;
                        if (r >= 0 && r < a.R) dst = dl + (r * a.ld) * 2;
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
                    if (it >= 1) {
                        ptx::bulk_wait_read<1>();             // the store of row it-1 has left smem
                        if (it - 1 + S < n_it) issue_load(it - 1 + S);
                    }
                } else {
                    if (it + S < n_it) issue_load(it + S);    // registers hold the row: reuse now
                }
            }
            if (!ok) {
                ctl->abort = 1;
                atomicOr(a.stats + 3, TPPO_DEV_WAIT_TIMEOUT);
                // let the copies that are still in flight into this CTA's shared memory land
                const int64_t first = issued > int64_t(S) ? issued - int64_t(S) : 0;
                for (int64_t it = first; it < issued; ++it)
                    ptx::mbar_wait<false>(ptx::smem_addr(&ctl->full[it % S]), uint32_t(it / S) & 1u);
            }
            ptx::bulk_wait<0>();
        }
        __syncwarp();
    } else {
        // ================================ compute warps ======================================
        const int lane = tid & 31, warp = tid >> 5;
        const float inv_denom = policy_inv_denom(a, n);
        RowMeta meta_next;
        float A_next = 0.f, old_next = 0.f;
        if (n_it > 0) {
            meta_next = policy_row_meta(a, cid);
            if (meta_next.ok) { A_next = __ldg(a.adv + meta_next.aux); old_next = __ldg(a.old_logp + meta_next.aux); }
        }
        bool ok = true;
        for (int64_t it = 0; it < n_it; ++it) {
            const uint32_t st = uint32_t(it % S);
            const int64_t j = cid + it * ncl;
            const RowMeta meta = meta_next;
            const float A = A_next, old_lp = old_next;
            if (it + 1 < n_it) {   // fetch the next row's scalars one row ahead
                meta_next = policy_row_meta(a, j + ncl);
                if (meta_next.ok) { A_next = __ldg(a.adv + meta_next.aux); old_next = __ldg(a.old_logp + meta_next.aux); }
            }
            if (!ptx::mbar_wait<false>(ptx::smem_addr(&ctl->full[st]), uint32_t(it / S) & 1u)) { ok = false; break; }

            // ---- slice -> registers ------------------------------------------------------
            const uint32_t sbase = stage0 + st * cfg.stage_stride;
            uint4 xw[kClMaxUnits];
#pragma unroll
            for (int k = 0; k < kClMaxUnits; ++k) {
                const uint32_t u = uint32_t(tid) + uint32_t(k) * kClComputeThreads;
                xw[k] = (u < nu && meta.row_ok) ? ptx::lds128(sbase + u * 16u)
                                                : make_uint4(kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair);
            }
            if (!GRAD) {   // the stage can be refilled as soon as every warp holds its units
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
            m_t = fmaxf(m_t, -1.0e30f);                 // a thread with no unit: keep finite
            // ---- exponentials relative to the thread-local max, kept in registers ---------
            const float off_t = m_t * kLog2e;
            float e[kClMaxUnits][8];
            float s_t = 0.f;
#pragma unroll
            for (int k = 0; k < kClMaxUnits; ++k) {
                const uint32_t w[4] = {xw[k].x, xw[k].y, xw[k].z, xw[k].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    e[k][2 * q] = ex2(fmaf(bf16_lo(w[q]), kLog2e, -off_t));
                    e[k][2 * q + 1] = ex2(fmaf(bf16_hi(w[q]), kLog2e, -off_t));
                    s_t += e[k][2 * q] + e[k][2 * q + 1];
                }
            }
            // ---- the target logit, if one of this thread's elements -------------------------
            const int32_t yu = (meta.y >> 3) - int32_t(u0);
            const bool y_here = meta.ok && yu >= 0 && yu < int32_t(nu);     // in this CTA's slice
            const bool y_mine = y_here && (yu % kClComputeThreads) == tid;
            const int yk = yu / kClComputeThreads, ye = meta.y & 7;
            if (y_mine) {
                uint32_t word = 0;
#pragma unroll
                for (int k = 0; k < kClMaxUnits; ++k) {
                    if (k == yk) {
                        const uint32_t w[4] = {xw[k].x, xw[k].y, xw[k].z, xw[k].w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) if (q == (ye >> 1)) word = w[q];
                    }
                }
                ctl->wxy = (ye & 1) ? bf16_hi(word) : bf16_lo(word);
            }
            // ---- warp, CTA and cluster reduction of (max, sum) ------------------------------
            const float wm = warp_max(m_t);
            const float ws = warp_sum(s_t * ex2((m_t - wm) * kLog2e));
            if (lane == 0) ctl->wpart[warp] = make_float2(wm, ws);
            __syncwarp();        // the target-logit write of any lane precedes lane 0's arrive
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->wready));
            const uint32_t par = uint32_t(it) & 1u;
            if (warp == 0) {
                if (!ptx::mbar_wait<false>(ptx::smem_addr(&ctl->wready), par)) { ok = false; break; }
                const float2 p = lane < kClComputeWarps ? ctl->wpart[lane] : make_float2(-1.0e30f, 0.f);
                const float cm = warp_max(p.x);
                const float cs = warp_sum(p.y * ex2((p.x - cm) * kLog2e));
                const float xy = y_here ? ctl->wxy : 0.f;
                __syncwarp();     // every lane has read the shared partials before any is released
                if (lane < C) {   // lane c delivers this CTA's partial to CTA c
                    const uint32_t dst = ptx::map_to_cta(ptx::smem_addr(&ctl->part[par][rank]), lane);
                    ptx::st_cluster_f32x4(dst, cm, cs, xy, 0.f);
                    ptx::mbar_arrive_remote(ptx::map_to_cta(ptx::smem_addr(&ctl->xchg[par]), lane));
                }
            }
            if (!ptx::mbar_wait<true>(ptx::smem_addr(&ctl->xchg[par]), uint32_t(it >> 1) & 1u)) { ok = false; break; }
            float Mx = -1.0e30f;
#pragma unroll
            for (int c = 0; c < C; ++c) Mx = fmaxf(Mx, ctl->part[par][c].x);
            float Ssum = 0.f, xy = 0.f;
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const float4 p = ctl->part[par][c];
                Ssum += p.y * ex2((p.x - Mx) * kLog2e);
                xy += p.z;
            }
            RowLoss rl;
            rl.logp = 0.f; rl.loss = 0.f; rl.coef = 0.f; rl.clip = 0;
            if (meta.ok) rl = ppo_row(xy, Mx + logf(Ssum), old_lp, A, a.eps_low, a.eps_high, inv_denom);
            if (rank == 0 && tid == 0) {
                if (!meta.ok) atomicOr(a.stats + 3, policy_bad_bits(meta, a));
                if (a.logp) a.logp[j] = rl.logp;
                if (a.token_loss) a.token_loss[j] = rl.loss;
                a.row_loss[j] = rl.loss;
                a.row_clip[j] = uint8_t(rl.clip);
            }
            if (GRAD) {
                // ---- factor * (softmax - onehot), one rounding to bf16, back into the slice --
                const float scale = meta.ok ? rl.coef * ex2((m_t - Mx) * kLog2e) / Ssum : 0.f;
#pragma unroll
                for (int k = 0; k < kClMaxUnits; ++k) {
                    const uint32_t u = uint32_t(tid) + uint32_t(k) * kClComputeThreads;
                    float g[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) g[q] = meta.ok ? e[k][q] * scale : 0.f;
                    if (y_mine && k == yk) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) if (q == ye) g[q] -= rl.coef;
                    }
                    if (u < nu) {
                        ptx::sts128(sbase + u * 16u,
                                    make_uint4(pack_bf16x2(g[0], g[1]), pack_bf16x2(g[2], g[3]),
                                               pack_bf16x2(g[4], g[5]), pack_bf16x2(g[6], g[7])));
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->done[st]));
            }
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

template <int C, bool GRAD>
static int plan_and_launch(const PolicyArgs& a, cudaStream_t s, int forced_stages) {
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

    auto kern = policy_cluster_kernel<C, GRAD>;
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
    lc.gridDim = dim3(unsigned(clusters * C), 1, 1);
    ClusterLaunch cfg{stages, stride};
    if (cudaLaunchKernelEx(&lc, kern, a, cfg) != cudaSuccess) return TPPO_ERR_CUDA;
    return TPPO_OK;
}

// variant: bits 0-3 cluster size (0 = default 4), bits 4-7 stage cap (0 = as many as fit)
int launch_policy_cluster(const PolicyArgs& a, cudaStream_t s, int variant) {
    const int c = (variant & 15) ? (variant & 15) : 4;
    const int st = (variant >> 4) & 15;
    const bool grad = a.mode != TPPO_DLOGITS_NONE;
    switch (c) {
        case 2: return grad ? plan_and_launch<2, true>(a, s, st) : plan_and_launch<2, false>(a, s, st);
        case 4: return grad ? plan_and_launch<4, true>(a, s, st) : plan_and_launch<4, false>(a, s, st);
        case 8: return grad ? plan_and_launch<8, true>(a, s, st) : plan_and_launch<8, false>(a, s, st);
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

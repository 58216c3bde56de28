// CTA-pair version of the persistent bf16 GEMM skeleton (see umma_gemm.cuh): two CTAs of a cluster
// own one 256 x 256 accumulator tile, 128 rows each.  Every CTA stages its own 128 rows of A and
// its own 128 of the 256 N rows of B (32 KB per stage instead of 48, six stages instead of four),
// the leader CTA issues tcgen05.mma.cta_group::2, and both CTAs run the caller's epilogue on the
// accumulator rows in their own tensor memory.  Per 64-deep step a CTA pulls 256 operand rows from
// L2 for 256 x 256 outputs instead of 384 for 128 x 256: a third less shared-memory fill and L2
// traffic per FLOP.  No TMA multicast: each CTA loads what it stages.
//
// Barriers (all waits bounded, see umma_gemm.cuh):
//   full[s]      in the leader; both producers announce their 32 KB on it, both CTAs' TMA loads
//                count their bytes on it
//   empty[s]     in each CTA; the leader's MMA thread commits onto both when a stage is consumed
//   acc_full[a]  in each CTA; committed by the leader when a tile's last MMA is issued
//   acc_empty[a] in the leader; the eight epilogue warps of the pair arrive on it
#pragma once

#include "umma_gemm.cuh"

namespace tppo {

constexpr int kPairStages = 6;
constexpr uint32_t kPairBBytes = (kTileN / 2) * kTileK * 2;          // 16 KB: half of B's N rows
constexpr uint32_t kPairStageBytes = kABytes + kPairBBytes;          // 32 KB per CTA and stage
constexpr size_t kPairSmemBytes = size_t(kPairStages) * kPairStageBytes + 1024 + 256;

// Tile coordinates in units of CTA pairs: g.m_tiles counts 128-row tiles; a pair covers two.
__device__ __forceinline__ void pair_tile_coords(const GemmShape& g, int m_pairs, int t, int& mp,
                                                 int& nt) {
    const int gm_max = max(g.group_m / 2, 1);
    const int per_group = gm_max * g.n_tiles;
    const int gi = t / per_group;
    const int first = gi * gm_max;
    const int gm = min(gm_max, m_pairs - first);
    const int in = t - gi * per_group;
    mp = first + in % gm;
    nt = in / gm;
}

template <int AMAJ, int BMAJ, class Epi>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
umma_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a,
                      const __grid_constant__ CUtensorMap map_b, const GemmShape g, const Epi epi,
                      int32_t* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t bars = base + kPairStages * kPairStageBytes;
    const uint32_t full_bar = bars;                               // [kPairStages]
    const uint32_t empty_bar = bars + 8 * kPairStages;            // [kPairStages]
    const uint32_t acc_full_bar = bars + 16 * kPairStages;        // [2]
    const uint32_t acc_empty_bar = acc_full_bar + 16;             // [2]
    const uint32_t tmem_slot = acc_empty_bar + 16;
    uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();                 // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int n_pairs = gridDim.x >> 1;
    const int m_pairs = (g.m_tiles + 1) / 2;
    const int total = m_pairs * g.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            ptx::mbar_init(full_bar + 8 * s, 2);                  // one announcement per CTA
            ptx::mbar_init(empty_bar + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full_bar + 8 * a, 1);
            ptx::mbar_init(acc_empty_bar + 8 * a, 8);             // four epilogue warps per CTA
        }
        ptx::fence_mbar_init_cluster();
        umma::prefetch_tensormap(&map_a);
        umma::prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        umma::tmem_alloc_pair(tmem_slot, 512);
        umma::tmem_relinquish_pair();
    }
    umma::fence_before_thread_sync();
    ptx::cluster_sync_all();        // both CTAs' barriers exist before anyone arrives on them
    umma::fence_after_thread_sync();
    const uint32_t tmem_base = *tmem_slot_ptr;

    bool timed_out = false;
    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            for (int t = pair; t < total && !timed_out; t += n_pairs) {
                int mp, nt;
                pair_tile_coords(g, m_pairs, t, mp, nt);
                const int am = g.a_mn_off + (2 * mp + int(rank)) * kTileM;
                const int bn = g.b_mn_off + nt * kTileN + int(rank) * (kTileN / 2);
                for (int ks = 0; ks < g.k_steps; ++ks) {
                    if (!ptx::mbar_wait<false>(empty_bar + 8 * stage, phase ^ 1u)) {
                        timed_out = true;
                        break;
                    }
                    const uint32_t fb = ptx::map_to_cta(full_bar + 8 * stage, 0);   // leader's
                    const uint32_t sa = base + stage * kPairStageBytes;
                    const uint32_t sb = sa + kABytes;
                    ptx::mbar_arrive_expect_tx_cluster(fb, kPairStageBytes);
                    const int ak = g.a_k_off + ks * kTileK;
                    const int bk = g.b_k_off + ks * kTileK;
                    if (AMAJ == 0) {
                        umma::tma_load_2d_pair(sa, &map_a, fb, ak, am);
                    } else {
#pragma unroll
                        for (int q = 0; q < kTileM / 64; ++q)
                            umma::tma_load_2d_pair(sa + q * kBoxBytes64, &map_a, fb, am + 64 * q, ak);
                    }
                    if (BMAJ == 0) {
                        umma::tma_load_2d_pair(sb, &map_b, fb, bk, bn);
                    } else {
#pragma unroll
                        for (int q = 0; q < kTileN / 128; ++q)
                            umma::tma_load_2d_pair(sb + q * kBoxBytes64, &map_b, fb, bn + 64 * q, bk);
                    }
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = umma::instr_desc_bf16(2 * kTileM, kTileN, AMAJ, BMAJ);
            constexpr uint32_t a_kstep = AMAJ ? 16 * 128 : 32;
            constexpr uint32_t b_kstep = BMAJ ? 16 * 128 : 32;
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            for (int t = pair; t < total && !timed_out; t += n_pairs, ++local) {
                const int acc = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!ptx::mbar_wait<true>(acc_empty_bar + 8 * acc, acc_phase ^ 1u)) {
                    timed_out = true;
                    break;
                }
                umma::fence_after_thread_sync();
                const uint32_t d = tmem_base + acc * kTileN;
                for (int ks = 0; ks < g.k_steps; ++ks) {
                    if (!ptx::mbar_wait<true>(full_bar + 8 * stage, phase)) {
                        timed_out = true;
                        break;
                    }
                    umma::fence_after_thread_sync();
                    const uint32_t sa = base + stage * kPairStageBytes;
                    const uint32_t sb = sa + kABytes;
                    const uint64_t ad = AMAJ ? umma::smem_desc(sa, kBoxBytes64, 1024)
                                             : umma::smem_desc(sa, 16, 1024);
                    const uint64_t bd = BMAJ ? umma::smem_desc(sb, kBoxBytes64, 1024)
                                             : umma::smem_desc(sb, 16, 1024);
#pragma unroll
                    for (int j = 0; j < kTileK / 16; ++j)
                        umma::mma_bf16_pair(d, umma::smem_desc_advance(ad, j * a_kstep),
                                            umma::smem_desc_advance(bd, j * b_kstep), idesc,
                                            (ks | j) != 0 ? 1u : 0u);
                    // the stage is reusable in both CTAs once these MMAs have read it
                    umma::mma_commit_pair(ptx::map_to_cta(empty_bar + 8 * stage, 0));
                    umma::mma_commit_pair(ptx::map_to_cta(empty_bar + 8 * stage, 1));
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                }
                if (timed_out) break;
                umma::mma_commit_pair(ptx::map_to_cta(acc_full_bar + 8 * acc, 0));
                umma::mma_commit_pair(ptx::map_to_cta(acc_full_bar + 8 * acc, 1));
            }
        }
    } else {
        // ---------------- epilogue (both CTAs, own accumulator rows) ----------------
        const int q = warp & 3;
        const int row = q * 32 + lane;
        int local = 0;
        for (int t = pair; t < total; t += n_pairs, ++local) {
            int mp, nt;
            pair_tile_coords(g, m_pairs, t, mp, nt);
            const int acc = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1;
            if (!ptx::mbar_wait<true>(acc_full_bar + 8 * acc, acc_phase)) {
                timed_out = true;
                break;
            }
            umma::fence_after_thread_sync();
            epi(2 * mp + int(rank), nt, row, tmem_base + acc * kTileN + (uint32_t(q * 32) << 16));
            umma::fence_before_thread_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(acc_empty_bar + 8 * acc, 0));
        }
    }
    if (timed_out) atomicOr(status, TPPO_DEV_WAIT_TIMEOUT);
    umma::fence_before_thread_sync();
    ptx::cluster_sync_all();        // nobody leaves while the peer may still arrive on its barriers
    if (warp == 1) {
        __syncwarp();
        umma::tmem_dealloc_pair(tmem_base, 512);
    }
}

template <int AMAJ, int BMAJ, class Epi>
int launch_umma_gemm_pair(const CUtensorMap& a, const CUtensorMap& b, const GemmShape& g,
                          const Epi& epi, int32_t* status, cudaStream_t s) {
    auto kernel = umma_gemm_pair_kernel<AMAJ, BMAJ, Epi>;
    TPPO_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         int(kPairSmemBytes)));
    const int total = ((g.m_tiles + 1) / 2) * g.n_tiles;
    if (total <= 0) return TPPO_OK;
    // Tiles are dealt out statically, so every pair of the grid has to be resident at once: ask how
    // many 2-CTA clusters of this kernel the device holds (not every SM can be paired) and cache
    // the answer per device.
    static int resident[64] = {};
    int dev = 0;
    TPPO_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return TPPO_ERR_CUDA;
    int max_pairs = __atomic_load_n(&resident[dev], __ATOMIC_ACQUIRE);
    if (max_pairs == 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kNumSms, 1, 1);
        cfg.blockDim = dim3(kGemmThreads, 1, 1);
        cfg.dynamicSmemBytes = kPairSmemBytes;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        TPPO_CUDA_CHECK(cudaOccupancyMaxActiveClusters(&max_pairs, kernel, &cfg));
        if (max_pairs < 1) return TPPO_ERR_CUDA;
        if (max_pairs > kNumSms / 2) max_pairs = kNumSms / 2;
        __atomic_store_n(&resident[dev], max_pairs, __ATOMIC_RELEASE);
    }
    const int pairs = total < max_pairs ? total : max_pairs;
    kernel<<<2 * pairs, kGemmThreads, kPairSmemBytes, s>>>(a, b, g, epi, status);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

}  // namespace tppo

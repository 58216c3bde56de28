// Persistent bf16 tensor-core GEMM skeleton for sm_100a: D[128 x 256 tile] = A * B with fp32
// accumulation in tensor memory, operands staged by tiled TMA loads through a shared-memory ring,
// and a caller-supplied epilogue that reads the accumulator straight from tensor memory.
//
// One CTA per SM, 192 threads:
//   warp 0     one lane issues the TMA loads of both operands, stage by stage
//   warp 1     owns the tensor-memory allocation; one lane issues tcgen05.mma and the commits that
//              free a stage (operands consumed) or publish an accumulator (tile finished)
//   warps 2-5  epilogue: each warp reads its 32 accumulator rows (TMEM lanes) 32 columns at a time
// Two 256-column accumulators alternate, so the epilogue of tile i overlaps the main loop of tile
// i+1.  Every wait is bounded; a wait that runs out raises TPPO_DEV_WAIT_TIMEOUT in *status, the CTA
// stops taking tiles, and tensor memory is still released before exit.
#pragma once

#include "common.cuh"
#include "ptx.cuh"
#include "umma.cuh"

namespace tppo {

constexpr int kTileM = 128;
constexpr int kTileN = 256;
constexpr int kTileK = 64;           // one 128-byte swizzled row of bf16
constexpr int kStages = 4;
constexpr int kGemmThreads = 192;
constexpr uint32_t kABytes = kTileM * kTileK * 2;     // 16 KB
constexpr uint32_t kBBytes = kTileN * kTileK * 2;     // 32 KB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kBoxBytes64 = 64 * kTileK * 2;     // a 64 x 64 box of an MN-major operand
constexpr size_t kGemmSmemBytes = size_t(kStages) * kStageBytes + 1024 /*alignment slack*/ + 256;

// Problem geometry in tiles plus the element offsets added to every TMA coordinate (so that one
// tensor map over a whole matrix can serve a window of it).
struct GemmShape {
    int32_t m_tiles, n_tiles, k_steps;
    int32_t a_mn_off, a_k_off, b_mn_off, b_k_off;
    int32_t group_m;     // m-tiles per raster group: tiles of a group run next to each other in time
};

__device__ __forceinline__ void gemm_tile_coords(const GemmShape& g, int t, int& mt, int& nt) {
    const int per_group = g.group_m * g.n_tiles;
    const int gi = t / per_group;
    const int first = gi * g.group_m;
    const int gm = min(g.group_m, g.m_tiles - first);
    const int in = t - gi * per_group;
    mt = first + in % gm;
    nt = in / gm;
}

// AMAJ / BMAJ: 0 = the contraction index is contiguous in global memory (tensor map: inner
// dimension k, box 64 x 128 for A and 64 x 256 for B), 1 = the M / N index is contiguous (tensor
// map: inner dimension M or N, box 64 x 64; two boxes per stage for A, four for B).
//
// Epi must provide
//   __device__ void operator()(int mt, int nt, int row, uint32_t taddr) const
// called by all 32 lanes of an epilogue warp with row = this thread's row inside the tile and
// taddr = TMEM address of column 0 of that row (lane offset included).
template <int AMAJ, int BMAJ, class Epi>
__global__ void __launch_bounds__(kGemmThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const GemmShape g, const Epi epi, int32_t* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                 // operand tiles: 1024-byte aligned
    const uint32_t bars = base + kStages * kStageBytes;           // barriers behind the ring
    const uint32_t full_bar = bars;                               // [kStages]
    const uint32_t empty_bar = bars + 8 * kStages;                // [kStages]
    const uint32_t acc_full_bar = bars + 16 * kStages;            // [2]
    const uint32_t acc_empty_bar = acc_full_bar + 16;             // [2]
    const uint32_t tmem_slot = acc_empty_bar + 16;                // u32: TMEM base address
    uint32_t* tmem_slot_ptr =
        reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total = g.m_tiles * g.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full_bar + 8 * s, 1);
            ptx::mbar_init(empty_bar + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full_bar + 8 * a, 1);
            ptx::mbar_init(acc_empty_bar + 8 * a, 4);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        umma::prefetch_tensormap(&map_a);
        umma::prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        umma::tmem_alloc(tmem_slot, 512);
        umma::tmem_relinquish();
    }
    umma::fence_before_thread_sync();
    __syncthreads();
    umma::fence_after_thread_sync();
    const uint32_t tmem_base = *tmem_slot_ptr;

    bool timed_out = false;
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            for (int t = blockIdx.x; t < total && !timed_out; t += gridDim.x) {
                int mt, nt;
                gemm_tile_coords(g, t, mt, nt);
                const int am = g.a_mn_off + mt * kTileM;
                const int bn = g.b_mn_off + nt * kTileN;
                for (int ks = 0; ks < g.k_steps; ++ks) {
                    if (!ptx::mbar_wait<false>(empty_bar + 8 * stage, phase ^ 1u)) {
                        timed_out = true;
                        break;
                    }
                    const uint32_t fb = full_bar + 8 * stage;
                    const uint32_t sa = base + stage * kStageBytes;
                    const uint32_t sb = sa + kABytes;
                    ptx::mbar_arrive_expect_tx(fb, kStageBytes);
                    const int ak = g.a_k_off + ks * kTileK;
                    const int bk = g.b_k_off + ks * kTileK;
                    if (AMAJ == 0) {
                        umma::tma_load_2d(sa, &map_a, fb, ak, am);
                    } else {
#pragma unroll
                        for (int q = 0; q < kTileM / 64; ++q)
                            umma::tma_load_2d(sa + q * kBoxBytes64, &map_a, fb, am + 64 * q, ak);
                    }
                    if (BMAJ == 0) {
                        umma::tma_load_2d(sb, &map_b, fb, bk, bn);
                    } else {
#pragma unroll
                        for (int q = 0; q < kTileN / 64; ++q)
                            umma::tma_load_2d(sb + q * kBoxBytes64, &map_b, fb, bn + 64 * q, bk);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = umma::instr_desc_bf16(kTileM, kTileN, AMAJ, BMAJ);
            // byte step between the four 16-wide k slices of a stage
            constexpr uint32_t a_kstep = AMAJ ? 16 * 128 : 32;
            constexpr uint32_t b_kstep = BMAJ ? 16 * 128 : 32;
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            for (int t = blockIdx.x; t < total && !timed_out; t += gridDim.x, ++local) {
                const int acc = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!ptx::mbar_wait<false>(acc_empty_bar + 8 * acc, acc_phase ^ 1u)) {
                    timed_out = true;
                    break;
                }
                umma::fence_after_thread_sync();
                const uint32_t d = tmem_base + acc * kTileN;
                for (int ks = 0; ks < g.k_steps; ++ks) {
                    if (!ptx::mbar_wait<false>(full_bar + 8 * stage, phase)) {
                        timed_out = true;
                        break;
                    }
                    umma::fence_after_thread_sync();
                    const uint32_t sa = base + stage * kStageBytes;
                    const uint32_t sb = sa + kABytes;
                    const uint64_t ad = AMAJ ? umma::smem_desc(sa, kBoxBytes64, 1024)
                                             : umma::smem_desc(sa, 16, 1024);
                    const uint64_t bd = BMAJ ? umma::smem_desc(sb, kBoxBytes64, 1024)
                                             : umma::smem_desc(sb, 16, 1024);
#pragma unroll
                    for (int j = 0; j < kTileK / 16; ++j)
                        umma::mma_bf16(d, umma::smem_desc_advance(ad, j * a_kstep),
                                       umma::smem_desc_advance(bd, j * b_kstep), idesc,
                                       (ks | j) != 0 ? 1u : 0u);
                    umma::mma_commit(empty_bar + 8 * stage);       // stage reusable once consumed
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (timed_out) break;
                umma::mma_commit(acc_full_bar + 8 * acc);          // accumulator complete
            }
        }
    } else {
        // ---------------- epilogue ----------------
        const int q = warp & 3;                                    // TMEM lane quarter of this warp
        const int row = q * 32 + lane;
        int local = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++local) {
            int mt, nt;
            gemm_tile_coords(g, t, mt, nt);
            const int acc = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1;
            if (!ptx::mbar_wait<false>(acc_full_bar + 8 * acc, acc_phase)) {
                timed_out = true;
                break;
            }
            umma::fence_after_thread_sync();
            epi(mt, nt, row, tmem_base + acc * kTileN + (uint32_t(q * 32) << 16));
            umma::fence_before_thread_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty_bar + 8 * acc);
        }
    }
    if (timed_out) atomicOr(status, TPPO_DEV_WAIT_TIMEOUT);
    umma::fence_before_thread_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        umma::tmem_dealloc(tmem_base, 512);
    }
}

// ---- host side ----------------------------------------------------------------------------------
// Tensor map over a row-major bf16 matrix [rows, cols] (cols contiguous, row stride ld elements),
// 128-byte swizzle, boxes of 64 columns by box_rows rows.  Returns false when the driver's encoder
// is unavailable or rejects the arguments (base 16-byte aligned, ld*2 a multiple of 16).
bool make_bf16_tensor_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols,
                          uint64_t ld, uint32_t box_rows);

template <int AMAJ, int BMAJ, class Epi>
int launch_umma_gemm(const CUtensorMap& a, const CUtensorMap& b, const GemmShape& g, const Epi& epi,
                     int32_t* status, cudaStream_t s) {
    auto kernel = umma_gemm_kernel<AMAJ, BMAJ, Epi>;
    // per device and cheap, so it is simply set on every launch
    TPPO_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         int(kGemmSmemBytes)));
    const int total = g.m_tiles * g.n_tiles;
    if (total <= 0) return TPPO_OK;
    const int grid = total < kNumSms ? total : kNumSms;
    kernel<<<grid, kGemmThreads, kGemmSmemBytes, s>>>(a, b, g, epi, status);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}

}  // namespace tppo

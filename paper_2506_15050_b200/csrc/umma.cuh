// Inline-PTX wrappers for the sm_100a tensor-core path: tensor memory (TMEM) allocation,
// tcgen05.mma issue / commit / load, shared-memory matrix descriptors, the instruction descriptor
// and tiled TMA loads, in single-CTA (cta_group::1) and CTA-pair (cta_group::2) forms; no multicast
// anywhere.
#pragma once

#include <cuda.h>          // CUtensorMap (type only; the encoder is looked up at run time)
#include <cuda_runtime.h>
#include <stdint.h>

namespace tppo {
namespace umma {

// One lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// ---- tensor memory --------------------------------------------------------------------------
// Whole-warp calls.  `ncols` is a power of two in [32, 512]; the base address (lane 0, first
// column) is written to the shared-memory word at `smem_dst`.
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void fence_before_thread_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void fence_after_thread_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// ---- descriptors ------------------------------------------------------------------------------
// Operand tiles sit in shared memory as rows of 128 bytes (64 bf16) with the 128-byte swizzle, the
// layout a tiled TMA load with CU_TENSOR_MAP_SWIZZLE_128B produces; tile bases are 1024-byte
// aligned.
//   K-major operand (contraction index contiguous in memory): row = one M/N index, 64 k values.
//     Eight-row groups are 1024 bytes apart (stride offset); the leading offset is not used.
//   MN-major operand (M/N index contiguous in memory): row = one k index, 64 M/N values.  A block
//     of 64 M/N values by `k_rows` k values is contiguous; eight-k groups are 1024 bytes apart
//     (stride offset) and the next block of 64 M/N values starts k_rows*128 bytes later (leading
//     offset).
// Field positions: start address >> 4 in bits [0,14), leading offset >> 4 in [16,30), stride offset
// >> 4 in [32,46), descriptor version 1 in [46,48), swizzle mode in [61,64) (2 = 128-byte).
__device__ __forceinline__ uint64_t smem_desc(uint32_t smem_addr, uint32_t leading_bytes,
                                              uint32_t stride_bytes) {
    uint64_t d = 0;
    d |= uint64_t((smem_addr & 0x3ffffu) >> 4);
    d |= uint64_t((leading_bytes >> 4) & 0x3fffu) << 16;
    d |= uint64_t((stride_bytes >> 4) & 0x3fffu) << 32;
    d |= uint64_t(1) << 46;
    d |= uint64_t(2) << 61;
    return d;
}
// The same descriptor moved by `bytes` inside its tile.
__device__ __forceinline__ uint64_t smem_desc_advance(uint64_t d, uint32_t bytes) {
    return d + uint64_t(bytes >> 4);
}

// Instruction descriptor of a dense bf16 x bf16 -> fp32 MMA (kind::f16): accumulator format fp32 in
// bits [4,6), A and B formats (1 = bf16) in [7,10) and [10,13), operand majors (1 = M/N index
// contiguous) in bits 15 and 16, N >> 3 in [17,23), M >> 4 in [24,29).
__host__ __device__ constexpr uint32_t instr_desc_bf16(int m, int n, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(a_mn_major) << 15) |
           (uint32_t(b_mn_major) << 16) | (uint32_t(n >> 3) << 17) | (uint32_t(m >> 4) << 24);
}

// D[tmem] = A*B (accumulate == 0) or D += A*B, one 128 x N x 16 bf16 step, issued by one thread.
__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc,
                                         uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives once on the mbarrier when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane (warp w reads lanes 32*(w%4)..+31; the
// lane offset is part of `taddr`).  Whole-warp call; follow with tmem_ld_wait before using v.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]),
          "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]),
          "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---- tiled TMA load (no multicast) ------------------------------------------------------------
// Copies the box of the tensor map that starts at element (x, y) -- x along the contiguous
// dimension, x * element size a multiple of 16 bytes -- into shared memory and counts its bytes on
// the mbarrier.  Out-of-range parts of the box are filled with zeros and still counted.
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar,
                                            int32_t x, int32_t y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
// Tiled store of a box from shared memory (the caller commits and waits on the bulk group).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src_smem, int32_t x,
                                             int32_t y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src_smem), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// ---- CTA-pair forms (cta_group::2) ----------------------------------------------------------
// Two CTAs of a cluster (ranks 0 and 1) share one MMA of 256 rows: each stages its own 128 rows of
// A and its own half of B's N rows, the leader (rank 0) issues the instruction, and each CTA's
// tensor memory receives its 128 rows of the accumulator.  Allocation and release are done by the
// same warp of both CTAs.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}
// One 256 x N x 16 bf16 step over the CTA pair, issued by one thread of the leader CTA.  The
// descriptors name the leader's shared memory; the peer's operands sit at the same offsets.
__device__ __forceinline__ void mma_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc,
                                              uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives once on the mbarrier at shared::cluster address `bar` (this CTA's or the peer's) when
// every pair MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit_pair(uint32_t cluster_bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(cluster_bar) : "memory");
}
// Tiled TMA load into this CTA's shared memory whose bytes are counted on an mbarrier that may
// live in the peer CTA (shared::cluster address).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const CUtensorMap* map,
                                                 uint32_t cluster_bar, int32_t x, int32_t y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(cluster_bar), "r"(x), "r"(y)
        : "memory");
}

}  // namespace umma
}  // namespace tppo

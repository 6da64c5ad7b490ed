// Blackwell tensor-core plumbing used by the scoring kernels: TMA tensor maps (host side),
// tiled TMA loads, tensor-memory allocation, tcgen05.mma descriptors/issue/commit and
// tensor-memory loads (device side).
//
// Operand tiles are 128 rows x 128 bf16, stored in shared memory as two halves of
// 128 rows x 64 elements (128 bytes per row) with the 128-byte swizzle: exactly what a TMA
// load with box {64, 128} and SWIZZLE_128B writes, and what a K-major tcgen05 shared-memory
// descriptor with SWIZZLE_128B reads.  Tiles must start on a 1024-byte boundary.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace skipkv {

constexpr int kOpRows = 128;                       // rows of an operand tile
constexpr int kOpHalfBytes = kOpRows * 128;        // one 64-element half: 16 KB
constexpr int kOpBytes = 2 * kOpHalfBytes;         // 32 KB

// ---- host: tensor maps ------------------------------------------------------------------
// 2-D view [rows][128] bf16 of a row-major buffer, box = 64 elements x box_rows rows, 128-byte swizzle.
int tmap_rows(CUtensorMap* out, const void* base, uint64_t rows, uint32_t box_rows);
// 3-D view of the window queries [heads][window][128] bf16 (dims fastest first: channel, window
// position, head), box = 64 channels x box_w window positions x box_heads heads.
int tmap_qwin(CUtensorMap* out, const void* base, uint64_t heads, uint32_t window, uint32_t box_w, uint32_t box_heads);

#ifdef __CUDACC__
// ---- device -------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(smem_dst)),
        "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
            smem_u32(smem_dst)),
        "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tmap_prefetch(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Tensor memory: allocation is a warp-wide operation; the base address lands in shared memory.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand half-tile with the 128-byte swizzle:
// rows 128 bytes apart inside a group of 8, groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
    return uint64_t((smem_addr >> 4) & 0x3fffu) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) |
           (uint64_t(1) << 46) | (uint64_t(2) << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = N = 128.
constexpr uint32_t kIdescBf16M128N128 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// D[128 x 128] (+)= A[128 x 16] * B[128 x 16]^T, issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The full K = 128 contraction of two operand tiles (8 steps of 16): 4 per 64-element half.
__device__ __forceinline__ void umma_tile_128x128x128(uint32_t tmem_d, uint32_t a_smem, uint32_t b_smem, bool accumulate_first) {
    const uint64_t da = umma_desc_sw128(a_smem), db = umma_desc_sw128(b_smem);
#pragma unroll
    for (int half = 0; half < 2; ++half)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            const uint64_t off = uint64_t(half * (kOpHalfBytes >> 4) + ks * 2);      // in 16-byte units
            umma_bf16(tmem_d, da + off, db + off, kIdescBf16M128N128, (accumulate_first || half || ks) ? 1u : 0u);
        }
}
// Arrive on an mbarrier when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 consecutive fp32 columns of this thread's tensor-memory lane (lane = 32*(warp%4) + laneid).
// The wait is part of the same statement so the registers are defined when it returns.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
#endif  // __CUDACC__

}  // namespace skipkv

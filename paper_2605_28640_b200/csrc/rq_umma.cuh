// Fifth-generation tensor-core plumbing (tcgen05): operand descriptors for tiles in shared memory,
// tensor-memory allocation, issue and completion of a matrix product, and reading the
// accumulator back into registers.  One CTA per product (cta_group::1), bf16 operands, fp32
// accumulator.
//
// Operand tiles are K-major (a row's K elements are consecutive in the source) and stored without
// swizzle as 8-row x 16-byte core matrices: element (row r, 16-byte piece c of the row's K extent)
// lives at  (r / 8) * SBO + c * LBO + (r % 8) * 16  with LBO = 128 (the pieces of one 8-row group
// follow each other) and SBO = pieces * 128 (then the next 8 rows).  One instruction consumes
// K = 16 elements = two pieces; the descriptor of the k-th step starts 256 bytes further on.
#pragma once
#include <stdint.h>

#include "rq_async.cuh"

namespace rq {

constexpr uint32_t kUmmaLbo = 128;             // bytes between the two 16-byte pieces of one K step

// byte offset of piece (row, piece) in a tile whose rows hold `pieces` 16-byte pieces
__device__ __forceinline__ uint32_t umma_tile_offset(int row, int piece, int pieces)
{
    return (uint32_t)(row >> 3) * (uint32_t)(pieces * 128) + (uint32_t)piece * kUmmaLbo + (uint32_t)(row & 7) * 16u;
}

// shared-memory matrix descriptor: start address, leading and stride byte offsets (all without
// their 4 low bits), descriptor version 1, no swizzle
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t sbo_bytes)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(kUmmaLbo >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46);
}

// The same tiles with the 128-byte swizzle, which is what a tiled bulk-tensor copy (TMA) with
// CU_TENSOR_MAP_SWIZZLE_128B writes: the K extent is cut into halves of 64 elements (128 bytes); a half
// holds its rows 128 bytes apart, groups of 8 rows 1024 bytes apart, and inside a row the 16-byte piece p
// sits at ((p ^ (row % 8)) * 16).  Tile bases are 1024-byte aligned.  A K step of 16 elements is 32 bytes
// further on inside the half.
__device__ __forceinline__ uint32_t umma_sw128_offset(int row, int piece)   // piece: 0..7 inside the half
{
    return (uint32_t)(row >> 3) * 1024u + (uint32_t)(row & 7) * 128u + (uint32_t)((piece ^ (row & 7)) * 16);
}
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Tiled bulk-tensor copy of one box of a rank-4 tensor map into shared memory; completion (the box's
// bytes) is counted on the barrier.  One thread.
__device__ __forceinline__ void tma_load_4d(void *dst_smem, const void *tmap, int c0, int c1, int c2, int c3, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(
            smem_addr(dst_smem)),
        "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_addr(bar))
        : "memory");
}

// The same box brought into L2 only (no shared memory, no barrier): a hint issued a few tiles ahead of the copy
// itself, so that the copy finds its bytes in L2.  One thread.
__device__ __forceinline__ void tma_prefetch_4d(const void *tmap, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(tmap), "r"(c0), "r"(c1), "r"(c2),
                 "r"(c3)
                 : "memory");
}

// instruction descriptor of D[M x N] (fp32) = A[M x 16] (bf16, K-major) * B[N x 16]^T (bf16, K-major)
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Tensor memory: `cols` columns (a power of two, at least 32) of all 128 lanes.  Executed by one
// whole warp; the base address arrives in *dst (shared memory).
__device__ __forceinline__ void tmem_alloc(uint32_t *dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(dst)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// one product step, issued by ONE thread; accumulate = 0 overwrites D
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the same with the A operand in tensor memory: lane = row, a 32-bit column holds two consecutive bf16 of the
// row's K extent (the lower index in the low half), so a K step of 16 elements is 8 columns
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the barrier gets one arrival when every product issued by this thread so far has completed
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ void tcgen05_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's lane (lane = 32 * (warp % 4) + lane id; the lane
// field of taddr must be the warp's own 32 * (warp % 4)).  Whole warp.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
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

// 16 consecutive 32-bit columns of this thread's lane written from registers.  Whole warp; follow the last
// store of a batch with tmem_st_wait() before the data is handed on.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

}  // namespace rq

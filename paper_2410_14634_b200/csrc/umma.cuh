// Fifth-generation tensor-core (tcgen05) primitives for sm_100a, as inline PTX:
// tensor-memory allocation, matrix descriptors for shared-memory operands,
// the MMA issue, its completion signal on an mbarrier, and the load that brings
// accumulators from tensor memory back to registers.
//
// Operand layout used throughout (the "no swizzle, K-major" canonical form):
// an operand of R rows and 8 (tf32) or 16 (bf16) contraction elements per MMA is
// held as two planes of R 16-byte rows; row r of plane p sits at
//   base + p * plane_bytes + r * 16.
// With 128 bytes between 8-row groups the rows of a plane are one linear array,
// so an operand may START AT ANY ROW: moving the start address by s * 16 bytes
// shifts the whole operand by s rows.  The kernels use this to apply a spatial
// tap as a row offset instead of re-packing the pixels.
#pragma once

#include <stdint.h>

#include "tma.cuh"

namespace invconv {
namespace umma {

// 64-bit shared-memory matrix descriptor: start address, byte offset between the two K planes of one MMA
// ("leading" offset), byte offset between 8-row groups ("stride" offset, 128 = linear rows), no swizzle.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t plane_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((plane_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(128u >> 4) << 32;
    d |= (uint64_t)1 << 46;                      // descriptor version of this architecture
    return d;
}

// Moves a descriptor's start address by `bytes` (a multiple of 16; may be negative).
__device__ __forceinline__ uint64_t advance_desc(uint64_t d, int bytes) { return d + (uint64_t)(int64_t)(bytes >> 4); }

// 32-bit instruction descriptor: fp32 accumulate, both operands K-major, M = 128, N given.
constexpr uint32_t kFmtBF16 = 1, kFmtTF32 = 2;
__host__ __device__ constexpr uint32_t make_idesc(uint32_t fmt, uint32_t n)
{
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// Allocate / free `cols` (a power of two >= 32) columns of tensor memory; executed by one whole warp.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t tmem_addr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_addr), "r"(cols) : "memory");
}

__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[128 x N] (+)= A[128 x K] * B[N x K]^T, issued by one thread.  accumulate == 0 overwrites D.
__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}

// The mbarrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void commit(unsigned long long* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 16 consecutive accumulator columns of the calling thread's lane (warp w of a warpgroup reads lanes
// 32w..32w+31).  The load is asynchronous: the registers hold the values only after tmem_ld_fence, which
// names them as in/out operands so that the compiler keeps every use behind it.
__device__ __forceinline__ void tmem_ld16(uint32_t tmem_addr, uint32_t (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(tmem_addr));
}
__device__ __forceinline__ void tmem_ld_fence(uint32_t (&r)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :: "memory");
}

// The same for 8 and for 4 columns.
__device__ __forceinline__ void tmem_ld8(uint32_t tmem_addr, uint32_t (&r)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(tmem_addr));
}
__device__ __forceinline__ void tmem_ld_fence(uint32_t (&r)[8])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7])
                 :: "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t tmem_addr, uint32_t (&r)[4])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(tmem_addr));
}
__device__ __forceinline__ void tmem_ld_fence(uint32_t (&r)[4])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]) :: "memory");
}

}  // namespace umma
}  // namespace invconv

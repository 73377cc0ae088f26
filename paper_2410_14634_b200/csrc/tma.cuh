// Bulk asynchronous copies (TMA, untiled form) and the mbarrier that tracks
// them.  Source, destination and size of a bulk copy must be multiples of 16
// bytes.  No multicast form is used anywhere.
#pragma once

#include <stdint.h>

namespace invconv {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Bounded wait: polls until the phase completes or about one second of SM clock has passed (each poll may
// itself block for a hardware-defined short time), then gives up and reports false.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, unsigned parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > (1ll << 31)) return false;
    }
    return true;
}

// Bounded wait for kernels whose control flow must stay uniform when a wait gives up: `gave_up` is a flag in
// the CTA's shared memory.  The first wait that runs out (about 8 ms of SM clock) sets it; from then on no
// wait of the CTA blocks.  Callers keep running through all of their barriers and report the flag at the end.
__device__ __forceinline__ void mbar_wait_or_give_up(unsigned long long* bar, unsigned parity, volatile int* gave_up)
{
    if (mbar_try_wait(bar, parity)) return;
    if (*gave_up) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*gave_up) return;
        if (clock64() - t0 > (1ll << 24)) { *gave_up = 1; return; }
    }
}

// global -> shared, completion counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, unsigned bytes, unsigned long long* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// shared -> global, tracked by the issuing thread's bulk group.
__device__ __forceinline__ void bulk_s2g(void* dst_gmem, const void* src_smem, unsigned bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_gmem), "r"(smem_u32(src_smem)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

// Wait until the shared-memory source of every committed bulk store has been read.
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Order generic-proxy writes to shared memory before later async-proxy (bulk copy) reads.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Raise the pending byte count of the current phase without arriving.
__device__ __forceinline__ void mbar_expect_tx_only(unsigned long long* bar, unsigned bytes)
{
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(unsigned long long* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Address of this CTA's shared-memory location `local` in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_map_u32(uint32_t local, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    return remote;
}

// Asynchronous 4-byte store into a peer CTA's shared memory; the peer's mbarrier counts the bytes.
__device__ __forceinline__ void st_async_f32(uint32_t remote_addr, float v, uint32_t remote_bar)
{
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.u32 [%0], %1, [%2];" ::"r"(remote_addr),
                 "r"(__float_as_uint(v)), "r"(remote_bar)
                 : "memory");
}

// The same for four consecutive floats (16-byte aligned).
__device__ __forceinline__ void st_async_f32x4(uint32_t remote_addr, float4 v, uint32_t remote_bar)
{
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.u32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(remote_addr),
                 "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)), "r"(__float_as_uint(v.z)), "r"(__float_as_uint(v.w)),
                 "r"(remote_bar)
                 : "memory");
}

// Asynchronous global -> shared copies of 4 and 16 bytes (LDGSTS); `valid == false` writes zeros and reads
// nothing (the source address must still be a mapped one).
__device__ __forceinline__ void cp_async_f32(float* dst_smem, const float* src, bool valid)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(dst_smem)), "l"(src), "r"(valid ? 4 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_f32x4(float* dst_smem, const float* src, bool valid)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst_smem)), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Division by a run-time constant through a precomputed multiplier (valid for n < 2^31).
struct FastDiv {
    unsigned mul, shift, d;
};
__device__ __forceinline__ int fast_div(int n, FastDiv f)
{
    return (int)((__umulhi((unsigned)n, f.mul) + (unsigned)n) >> f.shift);
}


// Host side: the multiplier and shift for fast_div by d >= 1.
inline FastDiv make_fast_div(unsigned d)
{
    FastDiv f;
    f.d = d;
    unsigned sh = 0;
    while ((1ull << sh) < d) ++sh;
    f.shift = sh;
    f.mul = (unsigned)((((1ull << sh) - d) << 32) / d + 1);
    return f;
}

}  // namespace invconv

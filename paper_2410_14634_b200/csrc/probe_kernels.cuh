// Dependent-chain micro-benchmarks: the latency of ONE wavefront step for each
// way a solved diagonal can reach the threads that need it.  They carry no
// other work, so (H+W-1) times the measured step is a lower bound on any
// wavefront schedule built on that mechanism (Section 3.3: the diagonals are
// processed sequentially).
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"
#include "tma.cuh"

namespace invconv {
namespace cg = cooperative_groups;

// Mechanism 0: lane = image row; the newest value of the row above arrives by
// one shuffle and is folded in with one FMA.
__global__ void probe_shuffle_chain(int steps, unsigned long long* out)
{
    float v = 1.0f + 0.001f * threadIdx.x, own = 0.5f;
    const long long t0 = clock64();
    for (int i = 0; i < steps; ++i) {
        const float up = __shfl_up_sync(0xffffffffu, v, 1);
        const float part = fmaf(-0.125f, v, own);     // own-row tap: overlaps the shuffle
        v = fmaf(-0.25f, up, part);                    // the dependent part of the step
    }
    const long long t1 = clock64();
    if (threadIdx.x == 31) { out[0] = (unsigned long long)(t1 - t0); out[1] = (unsigned long long)__float_as_uint(v); }
}

// Mechanism 1: several warps share a diagonal through shared memory with one
// block barrier per step (ping-pong buffers).
__global__ void __launch_bounds__(256) probe_smem_chain(int steps, unsigned long long* out)
{
    __shared__ float buf[2][256];
    float v = 1.0f + 0.001f * threadIdx.x;
    const int up = (threadIdx.x + 255) & 255;
    const long long t0 = clock64();
    for (int i = 0; i < steps; ++i) {
        buf[i & 1][threadIdx.x] = v;
        __syncthreads();
        v = fmaf(-0.25f, buf[i & 1][up], 0.5f);
    }
    const long long t1 = clock64();
    if (threadIdx.x == 0) { out[0] = (unsigned long long)(t1 - t0); out[1] = (unsigned long long)__float_as_uint(v); }
}

// Mechanism 2: the diagonal is split across the two CTAs of a cluster; each
// CTA stores its part into the peer's shared memory and a cluster barrier
// publishes it.
__global__ void __launch_bounds__(128) probe_cluster_chain(int steps, unsigned long long* out)
{
    __shared__ float buf[2][128];
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned peer = cluster.block_rank() ^ 1u;
    float* remote = cluster.map_shared_rank(&buf[0][0], peer);
    float v = 1.0f + 0.001f * threadIdx.x;
    cluster.sync();
    const long long t0 = clock64();
    for (int i = 0; i < steps; ++i) {
        remote[(i & 1) * 128 + threadIdx.x] = v;
        cluster.sync();
        v = fmaf(-0.25f, buf[i & 1][(threadIdx.x + 127) & 127], 0.5f);
    }
    const long long t1 = clock64();
    cluster.sync();      // no CTA leaves while its peer may still write into it
    if (threadIdx.x == 0 && cluster.block_rank() == 0) {
        out[0] = (unsigned long long)(t1 - t0);
        out[1] = (unsigned long long)__float_as_uint(v);
    }
}

// Self-test of the bounded waits: one thread waits, for at most `limit_cycles` SM clock cycles, on an mbarrier
// that nothing ever completes; the wait runs out, the status word is raised and the kernel returns normally.
__global__ void probe_wait_timeout(unsigned limit_cycles)
{
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        bool done = false;
        while (!(done = mbar_try_wait(&bar, 0))) {
            if (clock64() - t0 > (long long)limit_cycles) break;
        }
        if (!done) raise_status(INVCONV_TIMEOUT);
    }
    __syncthreads();
}

}  // namespace invconv

// Dependent-chain micro-benchmarks: the latency of ONE wavefront step for each
// way a solved diagonal can reach the threads that need it.  They carry no
// other work, so (H+W-1) times the measured step is a lower bound on any
// wavefront schedule built on that mechanism (Section 3.3: the diagonals are
// processed sequentially).
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

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

// Mechanism 3: one dependent FMA chain (the latency of a single accumulator).
__global__ void probe_fma_chain(int steps, unsigned long long* out)
{
    float a = 1.0f + 0.001f * threadIdx.x;
    const float w = 0.999f, c = 0.001f;
    const long long t0 = clock64();
#pragma unroll 16
    for (int i = 0; i < steps; ++i) a = fmaf(a, w, c);
    const long long t1 = clock64();
    if (threadIdx.x == 0) { out[0] = (unsigned long long)(t1 - t0); out[1] = (unsigned long long)__float_as_uint(a); }
}

// Mechanism 4: a broadcast 16-byte shared-memory load feeding twelve FMAs on six accumulators (one group of
// the wide-channel kernels' inner loop); cycles per group.
__global__ void probe_group_chain(int steps, unsigned long long* out)
{
    __shared__ __align__(16) float buf[1024];
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) buf[i] = 0.001f * i;
    __syncthreads();
    float acc[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    float w[12];
#pragma unroll
    for (int i = 0; i < 12; ++i) w[i] = 0.01f * (i + 1) + 0.0001f * threadIdx.x;
    const int lane_off = (threadIdx.x >> 3) * 4;
    const long long t0 = clock64();
#pragma unroll 4
    for (int i = 0; i < steps; ++i) {
        const float4 x0 = *reinterpret_cast<const float4*>(buf + ((i * 8 + lane_off) & 1015));
        const float4 x1 = *reinterpret_cast<const float4*>(buf + ((i * 8 + lane_off + 4) & 1015));
        acc[0] = fmaf(w[0], x0.x, acc[0]); acc[1] = fmaf(w[1], x0.x, acc[1]); acc[2] = fmaf(w[2], x0.x, acc[2]);
        acc[3] = fmaf(w[0], x1.x, acc[3]); acc[4] = fmaf(w[1], x1.x, acc[4]); acc[5] = fmaf(w[2], x1.x, acc[5]);
        acc[0] = fmaf(w[3], x0.y, acc[0]); acc[1] = fmaf(w[4], x0.y, acc[1]); acc[2] = fmaf(w[5], x0.y, acc[2]);
        acc[3] = fmaf(w[3], x1.y, acc[3]); acc[4] = fmaf(w[4], x1.y, acc[4]); acc[5] = fmaf(w[5], x1.y, acc[5]);
        acc[0] = fmaf(w[6], x0.z, acc[0]); acc[1] = fmaf(w[7], x0.z, acc[1]); acc[2] = fmaf(w[8], x0.z, acc[2]);
        acc[3] = fmaf(w[6], x1.z, acc[3]); acc[4] = fmaf(w[7], x1.z, acc[4]); acc[5] = fmaf(w[8], x1.z, acc[5]);
        acc[0] = fmaf(w[9], x0.w, acc[0]); acc[1] = fmaf(w[10], x0.w, acc[1]); acc[2] = fmaf(w[11], x0.w, acc[2]);
        acc[3] = fmaf(w[9], x1.w, acc[3]); acc[4] = fmaf(w[10], x1.w, acc[4]); acc[5] = fmaf(w[11], x1.w, acc[5]);
    }
    const long long t1 = clock64();
    float s = acc[0] + acc[1] + acc[2] + acc[3] + acc[4] + acc[5];
    if (threadIdx.x == 0) { out[0] = (unsigned long long)(t1 - t0); out[1] = (unsigned long long)__float_as_uint(s); }
}

// Mechanism 5: the arithmetic of one wavefront step for three channels and a 3x3 kernel, registers only:
// six shuffles, 81 FMAs on 81 per-lane weights, window rotation; no shared memory.
__global__ void probe_step_c3k3(int steps, unsigned long long* out)
{
    float A[81];
#pragma unroll
    for (int i = 0; i < 81; ++i) A[i] = 0.001f * (i + 1) + 0.00001f * threadIdx.x;
    float own[3][2], up[2][3][2];
#pragma unroll
    for (int b = 0; b < 3; ++b)
#pragma unroll
        for (int q = 0; q < 2; ++q) { own[b][q] = 0.1f * b + q; up[0][b][q] = 0.2f; up[1][b][q] = 0.3f; }
    const long long t0 = clock64();
    for (int s0 = 0; s0 < steps; s0 += 2) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            float nu[2][3];
#pragma unroll
            for (int d = 0; d < 2; ++d)
#pragma unroll
                for (int b = 0; b < 3; ++b) nu[d][b] = __shfl_up_sync(0xffffffffu, own[b][(u - 1 - d + 4) % 2], d + 1);
            float acc[3] = {0.5f, 0.25f, 0.125f}, acc2[3] = {0.f, 0.f, 0.f};
#pragma unroll
            for (int dh = 0; dh < 3; ++dh)
#pragma unroll
                for (int dw = (dh == 0 ? 2 : 1); dw < 3; ++dw)
#pragma unroll
                    for (int b = 0; b < 3; ++b) {
                        const int slot = (u - dw + 4) % 2;
                        const float v = dh == 0 ? own[b][slot] : up[dh - 1][b][slot];
#pragma unroll
                        for (int a = 0; a < 3; ++a) {
                            if ((dh * 3 + dw) & 1) acc2[a] = fmaf(-A[((dh * 3 + dw) * 3 + b) * 3 + a], v, acc2[a]);
                            else acc[a] = fmaf(-A[((dh * 3 + dw) * 3 + b) * 3 + a], v, acc[a]);
                        }
                    }
#pragma unroll
            for (int a = 0; a < 3; ++a) acc[a] += acc2[a];
#pragma unroll
            for (int b = 0; b < 3; ++b)
#pragma unroll
                for (int a = 0; a < 3; ++a) acc[a] = fmaf(-A[(6 * 3 + b) * 3 + a], nu[1][b], acc[a]);
#pragma unroll
            for (int b = 0; b < 3; ++b)
#pragma unroll
                for (int a = 0; a < 3; ++a) acc[a] = fmaf(-A[(1 * 3 + b) * 3 + a], own[b][(u - 1 + 4) % 2], acc[a]);
#pragma unroll
            for (int b = 0; b < 3; ++b)
#pragma unroll
                for (int a = 0; a < 3; ++a) acc[a] = fmaf(-A[(3 * 3 + b) * 3 + a], nu[0][b], acc[a]);
#pragma unroll
            for (int b = 0; b < 3; ++b) { own[b][u] = acc[b]; up[0][b][u] = nu[0][b]; up[1][b][u] = nu[1][b]; }
        }
    }
    const long long t1 = clock64();
    if (threadIdx.x == 31) { out[0] = (unsigned long long)(t1 - t0); out[1] = (unsigned long long)__float_as_uint(own[0][0] + own[1][1] + own[2][0]); }
}

}  // namespace invconv

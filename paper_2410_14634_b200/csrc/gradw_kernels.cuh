// Weight gradient for wide channel counts (Theorem 2 in closed form):
//   grad_w[co][ci][K-1-dh][K-1-dw] = - sum_{n,h,w} grad_y[n,co,h,w] * x[n,ci,h-dh,w-dw]
// This is a correlation with contraction length B*H*W -- a batched reduction
// with C*C*K*K outputs, bound by the fp32 FMA pipe.
//
// Output-stationary tiling: a CTA owns one kernel row dh, a 16*TC x 16*TC tile
// of (co, ci) pairs and a share of the batch; thread (tc, ti) keeps the
// TC x TC x K partial sums of its channel pairs in registers.  For every image
// of its share the CTA stages the tile's grad_y and x channel planes in shared
// memory with bulk (TMA) copies -- channel planes are contiguous in NCHW -- and
// walks the rows in quads of four pixels: one 16-byte load per grad_y channel,
// two per x channel (the K-1 columns to the left come with the aligned quad
// before), 4*TC*TC*K FMAs.  The channel planes are padded in shared memory so
// that the 16 threads that differ in ci hit disjoint banks.
// Batch shares write partial sums; gradw_reduce_kernel adds them in a fixed
// order, negates and applies the channel mask.
#pragma once

#include "common.cuh"
#include "tma.cuh"

namespace invconv {

struct GradWParams {
    const float* gy;       // [B][C][H][W]
    const float* x;        // [B][C][H][W]
    float* partials;       // [nbc][K*K][C][C]   (tap = dh*K + dw, then co, then ci)
    int B, C, H, W;
    int nbc;               // batch shares
    int tiles;             // channel tiles per side
    int plane;             // floats per channel plane in shared memory (H*W + padding)
};

template <int TC, int K>
__global__ void __launch_bounds__(256) gradw_tile_kernel(GradWParams p)
{
    extern __shared__ __align__(128) float smem[];
    __shared__ unsigned long long bar;
    constexpr int TB = 16 * TC;                 // channels per tile side
    const int H = p.H, W = p.W, HW = H * W, C = p.C;
    const int tid = threadIdx.x;
    const int tc = tid >> 4, ti = tid & 15;
    int bid = blockIdx.x;
    const int share = bid % p.nbc; bid /= p.nbc;
    const int tci = bid % p.tiles; bid /= p.tiles;
    const int tco = bid % p.tiles; bid /= p.tiles;
    const int dh = bid;
    const int co0 = tco * TB, ci0 = tci * TB;
    const int nco = min(TB, C - co0), nci = min(TB, C - ci0);
    float* gys = smem;                          // [TB][plane]
    float* xs = smem + TB * p.plane;            // [TB][plane]

    float acc[TC][TC][K];
#pragma unroll
    for (int i = 0; i < TC; ++i)
#pragma unroll
        for (int j = 0; j < TC; ++j)
#pragma unroll
            for (int d = 0; d < K; ++d) acc[i][j][d] = 0.f;

    if (tid == 0) { mbar_init(&bar, 1); fence_mbar_init(); }
    for (int i = tid; i < 2 * TB * p.plane; i += blockDim.x) smem[i] = 0.f;   // channels beyond C stay zero
    __syncthreads();

    unsigned phase = 0;
    bool ok = true;
    for (int n = share; n < p.B; n += p.nbc) {
        if (tid < 32) {
            // one warp issues the per-channel bulk copies of this image's two tiles
            fence_proxy_async();
            if (tid == 0) mbar_expect_tx(&bar, (unsigned)((nco + nci) * HW * 4));
            __syncwarp();
            const float* gsrc = p.gy + ((size_t)n * C + co0) * HW;
            const float* xsrc = p.x + ((size_t)n * C + ci0) * HW;
            for (int c = tid; c < nco; c += 32) bulk_g2s(gys + c * p.plane, gsrc + (size_t)c * HW, (unsigned)HW * 4u, &bar);
            for (int c = tid; c < nci; c += 32) bulk_g2s(xs + c * p.plane, xsrc + (size_t)c * HW, (unsigned)HW * 4u, &bar);
        }
        ok = mbar_wait_bounded(&bar, phase);
        phase ^= 1u;
        if (!__syncthreads_and(ok)) { if (tid == 0) raise_status(INVCONV_TIMEOUT); break; }

        const float* gq[TC];
        const float* xq[TC];
#pragma unroll
        for (int i = 0; i < TC; ++i) gq[i] = gys + (tc * TC + i) * p.plane;
#pragma unroll
        for (int j = 0; j < TC; ++j) xq[j] = xs + (ti * TC + j) * p.plane;
        for (int h = dh; h < H; ++h) {
            for (int w0 = 0; w0 < W; w0 += 4) {
                float g[TC][4], v[TC][8];
#pragma unroll
                for (int i = 0; i < TC; ++i) {
                    const float4 t = *reinterpret_cast<const float4*>(gq[i] + h * W + w0);
                    g[i][0] = t.x; g[i][1] = t.y; g[i][2] = t.z; g[i][3] = t.w;
                }
#pragma unroll
                for (int j = 0; j < TC; ++j) {
                    const float* row = xq[j] + (h - dh) * W + w0;
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (K > 1 && w0 > 0) a = *reinterpret_cast<const float4*>(row - 4);
                    const float4 b = *reinterpret_cast<const float4*>(row);
                    v[j][0] = a.x; v[j][1] = a.y; v[j][2] = a.z; v[j][3] = a.w;
                    v[j][4] = b.x; v[j][5] = b.y; v[j][6] = b.z; v[j][7] = b.w;
                }
#pragma unroll
                for (int d = 0; d < K; ++d)
#pragma unroll
                    for (int px = 0; px < 4; ++px)
#pragma unroll
                        for (int i = 0; i < TC; ++i)
#pragma unroll
                            for (int j = 0; j < TC; ++j)
                                acc[i][j][d] = fmaf(g[i][px], v[j][4 + px - d], acc[i][j][d]);
            }
        }
        __syncthreads();       // everyone is done with this image before its planes are overwritten
    }

    float* dst = p.partials + (size_t)share * K * K * C * C;
#pragma unroll
    for (int i = 0; i < TC; ++i)
#pragma unroll
        for (int j = 0; j < TC; ++j) {
            const int co = co0 + tc * TC + i, ci = ci0 + ti * TC + j;
            if (co < C && ci < C) {
#pragma unroll
                for (int d = 0; d < K; ++d) dst[((size_t)(dh * K + d) * C + co) * C + ci] = acc[i][j][d];
            }
        }
}

// grad_w[co][ci][K-1-dh][K-1-dw] = -(sum over shares), zero outside the channel mask of the centre tap.
__global__ void __launch_bounds__(256) gradw_reduce_kernel(const float* __restrict__ partials, float* __restrict__ grad_w,
                                                           int nbc, int C, int K)
{
    const int NA = K * K * C * C;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < NA; e += gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int b = 0; b < nbc; ++b) s += __ldcg(partials + (size_t)b * NA + e);
        const int ci = e % C, co = (e / C) % C, tap = e / (C * C);
        const int dh = tap / K, dw = tap % K;
        grad_w[((co * C + ci) * K + (K - 1 - dh)) * K + (K - 1 - dw)] = (tap == 0 && ci > co) ? 0.f : -s;
    }
}

struct GradWPlan {
    bool ok = false;
    int TC = 3, tiles = 1, nbc = 1, plane = 0, grid = 0;
    size_t smem = 0;
};

inline GradWPlan plan_gradw(int B, int C, int H, int W, int K, size_t max_smem, int sm_count)
{
    GradWPlan pl;
    if (!(K == 1 || K == 2 || K == 3 || K == 5)) return pl;
    if (W % 4 != 0 || B < 1) return pl;
    pl.TC = C <= 16 ? 1 : 3;
    const int TB = 16 * pl.TC;
    pl.tiles = (C + TB - 1) / TB;
    const int HW = H * W;
    int pad = 0;
    for (; pad < 32; pad += 4) {
        const int m = (pl.TC * (HW + pad)) % 32;
        if (m % 8 == 4) break;
    }
    if (pad >= 32) pad = 4;
    pl.plane = HW + pad;
    pl.smem = sizeof(float) * 2 * (size_t)TB * pl.plane;
    if (pl.smem > max_smem) return pl;
    int nbc = (2 * sm_count) / (K * pl.tiles * pl.tiles);
    if (nbc < 1) nbc = 1;
    if (nbc > B) nbc = B;
    // even out the images per share
    const int per = (B + nbc - 1) / nbc;
    nbc = (B + per - 1) / per;
    pl.nbc = nbc;
    pl.grid = K * pl.tiles * pl.tiles * nbc;
    pl.ok = true;
    return pl;
}

}  // namespace invconv

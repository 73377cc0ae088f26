// y = f(x): the masked, top-left-padded convolution itself (Eq. 1 over channels;
// the sampling direction, Section 4.3) for few channels.
//
// A few warps per image, each a band of rows.  The image arrives in shared memory by one bulk (TMA)
// copy; lane = column, a warp walks down its rows keeping a K x K window of x
// per input channel in registers (one new row of K values per step, the window
// rotates by register renaming), so every output pixel costs C*K shared-memory
// loads for C*C*K*K FMAs, and each (channel, row) of y leaves as one coalesced
// 128-byte store.  The channel mask of the bottom-right tap is applied while the
// kernel is read.  Bound: HBM (8 bytes per element).
#pragma once

#include "common.cuh"
#include "tma.cuh"

namespace invconv {

struct ConvParams {
    const float* x;
    const float* w;
    float* y;
    int B, H, W;
    int ipc;       // images per CTA
    int wpi;       // warps per image (row bands)
    int bulk;      // images are 16-byte aligned multiples of 16 bytes
};

template <int C, int K>
__global__ void __launch_bounds__(256) masked_conv_warp_kernel(ConvParams p)
{
    extern __shared__ __align__(128) float smem[];
    constexpr int NW = C * C * K * K;
    constexpr bool WREG = NW <= 108;
    const int H = p.H, W = p.W, HW = H * W, CHW = C * HW;
    const int imgf = (CHW + 31) & ~31;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int li = warp / p.wpi, wb = warp - li * p.wpi;
    const int n = blockIdx.x * p.ipc + li;
    const bool has_img = n < p.B;
    const int band = (H + p.wpi - 1) / p.wpi;
    const int hb0 = wb * band, hb1 = min(H, hb0 + band);
    float* ws = smem;                                                   // masked kernel [co][ci][dh][dw]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + ((NW + 31) & ~31));
    float* xs = smem + ((NW + 31) & ~31) + 32 + li * imgf;

    if (has_img && p.bulk && wb == 0 && lane == 0) {
        mbar_init(&bars[li], 1);
        fence_mbar_init();
        mbar_expect_tx(&bars[li], (unsigned)CHW * 4u);
        bulk_g2s(xs, p.x + (size_t)n * CHW, (unsigned)CHW * 4u, &bars[li]);
    }
    if (has_img && !p.bulk) {
        const float* src = p.x + (size_t)n * CHW;
        for (int i = wb * 32 + lane; i < CHW; i += p.wpi * 32) xs[i] = __ldg(src + i);
    }
    for (int e = threadIdx.x; e < NW; e += blockDim.x) {
        const int dw = e % K, dh = (e / K) % K, ci = (e / (K * K)) % C, co = e / (K * K * C);
        const bool masked_out = (dh == 0 && dw == 0 && ci > co);
        ws[e] = masked_out ? 0.f : __ldg(p.w + ((co * C + ci) * K + (K - 1 - dh)) * K + (K - 1 - dw));
    }
    __syncthreads();
    if (!has_img) return;
    float wr[WREG ? NW : 1];
    if constexpr (WREG) {
#pragma unroll
        for (int e = 0; e < NW; ++e) wr[e] = ws[e];
    }
    if (p.bulk) {
        const bool ok = mbar_wait_bounded(&bars[li], 0);
        if (!__all_sync(0xffffffffu, ok)) { if (lane == 0) raise_status(INVCONV_TIMEOUT); return; }
    }
    float* dst = p.y + (size_t)n * CHW;
    for (int w0 = 0; w0 < W; w0 += 32) {
        const int w = w0 + lane;
        const bool col_ok = w < W;
        float xr[K][C][K];
#pragma unroll
        for (int r = 0; r < K; ++r)
#pragma unroll
            for (int ci = 0; ci < C; ++ci)
#pragma unroll
                for (int dw = 0; dw < K; ++dw) xr[r][ci][dw] = 0.f;
#pragma unroll
        for (int q = 1; q < K; ++q) {                     // the K-1 rows above the band
            const int row = hb0 - q;
#pragma unroll
            for (int ci = 0; ci < C; ++ci)
#pragma unroll
                for (int dw = 0; dw < K; ++dw) {
                    const bool in = row >= 0 && col_ok && w - dw >= 0;
                    const float t = xs[ci * HW + (in ? row * W + w - dw : 0)];
                    xr[(K - q) % K][ci][dw] = in ? t : 0.f;
                }
        }
        for (int hb = hb0; hb < hb1; hb += K) {
#pragma unroll
            for (int r = 0; r < K; ++r) {
                const int h = hb + r;
                if (h < hb1) {
#pragma unroll
                    for (int ci = 0; ci < C; ++ci)
#pragma unroll
                        for (int dw = 0; dw < K; ++dw) {
                            const bool in = col_ok && w - dw >= 0;
                            const float t = xs[ci * HW + h * W + (in ? w - dw : 0)];      // clamped: no branch
                            xr[r][ci][dw] = in ? t : 0.f;
                        }
                    float acc[C];
#pragma unroll
                    for (int co = 0; co < C; ++co) acc[co] = 0.f;
#pragma unroll
                    for (int co = 0; co < C; ++co)
#pragma unroll
                        for (int ci = 0; ci < C; ++ci)
#pragma unroll
                            for (int dh = 0; dh < K; ++dh)
#pragma unroll
                                for (int dw = 0; dw < K; ++dw) {
                                    const int e = ((co * C + ci) * K + dh) * K + dw;
                                    const float wv = WREG ? wr[WREG ? e : 0] : ws[e];
                                    acc[co] = fmaf(wv, xr[(r - dh + K) % K][ci][dw], acc[co]);
                                }
                    if (col_ok) {
#pragma unroll
                        for (int co = 0; co < C; ++co) dst[co * HW + h * W + w] = acc[co];
                    }
                }
            }
        }
    }
}

template <int C, int K>
inline size_t masked_conv_smem(int H, int W, int ipc)
{
    const size_t imgf = ((size_t)C * H * W + 31) & ~(size_t)31;
    return sizeof(float) * ((((size_t)C * C * K * K + 31) & ~(size_t)31) + 32 + imgf * ipc);
}

}  // namespace invconv

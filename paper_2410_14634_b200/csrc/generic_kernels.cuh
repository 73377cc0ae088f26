// Shape-agnostic kernels: correct for every (B, C, H, W, k) within the limits,
// with all operands in global memory.  They are the fallback of the dispatcher
// and the in-library cross-check of the specialised families.
#pragma once

#include "common.cuh"

namespace invconv {

// ---------------------------------------------------------------------------
// Wavefront substitution, one CTA per image (Section 3: the H+W-1
// anti-diagonals are visited in order, everything on one diagonal in parallel;
// Algorithm 1's schedule with a block barrier in place of "synchronize all
// threads").
//
// BWD = false:  solve  M x = rhs          (x = f^{-1}(y), Eq. 1 rearranged)
// BWD = true :  solve  M^T g = rhs        (grad_y = M^{-T} grad_x, Theorem 1 / Eq. 2)
// The transposed solve is the same walk on the image rotated by 180 degrees
// with the channel pair of every kernel entry swapped and channels visited in
// descending order.
//
// Per diagonal: phase A subtracts every off-centre tap (all channels, pixels on
// earlier diagonals) and parks the residual in `out`; phase B solves the small
// triangular channel system of the centre tap, one thread per pixel.
// ---------------------------------------------------------------------------
template <bool BWD>
__global__ void __launch_bounds__(256)
generic_wavefront_kernel(const float* __restrict__ rhs, const float* __restrict__ wgt,
                         float* out, Geom g)
{
    const int C = g.C, H = g.H, W = g.W, k = g.k;
    const size_t img = (size_t)blockIdx.x * C * H * W;
    const float* rhs_i = rhs + img;
    float* out_i = out + img;
    const int ctr = (k - 1) * k + (k - 1);
    const int kk = k * k;

    for (int d = 0; d < H + W - 1; ++d) {
        const int hlo = max(0, d - (W - 1));
        const int hhi = min(H - 1, d);
        const int npix = hhi - hlo + 1;

        for (int idx = threadIdx.x; idx < npix * C; idx += blockDim.x) {
            const int pix = idx / C;
            const int c = idx - pix * C;
            const int lh = hlo + pix, lw = d - lh;              // logical (rotated for BWD) pixel
            const int h = BWD ? H - 1 - lh : lh;
            const int w = BWD ? W - 1 - lw : lw;
            float acc = rhs_i[(c * H + h) * W + w];
            for (int c2 = 0; c2 < C; ++c2) {
                const float* wrow = BWD ? wgt + (size_t)(c2 * C + c) * kk : wgt + (size_t)(c * C + c2) * kk;
                for (int dh = 0; dh < k; ++dh) {
                    if (lh - dh < 0) break;
                    for (int dw = 0; dw < k; ++dw) {
                        if (lw - dw < 0) break;
                        if ((dh | dw) == 0) continue;
                        const int hh = BWD ? h + dh : h - dh;
                        const int wq = BWD ? w + dw : w - dw;
                        acc -= wrow[(k - 1 - dh) * k + (k - 1 - dw)] * __ldcg(out_i + (c2 * H + hh) * W + wq);
                    }
                }
            }
            __stcg(out_i + (c * H + h) * W + w, acc);
        }
        __syncthreads();

        for (int pix = threadIdx.x; pix < npix; pix += blockDim.x) {
            const int lh = hlo + pix, lw = d - lh;
            const int h = BWD ? H - 1 - lh : lh;
            const int w = BWD ? W - 1 - lw : lw;
            for (int i = 0; i < C; ++i) {
                const int c = BWD ? C - 1 - i : i;
                float v = __ldcg(out_i + (c * H + h) * W + w);
                for (int j = 0; j < i; ++j) {
                    const int c2 = BWD ? C - 1 - j : j;
                    const float t = BWD ? wgt[(size_t)(c2 * C + c) * kk + ctr] : wgt[(size_t)(c * C + c2) * kk + ctr];
                    v -= t * __ldcg(out_i + (c2 * H + h) * W + w);
                }
                v /= wgt[(size_t)(c * C + c) * kk + ctr];
                __stcg(out_i + (c * H + h) * W + w, v);
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------
// grad_w, one CTA per kernel entry (Theorem 2 in closed form):
//   grad_w[co][ci][k-1-dh][k-1-dw] = -sum_{n,h,w} grad_y[n,co,h,w] * x[n,ci,h-dh,w-dw]
// Entries outside the channel mask of the centre tap are written as 0.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
generic_grad_w_kernel(const float* __restrict__ grad_y, const float* __restrict__ x,
                      float* __restrict__ grad_w, Geom g, const LogdetFuse ld)
{
    const int C = g.C, H = g.H, W = g.W, k = g.k;
    int e = blockIdx.x;
    const int b = e % k; e /= k;
    const int a = e % k; e /= k;
    const int ci = e % C;
    const int co = e / C;
    const int dh = k - 1 - a, dw = k - 1 - b;
    const bool masked_out = (dh == 0 && dw == 0 && ci > co);

    float acc = 0.f;
    if (!masked_out && dh < H && dw < W) {
        const int hh = H - dh, ww = W - dw;
        const int per_img = hh * ww;
        const long long total = (long long)g.B * per_img;
        for (long long t = threadIdx.x; t < total; t += blockDim.x) {
            const int n = (int)(t / per_img);
            const int r = (int)(t - (long long)n * per_img);
            const int h = dh + r / ww, w = dw + r % ww;
            acc += grad_y[act_index(n, co, h, w, C, H, W)] * x[act_index(n, ci, h - dh, w - dw, C, H, W)];
        }
    }
    __shared__ float red[128];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int s = 64; s > 0; s >>= 1) {
        if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) grad_w[blockIdx.x] = finish_grad_w(red[0], co, ci, dh * k + dw, C, k, ld);
}

// ---------------------------------------------------------------------------
// y = f(x), one thread per output element (Eq. 1 over channels).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
generic_masked_conv_kernel(const float* __restrict__ x, const float* __restrict__ wgt,
                           float* __restrict__ y, Geom g, long long total)
{
    const int C = g.C, H = g.H, W = g.W, k = g.k;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const int w = (int)(t % W);
        long long r = t / W;
        const int h = (int)(r % H); r /= H;
        const int co = (int)(r % C);
        const int n = (int)(r / C);
        float acc = 0.f;
        for (int ci = 0; ci < C; ++ci) {
            const float* wrow = wgt + (size_t)(co * C + ci) * k * k;
            const float* xi = x + ((size_t)n * C + ci) * H * W;
            for (int dh = 0; dh < k && dh <= h; ++dh)
                for (int dw = 0; dw < k && dw <= w; ++dw) {
                    if ((dh | dw) == 0 && ci > co) continue;
                    acc += wrow[(k - 1 - dh) * k + (k - 1 - dw)] * __ldg(xi + (h - dh) * W + (w - dw));
                }
        }
        y[t] = acc;
    }
}

// ---------------------------------------------------------------------------
// logdet = H*W*sum_c log|w[c][c][k-1][k-1]|, one warp, double accumulation.
// ---------------------------------------------------------------------------
__global__ void logdet_kernel(const float* __restrict__ wgt, float* __restrict__ out, int C, int H, int W, int k)
{
    double s = 0.0;
    for (int c = threadIdx.x; c < C; c += 32)
        s += log(fabs((double)wgt[w_index(c, c, k - 1, k - 1, C, k)]));
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (threadIdx.x == 0) out[0] = (float)((double)H * (double)W * s);
}

// grad_w[c][c][k-1][k-1] += grad_logdet * H*W / w[c][c][k-1][k-1]: the derivative of grad_logdet * logdet.
__global__ void logdet_grad_kernel(const float* __restrict__ wgt, const float* __restrict__ grad_logdet,
                                   float* __restrict__ grad_w, int C, int H, int W, int k)
{
    const float g = grad_logdet[0] * (float)H * (float)W;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const int i = w_index(c, c, k - 1, k - 1, C, k);
        grad_w[i] += g / wgt[i];
    }
}

}  // namespace invconv

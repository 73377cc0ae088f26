// The inverse convolution together with the two layers that follow it in one step of the paper's
// Inverse-Flow model (Section 4, Fig. 3): Actnorm, z = s*x + b per channel, and the 1x1 convolution,
// u = V z per pixel.  Both act on one pixel at a time.  For the few-channel (warp) family they are applied
// inside the wavefront kernel while the image is in shared memory -- u is written beside x in the store
// epilogue, and grad_x = s * (V^T grad_u) is formed in the load prologue of the transposed solve -- so that x
// is not read back from memory; for the other families the step is composed from the layer's kernels and the
// per-pixel kernels below (the image is then still in L2).  The parameter gradients of the neighbours are sums
// over pixels of grad_u x^T and grad_u, reduced in a fixed order.
#include <cuda_runtime.h>

#include <cstdio>

#include "invconv.h"

#include "common.cuh"
#include "lib_internal.h"

using namespace invconv;
using invconv_internal::check_launch;

namespace {

constexpr int kMixPixels = 64;      // pixels per CTA tile of the per-pixel kernels

// out[n][o][p] = sum_c A[o][c] * in[n][c][p] + cb[o]  with
//   forward : A = V diag(s), cb = V b   (u from x)
//   backward: A = diag(s) V^T, cb = 0   (grad_x from grad_u)
// One CTA per (image, tile of 64 pixels); the input tile and A are staged in shared memory.
template <bool BWD>
__global__ void __launch_bounds__(256) flow_mix_kernel(const float* __restrict__ in, const float* __restrict__ V,
                                                       const float* __restrict__ s, const float* __restrict__ b,
                                                       float* __restrict__ out, int C, int HW, int tiles)
{
    extern __shared__ __align__(16) float fsm[];
    float* A = fsm;                         // [C][C + 1]
    float* cb = A + C * (C + 1);            // [C]
    float* tile = cb + C;                   // [C][kMixPixels]
    const int n = blockIdx.x / tiles, t0 = (blockIdx.x - n * tiles) * kMixPixels;
    const int np = min(kMixPixels, HW - t0);
    for (int e = threadIdx.x; e < C * C; e += blockDim.x) {
        const int o = e / C, c = e - o * C;
        A[o * (C + 1) + c] = BWD ? __ldg(s + o) * __ldg(V + c * C + o) : __ldg(V + o * C + c) * __ldg(s + c);
    }
    for (int o = threadIdx.x; o < C; o += blockDim.x) {
        float acc = 0.f;
        if (!BWD) for (int c = 0; c < C; ++c) acc = fmaf(__ldg(V + o * C + c), __ldg(b + c), acc);
        cb[o] = acc;
    }
    const float* src = in + (size_t)n * C * HW + t0;
    for (int e = threadIdx.x; e < C * kMixPixels; e += blockDim.x) {
        const int c = e / kMixPixels, p = e - c * kMixPixels;
        tile[e] = p < np ? __ldg(src + (size_t)c * HW + p) : 0.f;
    }
    __syncthreads();
    float* dst = out + (size_t)n * C * HW + t0;
    for (int e = threadIdx.x; e < C * kMixPixels; e += blockDim.x) {
        const int o = e / kMixPixels, p = e - o * kMixPixels;
        float acc = cb[o];
        for (int c = 0; c < C; ++c) acc = fmaf(A[o * (C + 1) + c], tile[c * kMixPixels + p], acc);
        if (p < np && INVCONV_CHECKED((size_t)n * C * HW + t0 + (size_t)o * HW + p, (size_t)gridDim.x / tiles * C * HW, 401))
            dst[(size_t)o * HW + p] = acc;
    }
}

// Partial sums over a share of the (image, pixel tile) items:
//   G1[o][c] = sum grad_u[n][o][p] * x[n][c][p],   g0[o] = sum grad_u[n][o][p]
// partials[share][C*C + C] (double).  Thread (o, c-lane) walks the pixels of a staged tile.  With few channels there are
// few entries, each one long sum that may cancel almost completely (and nothing larger to be measured against), so a
// thread that owns at most four entries adds the exact fp32 products in double; with many channels the sums
// stay fp32 (up to 68 per thread).
__global__ void __launch_bounds__(256) flow_mix_grad_kernel(const float* __restrict__ gu, const float* __restrict__ x,
                                                            double* __restrict__ partials, int B, int C, int HW, int tiles)
{
    extern __shared__ __align__(16) float fsm[];
    float* tg = fsm;                              // [C][kMixPixels + 1]
    float* tx = tg + C * (kMixPixels + 1);        // [C][kMixPixels + 1]
    const int items = B * tiles, NE = C * C + C;
    const int per = (NE + blockDim.x - 1) / blockDim.x;     // entries per thread (at most 65 for C = 128)
    const bool wide_acc = per <= 4;
    float acc[68];
    double dacc[4] = {0.0, 0.0, 0.0, 0.0};
    for (int q = 0; q < 68; ++q) acc[q] = 0.f;
    for (int it = blockIdx.x; it < items; it += gridDim.x) {
        const int n = it / tiles, t0 = (it - n * tiles) * kMixPixels;
        const int np = min(kMixPixels, HW - t0);
        const float* sg = gu + (size_t)n * C * HW + t0;
        const float* sx = x + (size_t)n * C * HW + t0;
        __syncthreads();
        for (int e = threadIdx.x; e < C * kMixPixels; e += blockDim.x) {
            const int c = e / kMixPixels, p = e - c * kMixPixels;
            tg[c * (kMixPixels + 1) + p] = p < np ? __ldg(sg + (size_t)c * HW + p) : 0.f;
            tx[c * (kMixPixels + 1) + p] = p < np ? __ldg(sx + (size_t)c * HW + p) : 0.f;
        }
        __syncthreads();
        if (wide_acc) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int e = threadIdx.x + q * blockDim.x;
                if (q >= per || e >= NE) break;
                double a = dacc[q];
                if (e < C * C) {
                    const int o = e / C, c = e - o * C;
                    const float* pg = tg + o * (kMixPixels + 1);
                    const float* px = tx + c * (kMixPixels + 1);
                    for (int p = 0; p < kMixPixels; ++p) a = fma((double)pg[p], (double)px[p], a);
                } else {
                    const float* pg = tg + (e - C * C) * (kMixPixels + 1);
                    for (int p = 0; p < kMixPixels; ++p) a += (double)pg[p];
                }
                dacc[q] = a;
            }
            continue;
        }
        for (int q = 0; q < per; ++q) {
            const int e = threadIdx.x + q * blockDim.x;
            if (e >= NE) break;
            float a = acc[q];
            if (e < C * C) {
                const int o = e / C, c = e - o * C;
                const float* pg = tg + o * (kMixPixels + 1);
                const float* px = tx + c * (kMixPixels + 1);
                for (int p = 0; p < kMixPixels; ++p) a = fmaf(pg[p], px[p], a);
            } else {
                const float* pg = tg + (e - C * C) * (kMixPixels + 1);
                for (int p = 0; p < kMixPixels; ++p) a += pg[p];
            }
            acc[q] = a;
        }
    }
    for (int q = 0; q < per; ++q) {
        const int e = threadIdx.x + q * blockDim.x;
        if (e < NE) partials[(size_t)blockIdx.x * NE + e] = wide_acc ? dacc[q < 4 ? q : 0] : (double)acc[q];
    }
}

// Sums the shares in order and forms the parameter gradients:
//   grad_V[o][c] = s[c] * G1[o][c] + b[c] * g0[o];  grad_s[c] = sum_o V[o][c] * G1[o][c];  grad_b[c] = sum_o V[o][c] * g0[o].
__global__ void __launch_bounds__(256) flow_mix_grad_final_kernel(const double* __restrict__ partials, int shares,
                                                                  const float* __restrict__ V, const float* __restrict__ s,
                                                                  const float* __restrict__ b, float* __restrict__ grad_V,
                                                                  float* __restrict__ grad_s, float* __restrict__ grad_b, int C)
{
    extern __shared__ __align__(16) double fsmd[];
    double* G = fsmd;                 // [C*C + C]
    const int NE = C * C + C;
    for (int e = threadIdx.x; e < NE; e += blockDim.x) {
        double a = 0.0;
        for (int sh = 0; sh < shares; ++sh) a += __ldcg(partials + (size_t)sh * NE + e);
        G[e] = a;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < C * C; e += blockDim.x) {
        const int o = e / C, c = e - o * C;
        grad_V[e] = (float)((double)__ldg(s + c) * G[e] + (double)__ldg(b + c) * G[C * C + o]);
    }
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        double gs = 0.0, gb = 0.0;
        for (int o = 0; o < C; ++o) {
            const double v = (double)__ldg(V + o * C + c);
            gs += v * G[o * C + c];
            gb += v * G[C * C + o];
        }
        grad_s[c] = (float)gs;
        grad_b[c] = (float)gb;
    }
}

// logdet[0] = H*W * ( -sum_c log|w[c][c][k-1][k-1]| + sum_c log|s[c]| + log|det V| ), in double; the determinant by
// Gaussian elimination with partial pivoting in shared memory (one CTA, C <= 128).
__global__ void __launch_bounds__(128) flow_logdet_kernel(const float* __restrict__ w, const float* __restrict__ s,
                                                          const float* __restrict__ V, float* __restrict__ logdet,
                                                          int C, int H, int W, int K)
{
    extern __shared__ __align__(16) double dsm[];
    double* M = dsm;                  // [C][C]
    __shared__ int piv;
    __shared__ double acc;
    const int tid = threadIdx.x;
    for (int e = tid; e < C * C; e += blockDim.x) M[e] = (double)__ldg(V + e);
    if (tid == 0) {
        double a = 0.0;
        for (int c = 0; c < C; ++c)
            a += log(fabs((double)__ldg(s + c))) - log(fabs((double)__ldg(w + ((size_t)(c * C + c) * K + (K - 1)) * K + (K - 1))));
        acc = a;
    }
    __syncthreads();
    for (int j = 0; j < C; ++j) {
        if (tid == 0) {
            int best = j;
            double bv = fabs(M[j * C + j]);
            for (int i = j + 1; i < C; ++i)
                if (fabs(M[i * C + j]) > bv) { bv = fabs(M[i * C + j]); best = i; }
            piv = best;
        }
        __syncthreads();
        if (piv != j)
            for (int c = tid; c < C; c += blockDim.x) { const double t = M[j * C + c]; M[j * C + c] = M[piv * C + c]; M[piv * C + c] = t; }
        __syncthreads();
        const double d = M[j * C + j];
        if (tid == 0) acc += log(fabs(d));
        for (int i = j + 1 + tid; i < C; i += blockDim.x) {
            const double f = M[i * C + j] / d;
            for (int c = j + 1; c < C; ++c) M[i * C + c] -= f * M[j * C + c];
        }
        __syncthreads();
    }
    if (tid == 0) logdet[0] = (float)((double)(H * W) * acc);
}

struct Scratch {
    void* p = nullptr;
    cudaStream_t st = nullptr;
    int acquire(size_t bytes, cudaStream_t s)
    {
        st = s;
        if (bytes == 0) return INVCONV_OK;
        { const int rc = invconv_internal::scratch_alloc(&p, bytes, st); if (rc) { p = nullptr; return rc; } }
        if (cudaMemsetAsync(p, 0, INVCONV_WS_CONTROL_BYTES, st) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
        return INVCONV_OK;
    }
    ~Scratch() { if (p) cudaFreeAsync(p, st); }
};

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

template <bool BWD>
int launch_mix(const float* in, const float* V, const float* s, const float* b, float* out, int B, int C, int HW, cudaStream_t st)
{
    const int tiles = (HW + kMixPixels - 1) / kMixPixels;
    const size_t sm = sizeof(float) * ((size_t)C * (C + 1) + C + (size_t)C * kMixPixels);
    auto kern = flow_mix_kernel<BWD>;
    const int rc = invconv_internal::set_smem_limit(kern, sm);
    if (rc) return rc;
    kern<<<B * tiles, 256, sm, st>>>(in, V, s, b, out, C, HW, tiles);
    return check_launch();
}

}  // namespace

namespace invconv_internal {

int flow_read_clear_status(int* status_out)
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    if (v != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
    }
    *status_out = v;
    return INVCONV_OK;
}

int flow_bounds_info(int* info)
{
#ifdef INVCONV_DEBUG_BOUNDS
    const int zero[4] = {0, 0, 0, 0};
    if (cudaMemcpyFromSymbol(info, g_bounds_record, 4 * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    cudaMemcpyToSymbol(g_bounds_record, zero, sizeof(zero));
#else
    info[0] = info[1] = info[2] = info[3] = 0;
#endif
    return INVCONV_OK;
}

}  // namespace invconv_internal

extern "C" {

int invconv_flow_step_forward(const float* y, const float* w, const float* s, const float* b, const float* V,
                              float* x, float* u, float* logdet, int B, int C, int H, int W, int k, void* stream)
{
    if (B < 0 || C < 1 || H < 1 || W < 1 || k < 1) return INVCONV_BAD_ARG;
    if (k > INVCONV_MAX_K || C > INVCONV_MAX_C) return INVCONV_UNSUPPORTED;
    if (!w || !s || !b || !V) return INVCONV_BAD_ARG;
    if (B > 0 && (!y || !x || !u || y == x || u == x || u == y)) return INVCONV_BAD_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (B > 0) {
        Scratch sc;
        const size_t need = invconv_workspace_bytes(B, C, H, W, k);
        const int ra = sc.acquire(need, st);
        if (ra) return ra;
        int rc = invconv_internal::warp_step_forward(y, w, s, b, V, x, u, Geom{B, C, H, W, k}, sc.p, st);
        if (rc == INVCONV_UNSUPPORTED) {
            rc = invconv_forward_ws(y, w, x, B, C, H, W, k, sc.p, need, stream);
            if (rc) return rc;
            rc = launch_mix<false>(x, V, s, b, u, B, C, H * W, st);
        }
        if (rc) return rc;
    }
    if (logdet) {
        auto kern = flow_logdet_kernel;
        const size_t sm = sizeof(double) * (size_t)C * C;
        const int rc = invconv_internal::set_smem_limit(kern, sm);
        if (rc) return rc;
        kern<<<1, 128, sm, st>>>(w, s, V, logdet, C, H, W, k);
        return check_launch();
    }
    return INVCONV_OK;
}

int invconv_flow_step_backward(const float* grad_u, const float* x, const float* w, const float* s, const float* b,
                               const float* V, float* grad_y, float* grad_w, float* grad_s, float* grad_b, float* grad_V,
                               int B, int C, int H, int W, int k, void* stream)
{
    if (B < 0 || C < 1 || H < 1 || W < 1 || k < 1) return INVCONV_BAD_ARG;
    if (k > INVCONV_MAX_K || C > INVCONV_MAX_C) return INVCONV_UNSUPPORTED;
    if (!w || !s || !b || !V || !grad_w || !grad_s || !grad_b || !grad_V) return INVCONV_BAD_ARG;
    if (B > 0 && (!grad_u || !x || !grad_y || grad_u == grad_y || x == grad_y)) return INVCONV_BAD_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int HW = H * W;
    const size_t act = up256(sizeof(float) * (size_t)B * C * HW);
    const size_t need = up256(invconv_workspace_bytes(B > 0 ? B : 1, C, H, W, k) + INVCONV_WS_CONTROL_BYTES);
    const int tiles = (HW + kMixPixels - 1) / kMixPixels;
    int shares = invconv_internal::sm_count() * 2;
    if (shares > B * tiles) shares = B * tiles;
    if (shares < 1) shares = 1;
    const size_t NE = (size_t)C * C + C;
    const size_t part = up256(sizeof(double) * NE * shares);
    Scratch sc;
    const int ra = sc.acquire(need + act + part, st);
    if (ra) return ra;
    char* base = static_cast<char*>(sc.p);
    float* grad_x = reinterpret_cast<float*>(base + need);
    double* partials = reinterpret_cast<double*>(base + need + act);
    int rc = INVCONV_OK;
    if (B > 0) {
        rc = invconv_internal::warp_step_backward(grad_u, x, w, s, V, grad_y, grad_w, Geom{B, C, H, W, k}, sc.p, st);
        if (rc == INVCONV_UNSUPPORTED) {
            rc = launch_mix<true>(grad_u, V, s, b, grad_x, B, C, HW, st);
            if (rc) return rc;
            rc = invconv_backward_ws(grad_x, x, w, grad_y, grad_w, B, C, H, W, k, sc.p, need, stream);
        }
        if (rc) return rc;
        const size_t sm = sizeof(float) * 2 * (size_t)C * (kMixPixels + 1);
        auto kern = flow_mix_grad_kernel;
        rc = invconv_internal::set_smem_limit(kern, sm);
        if (rc) return rc;
        kern<<<shares, 256, sm, st>>>(grad_u, x, partials, B, C, HW, tiles);
        rc = check_launch();
        if (rc) return rc;
    } else {
        rc = invconv_backward_ws(grad_u, x, w, grad_y, grad_w, 0, C, H, W, k, nullptr, 0, stream);   // zeroes grad_w
        if (rc) return rc;
        shares = 0;
    }
    const size_t smf = sizeof(double) * NE;
    auto kf = flow_mix_grad_final_kernel;
    rc = invconv_internal::set_smem_limit(kf, smf);
    if (rc) return rc;
    kf<<<1, 256, smf, st>>>(partials, shares, V, s, b, grad_V, grad_s, grad_b, C);
    return check_launch();
}

}  // extern "C"

// Weight gradient for many channels on the tcgen05 tensor cores (Theorem 2 in closed form):
//   G[dh][dw][co][ci] = sum_{n,h,w} grad_y[n,co,h,w] * x[n,ci,h-dh,w-dw]        (grad_w = -G on the mask)
// For one tap this is a matrix product with the pixels as the contraction index, contiguous in NCHW for both
// operands, so both are staged K-major without swizzle: [pixel / 4][channel][4 pixels] (see umma.cuh).
// grad_y is staged once per unit; x is staged once per column offset dw, already shifted by dw pixels with
// zeros where w - dw leaves the image (the 16-byte pixel quads of the two operands must line up, so the
// column offset cannot be a start address here); the row offset dh selects which rows of x are staged.
//
// A CTA owns one kernel row dh (its k accumulators [co x ci] live in tensor memory, k*C columns, each fed by
// one issuing warp -- at most four of them, the first also takes a fifth accumulator -- so that an accumulator
// always receives its products in the same order; twelve warps leave every scheduler three, which is what lets
// the producers keep a unit's loads in registers one unit ahead) and a share
// of the (image, row band) units; per unit the producer warps stage grad_y and the k shifted copies of x
// (rounded to tf32, single pass: grad_w's tolerance admits it, see the header of the library),
// double-buffered against the MMA issue.  Partial sums per share go to the workspace; gradw_reduce_kernel
// adds them in a fixed order.
#pragma once


#include "common.cuh"
#include "tma.cuh"
#include "umma.cuh"
#include "tensor_plan.h"

namespace invconv {

struct GradWTensorParams {
    const float* gy;       // [B][C][H][W]
    const float* x;        // [B][C][H][W]
    float* partials;       // [S][K*K][C][C]   (tap = dh*K + dw, then co, then ci)
    int B, C, H, W, K;
    int RB, Wp, nbands, S, nk;
    unsigned tmem_cols, planeA, planeB, stage_bytes;
};

__global__ void __maxnreg__(144) gradw_tensor_kernel(const GradWTensorParams p)
{
    extern __shared__ __align__(128) unsigned char gsmem[];
    const int tid = threadIdx.x, warp = tid >> 5;
    const int C = p.C, H = p.H, W = p.W, K = p.K, RB = p.RB;
    const int dh = blockIdx.x % K, share = blockIdx.x / K;
    const int nunits = p.B * p.nbands;
    const int HW = H * W;
    const int nchunk = RB * W / 4;                          // 4-pixel quads per staged channel row
    const unsigned planeC = p.planeA;                       // one quad of every channel (+ 16 bytes: staggers the banks)

    unsigned long long* bars = reinterpret_cast<unsigned long long*>(gsmem + 2 * (size_t)p.stage_bytes);
    unsigned long long* full = bars;          // [2] operands of a unit are staged
    unsigned long long* empty = bars + 2;     // [2] the MMAs that read them are done
    unsigned long long* done = bars + 4;      // all MMAs are done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
    volatile int* gave_up = reinterpret_cast<volatile int*>(bars + 6);

    const int NIW = K < kGradWTensorIssuers ? K : kGradWTensorIssuers;     // issuing warps
    if (tid == 0) {
        mbar_init(full + 0, 256); mbar_init(full + 1, 256);
        mbar_init(empty + 0, NIW); mbar_init(empty + 1, NIW);
        mbar_init(done, NIW);
        *gave_up = 0;
        fence_mbar_init();
    }
    // zero both stages once: padding pixels and the pixels in front of the x band stay zero for the whole launch
    for (unsigned e = tid; e < 2 * p.stage_bytes / 16; e += blockDim.x) reinterpret_cast<uint4*>(gsmem)[e] = make_uint4(0, 0, 0, 0);
    if (warp == 8) umma::tmem_alloc(tmem_slot, p.tmem_cols);
    fence_proxy_async();
    umma::fence_before_sync();
    __syncthreads();
    umma::fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    asm volatile("griddepcontrol.wait;" ::: "memory");        // grad_y comes from the previous launch on the stream

    auto wait_bar = [&](unsigned long long* bar, unsigned parity) {
        if (mbar_try_wait(bar, parity)) return;
        if (*gave_up) return;
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, parity)) {
            if (*gave_up) return;
            if (clock64() - t0 > (1ll << 24)) { *gave_up = 1; raise_status(INVCONV_TIMEOUT); return; }
        }
    };

    int my_units = 0;
    for (int u = share; u < nunits; u += p.S) ++my_units;

    if (warp < 8) {
        // ------------------------------------------------ stage grad_y and x of every unit
        const int QW = W / 4;
        const int items = C * RB * QW;                      // (channel, row of the band, quad of the row); at most 8 per thread
        // an item's place in the band and in the staged planes does not depend on the unit: worked out once
        int goff[8], soff[8], hl_[8];
        bool left[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = tid + j * 256;
            const int q = e % QW, hl = (e / QW) % RB, c = e / (QW * RB);     // quads of a channel's band are contiguous in memory
            goff[j] = e < items ? c * HW + hl * W + 4 * q : -1;
            soff[j] = (hl * QW + q) * (int)planeC + c * 16;
            hl_[j] = hl;
            left[j] = q > 0;
        }
        const size_t copy_bytes = (size_t)nchunk * planeC;
        const bool shuffle_left = (32 % QW) == 0;          // a row's quads never straddle a warp
        // four items of unit u: the loads ...
        auto load4 = [&](int u, int j0, float4 (&a)[4], float4 (&b1)[4]) {
            const int n = u / p.nbands, r = u - n * p.nbands;
            const float* gyb = p.gy + (size_t)n * C * HW + (size_t)r * RB * W;        // first row of the band
            const float* xb = p.x + (size_t)n * C * HW + ((size_t)r * RB - dh) * W;   // ... of the rows dh above it
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                a[j] = b1[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int h = r * RB + hl_[j0 + j];
                if (goff[j0 + j] >= 0 && h < H &&
                    INVCONV_CHECKED((size_t)n * C * HW + (size_t)r * RB * W + goff[j0 + j] + 3, (size_t)p.B * C * HW, 202)) {
                    a[j] = __ldg(reinterpret_cast<const float4*>(gyb + goff[j0 + j]));
                    if (h >= dh) b1[j] = __ldg(reinterpret_cast<const float4*>(xb + goff[j0 + j]));
                }
            }
        };
        // the quad to the left of each item's quad of x: from the neighbouring lane where a row's quads never
        // straddle a warp, else loaded (late: widths that are no power of two pay that latency)
        auto left4 = [&](int u, int j0, const float4 (&b1)[4], float4 (&b0)[4]) {
            if (shuffle_left) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float4 t;
                    t.x = __shfl_up_sync(0xffffffffu, b1[j].x, 1); t.y = __shfl_up_sync(0xffffffffu, b1[j].y, 1);
                    t.z = __shfl_up_sync(0xffffffffu, b1[j].z, 1); t.w = __shfl_up_sync(0xffffffffu, b1[j].w, 1);
                    b0[j] = left[j0 + j] ? t : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            } else {
                const int n = u / p.nbands, r = u - n * p.nbands;
                const float* xb = p.x + (size_t)n * C * HW + ((size_t)r * RB - dh) * W;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    b0[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    const int h = r * RB + hl_[j0 + j];
                    if (goff[j0 + j] >= 0 && h < H && h >= dh && left[j0 + j]) b0[j] = __ldg(reinterpret_cast<const float4*>(xb + goff[j0 + j] - 4));
                }
            }
        };
        // ... and the conversions and stores into stage `sa` (grad_y) / `sb` (the K shifted copies of x)
        auto store4 = [&](int j0, const float4 (&a)[4], const float4 (&b1)[4], const float4 (&b0)[4], unsigned char* sa, unsigned char* sb) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (goff[j0 + j] < 0) continue;
                if (!INVCONV_CHECKED(soff[j0 + j] + 15, copy_bytes, 201)) continue;
                unsigned char* da_ = sa + soff[j0 + j];
                unsigned char* db_ = sb + soff[j0 + j];
                *reinterpret_cast<float4*>(da_) = make_float4(tf32_hi(a[j].x), tf32_hi(a[j].y), tf32_hi(a[j].z), tf32_hi(a[j].w));
                const float x0 = tf32_hi(b0[j].x), x1 = tf32_hi(b0[j].y), x2 = tf32_hi(b0[j].z), x3 = tf32_hi(b0[j].w);
                const float x4 = tf32_hi(b1[j].x), x5 = tf32_hi(b1[j].y), x6 = tf32_hi(b1[j].z), x7 = tf32_hi(b1[j].w);
                // copy dw holds x[.., w - dw]: elements 4-dw .. 7-dw of the two loaded quads
                *reinterpret_cast<float4*>(db_) = make_float4(x4, x5, x6, x7);
                if (K > 1) *reinterpret_cast<float4*>(db_ + copy_bytes) = make_float4(x3, x4, x5, x6);
                if (K > 2) *reinterpret_cast<float4*>(db_ + 2 * copy_bytes) = make_float4(x2, x3, x4, x5);
                if (K > 3) *reinterpret_cast<float4*>(db_ + 3 * copy_bytes) = make_float4(x1, x2, x3, x4);
                if (K > 4) *reinterpret_cast<float4*>(db_ + 4 * copy_bytes) = make_float4(x0, x1, x2, x3);
            }
        };
        // The first four items of a unit are requested one unit ahead, so that their memory latency runs under
        // the conversions, stores and barrier waits of the unit before (a thread rarely has more than four).
        float4 na[4], nb1[4];
        if (share < nunits) load4(share, 0, na, nb1);
        int it = 0;
        for (int u = share; u < nunits; u += p.S, ++it) {
            const int st = it & 1;
            float4 a[4], b1[4], b0[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) { a[j] = na[j]; b1[j] = nb1[j]; }
            if (u + p.S < nunits) load4(u + p.S, 0, na, nb1);
            left4(u, 0, b1, b0);
            if (it >= 2) wait_bar(empty + st, ((it >> 1) - 1) & 1);
            unsigned char* sa = gsmem + (size_t)st * p.stage_bytes;
            unsigned char* sb = sa + copy_bytes;
            store4(0, a, b1, b0, sa, sb);
            if (4 * 256 < items) {
                load4(u, 4, a, b1);
                left4(u, 4, b1, b0);
                store4(4, a, b1, b0, sa, sb);
            }
            fence_proxy_async();
            mbar_arrive(full + st);
        }
        // ------------------------------------------------ accumulators -> partial sums (lane = co)
        if (warp < 4) {
            wait_bar(done, 0);
            umma::fence_after_sync();
            const int co = tid;
            const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
            for (int dw = 0; dw < K; ++dw) {
                float* dst = p.partials + ((size_t)share * K * K + (size_t)(dh * K + dw)) * C * C + (size_t)co * C;
                for (int c0 = 0; c0 < C; c0 += 16) {
                    uint32_t v[16];
                    umma::tmem_ld16(lane_addr + (uint32_t)(dw * C + c0), v);
                    umma::tmem_ld_fence(v);
                    if (co < C && INVCONV_CHECKED((dst - p.partials) + c0 + 15, (size_t)p.S * K * K * C * C, 203)) {
#pragma unroll
                        for (int j = 0; j < 16; j += 4)
                            *reinterpret_cast<float4*>(dst + c0 + j) =
                                my_units > 0 ? make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]))
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
            umma::fence_before_sync();
        }
    } else if ((tid & 31) == 0 && warp - 8 < NIW) {
        // ------------------------------------------------ MMA issue: warp 8 + i owns the accumulators of taps (dh, i), (dh, i + NIW)
        const uint32_t idesc = umma::make_idesc(umma::kFmtTF32, (uint32_t)C);
        const uint32_t kstep = 2 * (planeC >> 4), copy = (uint32_t)nchunk * (planeC >> 4);
        int it = 0;
        for (int u = share; u < nunits; u += p.S, ++it) {
            const int st = it & 1;
            wait_bar(full + st, (it >> 1) & 1);
            umma::fence_after_sync();
            const uint32_t sa = smem_u32(gsmem + (size_t)st * p.stage_bytes);
            for (int dw = warp - 8; dw < K; dw += NIW) {
                const uint32_t dcol = tmem + (uint32_t)(dw * C);
                uint64_t da = umma::make_desc(sa, planeC);
                uint64_t db = umma::make_desc(sa + (uint32_t)nchunk * planeC, planeC) + (uint64_t)(dw * copy);
                for (int ks = 0; ks < p.nk; ++ks) {
                    umma::mma_tf32(dcol, da, db, idesc, (it > 0 || ks > 0) ? 1u : 0u);
                    da += kstep; db += kstep;
                }
            }
            umma::commit(empty + st);
        }
        umma::commit(done);
    }
    umma::fence_before_sync();
    __syncthreads();
    if (warp == 8) {
        umma::fence_after_sync();
        umma::tmem_dealloc(tmem, p.tmem_cols);
    }
}

}  // namespace invconv

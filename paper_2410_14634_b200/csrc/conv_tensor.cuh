// The masked convolution y = f(x) (Eq. 1; the sampling direction, Section 4.3) for many channels on the tcgen05
// tensor cores: an implicit GEMM  y[pixel][co] = sum_{tap, ci} x[pixel - tap][ci] * w_masked[tap][ci][co].
//
// Accumulator lanes are the pixel slots of a band of RB rows of one image, rows padded on the left by k-1 zero
// slots (lane m = row * (W+k-1) + column).  The band, its k-1 rows above and the padding are staged once as
// shared-memory operand rows [channel/4][slot][4 channels] (K-major, no swizzle: rows form a linear array), so
// the x operand of tap (dh, dw) is the same buffer started (k-1-dh) rows and -dw slots later -- a start address.
// The weights of one tap, [chunk of 8 ci][co], stream from the packed copy made by conv_pack_kernel through a ring
// of up to eight stages (bulk TMA copies, no multicast; as many as shared memory holds, since the bytes in flight
// from L2 set the streaming rate).  Products carry the same split as the wavefront solve:
// hi(w) hi(x) as one tf32 MMA plus lo(w) bf(x) + bf(w) lo(x) as one bf16 MMA; that holds the 1e-5 parity bar
// of f, which single-pass tf32 does not.  Two warps issue MMAs, even and odd taps, each into its own
// accumulator, so every accumulator receives its products in program order; the epilogue adds the two.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"
#include "tma.cuh"
#include "umma.cuh"
#include "tensor_plan.h"

namespace invconv {

// Packs the masked kernel for the tensor-core convolution: per tap (dh, dw), chunk of 8 input channels and output
// channel co one 16-byte row per plane: planes 0, 1 hold hi(w) for ci = 4p .. 4p+3, plane 2 the bf16 remainders,
// plane 3 the bf16 values.  Layout [tap][chunk][plane][co][16 B].  One thread per (tap, chunk, co).
__global__ void __launch_bounds__(256) conv_pack_kernel(const float* __restrict__ w, unsigned char* __restrict__ pack, int C, int K)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int nchunk = C / 8, total = K * K * nchunk * C;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const int co = e % C, chunk = (e / C) % nchunk, tap = e / (C * nchunk);
        const int dh = tap / K, dw = tap - dh * K;
        float v[8], hi[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int ci = chunk * 8 + j;
            const bool masked_out = tap == 0 && ci > co;
            v[j] = masked_out ? 0.f : __ldg(w + w_index(co, ci, K - 1 - dh, K - 1 - dw, C, K));
            hi[j] = tf32_hi(v[j]);
        }
        unsigned char* blk = pack + ((size_t)tap * nchunk + chunk) * 4 * C * 16;
        *reinterpret_cast<float4*>(blk + ((size_t)0 * C + co) * 16) = make_float4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<float4*>(blk + ((size_t)1 * C + co) * 16) = make_float4(hi[4], hi[5], hi[6], hi[7]);
        uint4 lo, bf;
        const __nv_bfloat162 l0 = __floats2bfloat162_rn(v[0] - hi[0], v[1] - hi[1]), l1 = __floats2bfloat162_rn(v[2] - hi[2], v[3] - hi[3]);
        const __nv_bfloat162 l2 = __floats2bfloat162_rn(v[4] - hi[4], v[5] - hi[5]), l3 = __floats2bfloat162_rn(v[6] - hi[6], v[7] - hi[7]);
        const __nv_bfloat162 b0 = __floats2bfloat162_rn(v[0], v[1]), b1 = __floats2bfloat162_rn(v[2], v[3]);
        const __nv_bfloat162 b2 = __floats2bfloat162_rn(v[4], v[5]), b3 = __floats2bfloat162_rn(v[6], v[7]);
        lo.x = *reinterpret_cast<const uint32_t*>(&l0); lo.y = *reinterpret_cast<const uint32_t*>(&l1);
        lo.z = *reinterpret_cast<const uint32_t*>(&l2); lo.w = *reinterpret_cast<const uint32_t*>(&l3);
        bf.x = *reinterpret_cast<const uint32_t*>(&b0); bf.y = *reinterpret_cast<const uint32_t*>(&b1);
        bf.z = *reinterpret_cast<const uint32_t*>(&b2); bf.w = *reinterpret_cast<const uint32_t*>(&b3);
        *reinterpret_cast<uint4*>(blk + ((size_t)2 * C + co) * 16) = lo;
        *reinterpret_cast<uint4*>(blk + ((size_t)3 * C + co) * 16) = bf;
    }
}

struct ConvTensorParams {
    const float* x;              // [B][C][H][W]
    const unsigned char* pack;   // packed masked kernel, see conv_pack_kernel
    float* y;
    int B, C, H, W, K;
    int RB, Wp, nbands, ntiles, slots, spi;
    unsigned tmem_cols, x_bytes, wstage_bytes, off_w, off_bar;
};

__global__ void __launch_bounds__(kConvTensorThreads, 1) conv_tensor_kernel(const ConvTensorParams p)
{
    extern __shared__ __align__(128) unsigned char csmem[];
    const int tid = threadIdx.x, warp = tid >> 5;
    const int C = p.C, H = p.H, W = p.W, K = p.K, RB = p.RB, Wp = p.Wp, SL = p.slots;
    const int HW = H * W, KK = K * K, nchunk = C / 8, FRONT = K - 1;
    unsigned char* s_x = csmem;                                   // [chunk][plane 0..3][SL][16]
    unsigned char* s_w = csmem + p.off_w;                         // [stage][chunk][plane 0..3][C][16]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(csmem + p.off_bar);
    unsigned long long* xfull = bars + 0;        // the x tile is staged (256 arrivals)
    unsigned long long* wfull = bars + 1;        // [2 * spi] a tap's weights have arrived
    unsigned long long* wempty = bars + 9;       // [2 * spi] the MMAs that read them are done
    unsigned long long* accdone = bars + 17;     // both issuers' MMAs of the tile are done
    unsigned long long* tmemfree = bars + 18;    // the accumulators have been read (128 arrivals)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 19);
    volatile int* gave_up = reinterpret_cast<volatile int*>(bars + 20);
    const int SPI = p.spi;

    if (tid == 0) {
        mbar_init(xfull, 256);
        for (int s = 0; s < 2 * kConvTensorMaxSpi; ++s) { mbar_init(wfull + s, 1); mbar_init(wempty + s, 1); }
        mbar_init(accdone, 2);
        mbar_init(tmemfree, 128);
        *gave_up = 0;
        fence_mbar_init();
    }
    for (unsigned e = tid; e < p.x_bytes / 16; e += kConvTensorThreads) reinterpret_cast<uint4*>(s_x)[e] = make_uint4(0, 0, 0, 0);
    if (warp == 8) umma::tmem_alloc(tmem_slot, p.tmem_cols);
    fence_proxy_async();
    umma::fence_before_sync();
    __syncthreads();
    umma::fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    auto wait_bar = [&](unsigned long long* bar, unsigned parity) { mbar_wait_or_give_up(bar, parity, gave_up); };
    const unsigned chunk_bytes = 4u * SL * 16;

    if (warp < 8) {
        // ------------------------------------------------ stage the band of x (+ k-1 rows above) as operand rows
        const int rows = RB + K - 1;
        const int items = nchunk * rows * W;
        unsigned it = 0;
        for (int tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x, ++it) {
            const int n = tile / p.nbands, h0 = (tile - n * p.nbands) * RB;
            if (it > 0) wait_bar(accdone, (it - 1) & 1);         // the previous tile's MMAs have read the buffer
            const float* xn = p.x + (size_t)n * C * HW;
            for (int e = tid; e < items; e += 256) {
                const int w = e % W, hr = (e / W) % rows, chunk = e / (W * rows);
                const int h = h0 - (K - 1) + hr;
                float v[8];
                if (h >= 0 && h < H && INVCONV_CHECKED((size_t)n * C * HW + (size_t)(chunk * 8 + 7) * HW + h * W + w, (size_t)p.B * C * HW, 302)) {
                    const float* src = xn + (size_t)(chunk * 8) * HW + h * W + w;
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = __ldg(src + (size_t)j * HW);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = 0.f;
                }
                float hi[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) hi[j] = tf32_hi(v[j]);
                unsigned char* cb = s_x + (size_t)chunk * chunk_bytes;
                const int slot = FRONT + hr * Wp + w + K - 1;
                if (!INVCONV_CHECKED(slot, SL, 301)) continue;
                *reinterpret_cast<float4*>(cb + ((size_t)0 * SL + slot) * 16) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<float4*>(cb + ((size_t)1 * SL + slot) * 16) = make_float4(hi[4], hi[5], hi[6], hi[7]);
                const __nv_bfloat162 b0 = __floats2bfloat162_rn(v[0], v[1]), b1 = __floats2bfloat162_rn(v[2], v[3]);
                const __nv_bfloat162 b2 = __floats2bfloat162_rn(v[4], v[5]), b3 = __floats2bfloat162_rn(v[6], v[7]);
                const __nv_bfloat162 l0 = __floats2bfloat162_rn(v[0] - hi[0], v[1] - hi[1]), l1 = __floats2bfloat162_rn(v[2] - hi[2], v[3] - hi[3]);
                const __nv_bfloat162 l2 = __floats2bfloat162_rn(v[4] - hi[4], v[5] - hi[5]), l3 = __floats2bfloat162_rn(v[6] - hi[6], v[7] - hi[7]);
                uint4 bf, lo;
                bf.x = *reinterpret_cast<const uint32_t*>(&b0); bf.y = *reinterpret_cast<const uint32_t*>(&b1);
                bf.z = *reinterpret_cast<const uint32_t*>(&b2); bf.w = *reinterpret_cast<const uint32_t*>(&b3);
                lo.x = *reinterpret_cast<const uint32_t*>(&l0); lo.y = *reinterpret_cast<const uint32_t*>(&l1);
                lo.z = *reinterpret_cast<const uint32_t*>(&l2); lo.w = *reinterpret_cast<const uint32_t*>(&l3);
                *reinterpret_cast<uint4*>(cb + ((size_t)2 * SL + slot) * 16) = bf;      // pairs with lo(w)
                *reinterpret_cast<uint4*>(cb + ((size_t)3 * SL + slot) * 16) = lo;      // pairs with bf(w)
            }
            fence_proxy_async();
            mbar_arrive(xfull);
            // ------------------------------------------------ accumulators -> y (lane = padded pixel slot)
            if (warp < 4) {
                wait_bar(accdone, it & 1);
                umma::fence_after_sync();
                const int m = tid, hl = m / Wp, c = m - hl * Wp;
                const int h = h0 + hl, wq = c - (K - 1);
                const bool valid = m < RB * Wp && wq >= 0 && h < H;
                const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
                float* dst = p.y + (size_t)n * C * HW + (size_t)(valid ? h * W + wq : 0);
                for (int c0 = 0; c0 < C; c0 += 16) {
                    uint32_t a0[16], a1[16];
                    umma::tmem_ld16(lane_addr + (uint32_t)c0, a0);
                    umma::tmem_ld16(lane_addr + (uint32_t)(C + c0), a1);
                    umma::tmem_ld_fence(a0);
                    umma::tmem_ld_fence(a1);
                    if (valid && INVCONV_CHECKED((dst - p.y) + (size_t)(c0 + 15) * HW, (size_t)p.B * C * HW, 303)) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) dst[(size_t)(c0 + j) * HW] = __uint_as_float(a0[j]) + __uint_as_float(a1[j]);
                    }
                }
                umma::fence_before_sync();
                mbar_arrive(tmemfree);
            }
        }
    } else if (warp < 10) {
        // ------------------------------------------------ MMA issue: warp 8 the even taps, warp 9 the odd ones
        if ((tid & 31) == 0) {
            const int q = warp - 8;
            const uint32_t dcol = tmem + (uint32_t)(q * C);
            const uint32_t idesc_tf = umma::make_idesc(umma::kFmtTF32, (uint32_t)C), idesc_bf = umma::make_idesc(umma::kFmtBF16, (uint32_t)C);
            const uint32_t xa = smem_u32(s_x), wa = smem_u32(s_w);
            unsigned it = 0, nuse[kConvTensorMaxSpi] = {0, 0, 0, 0};     // uses so far of this issuer's stages
            for (int tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x, ++it) {
                wait_bar(xfull, it & 1);
                if (it > 0) wait_bar(tmemfree, (it - 1) & 1);
                umma::fence_after_sync();
                bool first = true;
                int sl = 0;
                for (int tap = q; tap < KK; tap += 2, sl = sl + 1 == SPI ? 0 : sl + 1) {
                    const int stage = q + 2 * sl;
                    wait_bar(wfull + stage, nuse[sl] & 1);
                    umma::fence_after_sync();
                    const int dh = tap / K, dw = tap - dh * K;
                    const uint32_t row0 = (uint32_t)(FRONT + (K - 1 - dh) * Wp - dw) * 16;
                    (void)INVCONV_CHECKED(FRONT + (K - 1 - dh) * Wp - dw + 127, SL, 304);
                    for (int ch = 0; ch < nchunk; ++ch) {
                        const uint32_t xb = xa + (uint32_t)ch * chunk_bytes + row0;
                        const uint32_t wb = wa + (uint32_t)stage * p.wstage_bytes + (uint32_t)ch * 4 * C * 16;
                        umma::mma_tf32(dcol, umma::make_desc(xb, (uint32_t)SL * 16), umma::make_desc(wb, (uint32_t)C * 16), idesc_tf, first ? 0u : 1u);
                        umma::mma_bf16(dcol, umma::make_desc(xb + 2u * SL * 16, (uint32_t)SL * 16),
                                       umma::make_desc(wb + 2u * C * 16, (uint32_t)C * 16), idesc_bf, 1u);
                        first = false;
                    }
                    umma::commit(wempty + stage);
                    ++nuse[sl];
                }
                umma::commit(accdone);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ weights: one bulk copy per tap into its issuer's next stage
        if (tid == 320) {
            asm volatile("griddepcontrol.wait;" ::: "memory");      // the packed kernel comes from the previous launch
            unsigned nuse[2 * kConvTensorMaxSpi] = {0, 0, 0, 0, 0, 0, 0, 0};
            for (int tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
                int jq[2] = {0, 0};
                for (int tap = 0; tap < KK; ++tap) {
                    const int q = tap & 1, sl = jq[q], stage = q + 2 * sl;
                    jq[q] = sl + 1 == SPI ? 0 : sl + 1;
                    if (nuse[stage] > 0) wait_bar(wempty + stage, (nuse[stage] - 1) & 1);
                    mbar_expect_tx(wfull + stage, p.wstage_bytes);
                    bulk_g2s(s_w + (size_t)stage * p.wstage_bytes, p.pack + (size_t)tap * p.wstage_bytes, p.wstage_bytes, wfull + stage);
                    ++nuse[stage];
                }
            }
        }
        __syncwarp();
    }
    umma::fence_before_sync();
    __syncthreads();
    if (tid == 0 && *gave_up) raise_status(INVCONV_TIMEOUT);
    if (warp == 8) {
        umma::fence_after_sync();
        umma::tmem_dealloc(tmem, p.tmem_cols);
    }
}

}  // namespace invconv

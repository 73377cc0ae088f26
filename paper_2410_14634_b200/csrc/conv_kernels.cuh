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
//
// Few large images would leave most SMs idle that way, so an image can also be cut into bands of rows, one CTA
// per band: the band and the K-1 rows above it arrive by one bulk copy per channel (rows of a channel are
// contiguous), everything else is the same walk.
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
    int bands = 1; // > 1: CTAs per image, each a band of `bh` rows (ipc = 1, bulk copies, W a multiple of 4)
    int bh = 0;
};

template <int C, int K>
__global__ void __launch_bounds__(256) masked_conv_warp_kernel(ConvParams p)
{
    extern __shared__ __align__(128) float smem[];
    constexpr int NW = C * C * K * K;
    constexpr bool WREG = NW <= 108;                        // the whole masked kernel fits a lane's registers
    // otherwise a warp computes one output channel only (its C*K*K weights in registers) and C warps share a band
    constexpr int CO = WREG ? C : 1;                        // output channels per warp
    constexpr int NWR = CO * C * K * K;
    const int H = p.H, W = p.W, HW = H * W, CHW = C * HW;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool banded = p.bands > 1;
    constexpr int WSPLIT = C / CO;                          // warps per band
    const int bwarp = warp / WSPLIT, co0 = (warp - bwarp * WSPLIT) * CO;
    const int li = banded ? 0 : bwarp / p.wpi, wb = banded ? bwarp : bwarp - li * p.wpi;
    const int n = banded ? blockIdx.x / p.bands : blockIdx.x * p.ipc + li;
    const bool has_img = n < p.B;
    // rows this CTA writes [rb0, rb1) and the first row it holds in shared memory
    const int rb0 = banded ? (blockIdx.x % p.bands) * p.bh : 0, rb1 = banded ? min(H, rb0 + p.bh) : H;
    const int rl0 = max(0, rb0 - (K - 1));
    const int RW = (rb1 - rl0) * W;                                     // floats per channel held in shared memory
    const int imgf = banded ? 0 : (CHW + 31) & ~31;
    const int band = (rb1 - rb0 + p.wpi - 1) / p.wpi;
    const int hb0 = rb0 + wb * band, hb1 = min(rb1, hb0 + band);
    float* ws = smem;                                                   // masked kernel [co][ci][dh][dw]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + ((NW + 31) & ~31));
    float* xs = smem + ((NW + 31) & ~31) + 32 + li * imgf - rl0 * W;    // xs[ci * RW + row * W + col], row >= rl0

    // nothing above touched global memory; x may come from the kernel before this one on the stream.  The next
    // kernel may be scheduled right away: it waits for this one to complete at its own griddepcontrol.wait.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (has_img && p.bulk && wb == 0 && co0 == 0 && lane == 0) {
        mbar_init(&bars[li], 1);
        fence_mbar_init();
        mbar_expect_tx(&bars[li], (unsigned)(C * RW) * 4u);
        if (banded) {
#pragma unroll
            for (int c = 0; c < C; ++c)
                bulk_g2s(xs + c * RW + rl0 * W, p.x + (size_t)n * CHW + (size_t)c * HW + (size_t)rl0 * W, (unsigned)RW * 4u, &bars[li]);
        } else {
            bulk_g2s(xs, p.x + (size_t)n * CHW, (unsigned)CHW * 4u, &bars[li]);
        }
    }
    if (has_img && !p.bulk) {
        const float* src = p.x + (size_t)n * CHW;
        for (int i = (wb * WSPLIT + co0 / CO) * 32 + lane; i < CHW; i += p.wpi * WSPLIT * 32) xs[i] = __ldg(src + i);
    }
    for (int e = threadIdx.x; e < NW; e += blockDim.x) {
        const int dw = e % K, dh = (e / K) % K, ci = (e / (K * K)) % C, co = e / (K * K * C);
        const bool masked_out = (dh == 0 && dw == 0 && ci > co);
        ws[e] = masked_out ? 0.f : __ldg(p.w + ((co * C + ci) * K + (K - 1 - dh)) * K + (K - 1 - dw));
    }
    __syncthreads();
    if (!has_img) return;
    float wr[NWR];
#pragma unroll
    for (int e = 0; e < NWR; ++e) wr[e] = ws[co0 * C * K * K + e];
    if (p.bulk) {
        const bool ok = mbar_wait_bounded(&bars[li], 0);
        if (!__all_sync(0xffffffffu, ok)) { if (lane == 0) raise_status(INVCONV_TIMEOUT); return; }
    }
    if (hb0 >= hb1) return;                                // a short last band leaves its trailing warps without rows
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
                    const float t = xs[ci * RW + (in ? row * W + w - dw : rl0 * W)];
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
                            const float t = xs[ci * RW + h * W + (in ? w - dw : 0)];      // clamped: no branch
                            xr[r][ci][dw] = in ? t : 0.f;
                        }
                    float acc[CO];
#pragma unroll
                    for (int co = 0; co < CO; ++co) acc[co] = 0.f;
#pragma unroll
                    for (int co = 0; co < CO; ++co)
#pragma unroll
                        for (int ci = 0; ci < C; ++ci)
#pragma unroll
                            for (int dh = 0; dh < K; ++dh)
#pragma unroll
                                for (int dw = 0; dw < K; ++dw)
                                    acc[co] = fmaf(wr[((co * C + ci) * K + dh) * K + dw], xr[(r - dh + K) % K][ci][dw], acc[co]);
                    if (col_ok) {
#pragma unroll
                        for (int co = 0; co < CO; ++co) dst[(co0 + co) * HW + h * W + w] = acc[co];
                    }
                }
            }
        }
    }
}

template <int C, int K>
inline size_t masked_conv_smem(int H, int W, int ipc)      // H: rows held per image (a band plus the K-1 rows above it)
{
    const size_t imgf = ((size_t)C * H * W + 31) & ~(size_t)31;
    return sizeof(float) * ((((size_t)C * C * K * K + 31) & ~(size_t)31) + 32 + imgf * ipc);
}

// ---------------------------------------------------------------------------
// y = f(x) for many channels: a dense contraction over (ci, dh, dw) with
// C*K*K multiply-adds per output element, bound by the fp32 FMA pipe.
//
// A CTA owns 16 output channels and up to 64 quads of four horizontally
// adjacent pixels (a band of rows of one image, or several small images).  A
// thread owns one quad and four output channels: 16 sums in registers.  The
// input channels arrive eight at a time, double-buffered with asynchronous
// copies: the x rows of the band (plus the K-1 rows above it; every staged row
// carries four zero columns on its left so that the K-1 pixels to the left of
// a quad come with the aligned quad before it) and the CTA's slice of the
// kernel, re-ordered to [ci][dh][co group][dw][co] with the channel mask of
// the bottom-right tap applied.  Per (ci, dh) a thread issues two 16-byte
// loads of x and K 16-byte broadcast loads of the kernel for 16*K FMAs.
// ---------------------------------------------------------------------------
struct ConvTileParams {
    const float* x;
    const float* w;
    float* y;
    int B, C, H, W;
    int RB, nbands;        // rows per band, bands per image
    int Q, IPC;            // quads per band, bands (items) per CTA
    int PW, PH;            // floats per staged row (4 + W rounded up to 4), staged rows per band (RB + K - 1)
    int cotiles;           // tiles of 16 output channels
    int vec;               // x and y are 16-byte aligned and W % 4 == 0
    FastDiv div_q, div_qpr, div_bands, div_ph;
};

constexpr int kConvCoT = 16, kConvCiT = 8;

template <int K>
__global__ void __launch_bounds__(256) masked_conv_tile_kernel(ConvTileParams p)
{
    constexpr int CO_T = kConvCoT, CI_T = kConvCiT, KK = K * K;
    constexpr int WBUF = CI_T * K * 4 * K * 4;          // floats of one kernel buffer: [ci][dh][cg][dw][4]
    extern __shared__ __align__(128) float smem[];
    const int C = p.C, H = p.H, W = p.W, PW = p.PW, PH = p.PH, RB = p.RB;
    const int plane = PH * PW;                           // one staged channel of one band
    const int XBUF = p.IPC * CI_T * plane;
    float* xsm = smem;                                   // [2][IPC][CI_T][PH][PW]
    float* wsm = smem + 2 * XBUF;                        // [2][WBUF]
    const int tid = threadIdx.x, NT = blockDim.x, SL = NT >> 2;
    const int cg = tid / SL, slot = tid - cg * SL;       // warps are uniform in cg (SL is a multiple of 32)
    const int cot = blockIdx.x % p.cotiles, group = blockIdx.x / p.cotiles;
    const int co0 = cot * CO_T;
    const int nitems = p.B * p.nbands;
    const int qpr = (PW - 4) >> 2;

    // this thread's quad
    const int li = fast_div(slot, p.div_q), q = slot - li * p.Q;
    const int r = fast_div(q, p.div_qpr), w0 = (q - r * qpr) * 4;
    const int item = group * p.IPC + li;
    const bool has_quad = li < p.IPC && item < nitems;
    const int n_img = fast_div(item, p.div_bands), band = item - n_img * p.nbands;
    const int h = band * RB + r;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    // the four zero columns on the left of every staged row (never overwritten)
    for (int i = tid; i < 2 * p.IPC * CI_T * PH; i += NT) *reinterpret_cast<float4*>(xsm + i * PW) = make_float4(0.f, 0.f, 0.f, 0.f);

    auto stage = [&](int chunk, int buf) {
        const int ci0 = chunk * CI_T;
        // kernel slice: source order (co, ci, a, b) so that consecutive threads read consecutive floats
        float* wb = wsm + buf * WBUF;
        for (int e = tid; e < CO_T * CI_T * KK; e += NT) {
            const int col = e / (CI_T * KK), rem = e - col * (CI_T * KK);
            const int cil = rem / KK, ab = rem - cil * KK, a = ab / K, b = ab - a * K;
            const int co = co0 + col, ci = ci0 + cil, dh = K - 1 - a, dw = K - 1 - b;
            const bool valid = co < C && ci < C && !(ab == KK - 1 && ci > co);
            const float* src = p.w + (valid ? ((size_t)(co * C + ci) * KK + ab) : 0);
            cp_async_f32(wb + (((cil * K + dh) * 4 + (col >> 2)) * K + dw) * 4 + (col & 3), src, valid);
        }
        // x rows of the band and the K-1 rows above it
        float* xb = xsm + buf * XBUF;
        if (p.vec) {
            const int per_item = CI_T * PH * qpr;
            for (int e = tid; e < p.IPC * per_item; e += NT) {
                const int l = e / per_item, rem = e - l * per_item;       // IPC and CI_T*PH*qpr are small: plain division
                const int row = fast_div(rem, p.div_qpr), qx = rem - row * qpr;
                const int cil = fast_div(row, p.div_ph), rr = row - cil * PH;
                const int it = group * p.IPC + l;
                const int n = fast_div(it, p.div_bands), bd = it - n * p.nbands;
                const int hh = bd * RB - (K - 1) + rr, ci = ci0 + cil;
                const bool valid = it < nitems && ci < C && hh >= 0 && hh < H;
                const float* src = p.x + (valid ? (((size_t)n * C + ci) * H + hh) * W + 4 * qx : 0);
                cp_async_f32x4(xb + (l * CI_T + cil) * plane + rr * PW + 4 + 4 * qx, src, valid);
            }
        } else {
            const int per_item = CI_T * PH * (PW - 4);
            for (int e = tid; e < p.IPC * per_item; e += NT) {
                const int l = e / per_item, rem = e - l * per_item;
                const int row = rem / (PW - 4), cx = rem - row * (PW - 4);
                const int cil = fast_div(row, p.div_ph), rr = row - cil * PH;
                const int it = group * p.IPC + l;
                const int n = fast_div(it, p.div_bands), bd = it - n * p.nbands;
                const int hh = bd * RB - (K - 1) + rr, ci = ci0 + cil;
                const bool valid = it < nitems && ci < C && hh >= 0 && hh < H && cx < W;
                const float* src = p.x + (valid ? (((size_t)n * C + ci) * H + hh) * W + cx : 0);
                cp_async_f32(xb + (l * CI_T + cil) * plane + rr * PW + 4 + cx, src, valid);
            }
        }
        cp_async_commit();
    };

    const int nchunks = (C + CI_T - 1) / CI_T;
    stage(0, 0);
    for (int chunk = 0; chunk < nchunks; ++chunk) {
        const int buf = chunk & 1;
        if (chunk + 1 < nchunks) { stage(chunk + 1, buf ^ 1); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncthreads();
        if (has_quad) {
            const float* xq = xsm + buf * XBUF + li * CI_T * plane + r * PW + w0;     // row r of the band is staged row r + K-1
            const float* wq = wsm + buf * WBUF + cg * K * 4;
#pragma unroll 2
            for (int cil = 0; cil < CI_T; ++cil) {
#pragma unroll
                for (int dh = 0; dh < K; ++dh) {
                    const float* xr = xq + cil * plane + (K - 1 - dh) * PW;
                    const float4 a = *reinterpret_cast<const float4*>(xr);
                    const float4 b = *reinterpret_cast<const float4*>(xr + 4);
                    const float vv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
                    for (int dw = 0; dw < K; ++dw) {
                        const float4 wv = *reinterpret_cast<const float4*>(wq + ((cil * K + dh) * 4 * K + dw) * 4);
#pragma unroll
                        for (int px = 0; px < 4; ++px) {
                            const float v = vv[4 + px - dw];
                            acc[px][0] = fmaf(v, wv.x, acc[px][0]);
                            acc[px][1] = fmaf(v, wv.y, acc[px][1]);
                            acc[px][2] = fmaf(v, wv.z, acc[px][2]);
                            acc[px][3] = fmaf(v, wv.w, acc[px][3]);
                        }
                    }
                }
            }
        }
        __syncthreads();       // the buffer is free for the copies of chunk + 2
    }

    if (has_quad && h < H) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int co = co0 + cg * 4 + j;
            if (co < C) {
                float* dst = p.y + (((size_t)n_img * C + co) * H + h) * W + w0;
                if (p.vec) *reinterpret_cast<float4*>(dst) = make_float4(acc[0][j], acc[1][j], acc[2][j], acc[3][j]);
                else {
#pragma unroll
                    for (int px = 0; px < 4; ++px)
                        if (w0 + px < W) dst[px] = acc[px][j];
                }
            }
        }
    }
}

struct ConvTilePlan {
    bool ok = false;
    int RB = 0, nbands = 0, Q = 0, IPC = 1, PW = 0, PH = 0, cotiles = 0, threads = 0, grid = 0;
    size_t smem = 0;
};

inline ConvTilePlan plan_conv_tile(int B, int C, int H, int W, int K, size_t max_smem, int sm_count)
{
    ConvTilePlan pl;
    if (B < 1 || K > 5 || C < 5) return pl;
    const int qpr = (W + 3) / 4;
    if (qpr > 64) return pl;
    pl.PW = 4 + 4 * qpr;
    pl.RB = 64 / qpr;
    if (pl.RB > H) pl.RB = H;
    pl.nbands = (H + pl.RB - 1) / pl.RB;
    pl.RB = (H + pl.nbands - 1) / pl.nbands;            // even bands
    pl.Q = pl.RB * qpr;
    pl.PH = pl.RB + K - 1;
    pl.cotiles = (C + kConvCoT - 1) / kConvCoT;
    const int items = B * pl.nbands;
    int ipc = 64 / pl.Q;
    if (ipc < 1) ipc = 1;
    const int ipc_min = pl.Q >= 32 ? 1 : (32 + pl.Q - 1) / pl.Q;       // fill at least one warp per output-channel group
    while (ipc > ipc_min && ((items + ipc - 1) / ipc) * pl.cotiles < 2 * sm_count) --ipc;   // enough CTAs first
    pl.IPC = ipc;
    const int slots = (ipc * pl.Q + 31) & ~31;
    pl.threads = 4 * slots;
    pl.smem = sizeof(float) * 2 * ((size_t)ipc * kConvCiT * pl.PH * pl.PW + (size_t)kConvCiT * K * 4 * K * 4);
    if (pl.threads > 256 || pl.smem > max_smem) return pl;
    pl.grid = ((items + ipc - 1) / ipc) * pl.cotiles;
    pl.ok = true;
    return pl;
}

}  // namespace invconv

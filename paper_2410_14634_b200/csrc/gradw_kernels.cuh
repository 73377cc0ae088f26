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

// ---------------------------------------------------------------------------
// The same tiling on the tensor pipe (TF32 inputs, fp32 accumulation): for a
// fixed tap the sum over pixels is a matrix product  G[co][ci] = sum_p
// grad_y[co][p] * x[ci][p - shift], M = co, N = ci, contraction over the
// pixels, which are the contiguous index of both operands in NCHW.  A warp
// owns one 16-row block of output channels and one kernel column dw and walks
// the rows h >= dh of the staged planes in chunks of eight pixels:
// mma.m16n8k8 with A = grad_y[16 co][8 pixels], B = x[8 pixels - shift][8 ci]
// for each of the tile's 8-channel groups.  Fragments are read straight from
// the padded channel planes (plane stride = 4 mod 32: the 8 x 4 elements of a
// fragment register fall in 32 different banks); the K-1 pixels to the left of
// column 0 and the rows above row 0 are zeros by predicate.  Inputs are
// rounded to TF32 (10-bit mantissa): the weight gradient's parity bar is 1e-3
// of its largest entry, which a single TF32 pass holds (the solves, at 1e-4,
// stay in fp32).  Needs W % 8 == 0; other shapes use the FMA kernel above.
// ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned to_tf32(float v)
{
    unsigned r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r;
}

__device__ __forceinline__ void mma_tf32_16x8x8(float (&d)[4], const unsigned (&a)[4], const unsigned (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// ALLDH (tiles of 16 channels): one CTA covers all K*K taps, warp = (dh, dw), so that a 12- or 16-channel
// layer still gives every CTA K*K warps and every image is staged once instead of once per kernel row.
template <int TC, int K, bool ALLDH = false>
__global__ void __launch_bounds__(32 * (ALLDH ? K * K : TC * K)) gradw_mma_kernel(GradWParams p)
{
    static_assert(!ALLDH || TC == 1, "all kernel rows in one CTA: tiles of 16 channels only");
    extern __shared__ __align__(128) float smem[];
    constexpr int TB = 16 * TC;                 // channels per tile side
    constexpr int NT8 = 2 * TC;                 // 8-channel groups of the ci tile
    const int H = p.H, W = p.W, HW = H * W, C = p.C;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
    const int g = lane >> 2, t = lane & 3;      // fragment coordinates
    const int mt = ALLDH ? 0 : warp / K;        // this warp's 16 output channels
    const int dw = ALLDH ? warp % K : warp - mt * K;   // ... and kernel column
    int bid = blockIdx.x;
    const int share = bid % p.nbc; bid /= p.nbc;
    const int tci = bid % p.tiles; bid /= p.tiles;
    const int tco = bid % p.tiles; bid /= p.tiles;
    const int dh = ALLDH ? warp / K : bid;
    const int co0 = tco * TB, ci0 = tci * TB;
    const int nco = min(TB, C - co0), nci = min(TB, C - ci0);
    float* gys = smem;                          // [TB][plane]
    float* xs = smem + TB * p.plane;            // [TB][plane]

    float acc[NT8][4];
#pragma unroll
    for (int i = 0; i < NT8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    // channels beyond C (padding of the last tile) stay zero; the others are overwritten by every image
    for (int c = nco + warp; c < TB; c += nwarps)
        for (int i = lane; i < p.plane; i += 32) gys[c * p.plane + i] = 0.f;
    for (int c = nci + warp; c < TB; c += nwarps)
        for (int i = lane; i < p.plane; i += 32) xs[c * p.plane + i] = 0.f;

    for (int n = share; n < p.B; n += p.nbc) {
        // stage the tile's channel planes with 16-byte asynchronous copies issued by all threads (a bulk copy
        // per channel plane would serialise in the copy engine at ~150 cycles each, more than the whole product)
        const float* gsrc = p.gy + ((size_t)n * C + co0) * HW;
        const float* xsrc = p.x + ((size_t)n * C + ci0) * HW;
        const int nq = HW >> 2;
        for (int c = warp; c < nco + nci; c += nwarps) {
            const bool isg = c < nco;
            const int cc = isg ? c : c - nco;
            const float* src = (isg ? gsrc : xsrc) + (size_t)cc * HW;
            float* dstp = (isg ? gys : xs) + cc * p.plane;
            for (int q = lane; q < nq; q += 32) cp_async_f32x4(dstp + 4 * q, src + 4 * q, true);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();

        const float* ga = gys + (mt * 16 + g) * p.plane + t;          // A: rows g and g + 8, pixel columns t and t + 4
        const float* xb = xs + g * p.plane + t - dw;                  // B: channel g of a group, pixels t and t + 4, shifted
        for (int h = dh; h < H; ++h) {
            for (int w0 = 0; w0 < W; w0 += 8) {
                const int pa = h * W + w0, pb = (h - dh) * W + w0;
                unsigned a[4];
                a[0] = to_tf32(ga[pa]);
                a[1] = to_tf32(ga[pa + 8 * p.plane]);
                a[2] = to_tf32(ga[pa + 4]);
                a[3] = to_tf32(ga[pa + 8 * p.plane + 4]);
                const bool v0 = w0 + t >= dw, v1 = w0 + t + 4 >= dw;   // pixels left of column 0 are padding
#pragma unroll
                for (int nt = 0; nt < NT8; ++nt) {
                    unsigned b[2];
                    b[0] = v0 ? to_tf32(xb[nt * 8 * p.plane + pb]) : 0u;
                    b[1] = v1 ? to_tf32(xb[nt * 8 * p.plane + pb + 4]) : 0u;
                    mma_tf32_16x8x8(acc[nt], a, b);
                }
            }
        }
        __syncthreads();       // everyone is done with this image before its planes are overwritten
    }

    float* dst = p.partials + (size_t)share * K * K * C * C + (size_t)(dh * K + dw) * C * C;
#pragma unroll
    for (int nt = 0; nt < NT8; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int co = co0 + mt * 16 + g + (j >> 1) * 8, ci = ci0 + nt * 8 + 2 * t + (j & 1);
            if (co < C && ci < C) dst[(size_t)co * C + ci] = acc[nt][j];
        }
}

// grad_w[co][ci][K-1-dh][K-1-dw] = -(sum over shares), zero outside the channel mask of the centre tap.
// LANES adjacent lanes share one entry: lane q adds the shares b = q, q+LANES, ... in that order (up to sixteen
// loads in flight), then the LANES sums are combined in a fixed order by shuffles -- the result does not depend
// on scheduling.  LANES = 4 shortens the chain of dependent loads where there are few entries (few CTAs);
// LANES = 1 (one thread per entry, fully coalesced rows) is faster where the entries alone fill the GPU.
template <int LANES>
__global__ void __launch_bounds__(256) gradw_reduce_kernel(const float* __restrict__ partials, float* __restrict__ grad_w,
                                                           int nbc, int C, int K, const LogdetFuse ld)
{
    constexpr int EPW = 32 / LANES;                      // entries per warp
    constexpr int INF = LANES == 1 ? 8 : 16;             // loads in flight per thread
    const int NA = K * K * C * C;
    const int q = threadIdx.x % LANES;
    const int nper = (nbc + LANES - 1) / LANES;          // shares per lane
    const int NAR = (NA + EPW - 1) / EPW * EPW;          // whole warps stay in the loop for the shuffles
    for (int e0 = (blockIdx.x * blockDim.x + threadIdx.x) / LANES; e0 < NAR; e0 += (gridDim.x * blockDim.x) / LANES) {
        const int e = e0 < NA ? e0 : NA - 1;
        float s = 0.f;
        for (int i0 = 0; i0 < nper; i0 += INF) {
            float v[INF];
#pragma unroll
            for (int j = 0; j < INF; ++j) {
                const int b = q + LANES * (i0 + j);
                v[j] = __ldcg(partials + (size_t)(b < nbc ? b : nbc - 1) * NA + e);
            }
#pragma unroll
            for (int j = 0; j < INF; ++j)
                if (q + LANES * (i0 + j) < nbc) s += v[j];
        }
#pragma unroll
        for (int o = 1; o < LANES; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (q == 0 && e0 < NA) {
            const int ci = e % C, co = (e / C) % C, tap = e / (C * C);
            const int dh = tap / K, dw = tap % K;
            grad_w[((co * C + ci) * K + (K - 1 - dh)) * K + (K - 1 - dw)] = finish_grad_w(s, co, ci, tap, C, K, ld);
        }
    }
}

struct GradWPlan {
    bool ok = false;
    int TC = 3, tiles = 1, nbc = 1, plane = 0, grid = 0;
    int nbc_all = 0, grid_all = 0;      // tiles of 16 channels on the tensor pipe: shares and CTAs when one CTA covers all taps
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
    if (pl.TC == 1) {
        int na = (2 * sm_count) / (pl.tiles * pl.tiles);
        if (na < 1) na = 1;
        if (na > B) na = B;
        const int pa = (B + na - 1) / na;
        na = (B + pa - 1) / pa;
        pl.nbc_all = na;
        pl.grid_all = pl.tiles * pl.tiles * na;
    }
    pl.ok = true;
    return pl;
}

// ---------------------------------------------------------------------------
// Weight gradient for few channels (C <= 4): the contraction runs over B*H*W
// pixels while there are only C*C*K*K sums, so the pixels are what is spread
// over the GPU.  A CTA takes (image, row band) items; it stages the band's
// grad_y rows and the x rows that reach K-1 rows above it in shared memory,
// one bulk (TMA) copy per channel (the rows of a band are contiguous in NCHW;
// a few large copies, because the copy engine takes on the order of a hundred
// cycles per copy whatever its size).  A warp owns one channel pair (co, ci);
// its lanes walk the
// band's quads of four pixels and keep the K*K sums in registers: per quad one
// 16-byte load of grad_y and, per kernel row, two of x and 4*K FMAs.  The
// lanes' sums are added by shuffles, the warps' and then the CTA's sums go to
// global memory, and the CTA that finishes last adds all CTAs' sums in CTA
// order, negates them and applies the channel mask -- the result does not
// depend on the order in which CTAs ran.
// ---------------------------------------------------------------------------
struct GradWSmallParams {
    const float* gy;       // [B][C][H][W]
    const float* x;        // [B][C][H][W]
    float* partials;       // [grid][NAP]   (tap = dh*K + dw, then co, then ci)
    float* grad_w;         // [C][C][K][K]
    unsigned* counter;     // zero on entry; the last CTA resets it
    int B, H, W;
    int RB, nbands;        // rows per band, bands per image
    int gst, xst;          // row strides of the staged grad_y and x bands (floats, multiples of 4)
    int stage;             // floats of dynamic shared memory (the last CTA stages partial sums there)
    int bulk;              // rows are 16-byte aligned multiples of 16 bytes: stage them with bulk copies
    FastDiv div_bands, div_gcpr, div_xcpr, div_rb, div_xr, div_qpr;
    LogdetFuse ld;         // the log-det's term on the diagonal of grad_w (optional)
};

template <int C, int K>
struct GradWSmallShape {
    static constexpr int NA = C * C * K * K, NAP = (NA + 3) & ~3, KK = K * K;
    static constexpr int NCOMBO = C * C;                                   // channel pairs (co, ci)
    static constexpr int WPC = C == 1 ? 16 : (C == 2 ? 4 : (C == 3 ? 2 : 1));   // warps per channel pair
    static constexpr int NW = NCOMBO * WPC, NT = 32 * NW, NSL = 32 * WPC;
    static_assert(KK <= 32 && NT <= 1024, "shape outside the kernel's limits");
};

template <int C, int K>
__global__ void __launch_bounds__(GradWSmallShape<C, K>::NT) gradw_small_kernel(GradWSmallParams p)
{
    using S = GradWSmallShape<C, K>;
    constexpr int NA = S::NA, NAP = S::NAP, KK = S::KK, NT = S::NT, NW = S::NW, NSL = S::NSL, WPC = S::WPC;
    extern __shared__ __align__(128) float smem[];
    __shared__ float red[NW * KK > NA ? NW * KK : NA];
    __shared__ unsigned long long bar;
    __shared__ unsigned ticket;
    const int H = p.H, W = p.W, HW = H * W, RB = p.RB, XR = RB + K - 1;
    const int gst = p.gst, xst = p.xst;
    float* gsm = smem;                           // [C][RB][gst]
    float* xsm = smem + C * RB * gst;            // [C][XR][xst]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int combo = warp / WPC, slice = (warp - combo * WPC) * 32 + lane;
    const int co = combo / C, ci = combo - co * C;
    const int gcpr = (gst + 31) >> 5, xcpr = (xst + 31) >> 5;      // 32-column chunks per staged row
    const int nrow_g = C * RB;                                     // staged grad_y rows of one band
    const int nwi_g = nrow_g * gcpr, nwi = nwi_g + C * XR * xcpr;  // (row, chunk) items of one band
    const int qpr = gst >> 2, nq = RB * qpr;

    float acc[K][K];
#pragma unroll
    for (int a = 0; a < K; ++a)
#pragma unroll
        for (int d = 0; d < K; ++d) acc[a][d] = 0.f;

    // shared-memory set-up needs nothing from the predecessor kernel
    if (tid == 0) { mbar_init(&bar, 1); fence_mbar_init(); }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();

    unsigned phase = 0;
    const int items = p.B * p.nbands;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int n = fast_div(item, p.div_bands), band = item - n * p.nbands;
        const int h0 = band * RB;
        const float* gsrc = p.gy + (size_t)n * C * HW;
        const float* xsrc = p.x + (size_t)n * C * HW;
        if (item != (int)blockIdx.x) __syncthreads();      // the previous band has been consumed
        if (p.bulk) {
            // rows outside the image are zeroed by plain stores; the rows inside arrive by one bulk copy per
            // channel and operand (row strides equal W here, so a band is contiguous on both sides)
            const int gv = min(RB, H - h0);                       // grad_y rows inside the image
            const int xlo = max(0, h0 - (K - 1)), xv = min(H, h0 + RB) - xlo;   // first x row inside, and how many
            const int xskip = xlo - (h0 - (K - 1));               // x rows above the image
            const int gz = (RB - gv) * W, xzt = xskip * W, xzb = (XR - xskip - xv) * W;    // floats to zero per channel
            if (gz > 0 || xzt > 0 || xzb > 0) {
#pragma unroll 1
                for (int c = 0; c < C; ++c) {
                    for (int i = tid; i < gz; i += NT) gsm[(c * RB + gv) * gst + i] = 0.f;
                    for (int i = tid; i < xzt; i += NT) xsm[c * XR * xst + i] = 0.f;
                    for (int i = tid; i < xzb; i += NT) xsm[(c * XR + xskip + xv) * xst + i] = 0.f;
                }
            }
            fence_proxy_async();
            if (warp == 0) {
                if (lane == 0) mbar_expect_tx(&bar, (unsigned)(C * (gv + xv) * W * 4));
                __syncwarp();
                if (lane < C) bulk_g2s(gsm + lane * RB * gst, gsrc + lane * HW + h0 * W, (unsigned)(gv * W * 4), &bar);
                else if (lane < 2 * C)
                    bulk_g2s(xsm + ((lane - C) * XR + xskip) * xst, xsrc + (lane - C) * HW + xlo * W, (unsigned)(xv * W * 4), &bar);
            }
            const bool ok = mbar_wait_bounded(&bar, phase);
            phase ^= 1u;
            if (!__syncthreads_and(ok)) { if (tid == 0) raise_status(INVCONV_TIMEOUT); break; }
        } else {
            for (int wi0 = warp; wi0 < nwi; wi0 += NW * 8) {     // eight loads in flight per thread, no branches
                float v[8];
                int so[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int wi = wi0 + NW * q;
                    const bool isg = wi < nwi_g;                // a grad_y row, else an x row
                    const int wj = isg ? wi : wi - nwi_g;
                    const int cpr = isg ? gcpr : xcpr, st = isg ? gst : xst, rows = isg ? RB : XR;
                    const int row = isg ? fast_div(wj, p.div_gcpr) : fast_div(wj, p.div_xcpr);
                    const int col = (wj - row * cpr) * 32 + lane;
                    const int c = isg ? fast_div(row, p.div_rb) : fast_div(row, p.div_xr);
                    const int h = h0 + row - c * rows - (isg ? 0 : K - 1), w = col;
                    const bool in_s = wi < nwi && col < st;
                    const bool in_g = in_s && w < W && h >= 0 && h < H;
                    const float val = __ldcg((isg ? gsrc : xsrc) + (in_g ? c * HW + h * W + w : 0));
                    v[q] = in_g ? val : 0.f;
                    so[q] = in_s ? (isg ? 0 : C * RB * gst) + row * st + col : -1;
                }
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (so[q] >= 0) smem[so[q]] = v[q];
            }
            __syncthreads();
        }
        const float* gq = gsm + co * RB * gst;
        const float* xq = xsm + ci * XR * xst;
        for (int q = slice; q < nq; q += NSL) {
            const int r = fast_div(q, p.div_qpr), w0 = (q - r * qpr) * 4;
            const float4 g = *reinterpret_cast<const float4*>(gq + r * gst + w0);
            const float gg[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
            for (int dh = 0; dh < K; ++dh) {
                const float* xr = xq + (r + K - 1 - dh) * xst + w0;       // band row r meets x row r - dh
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);               // the K-1 columns to the left of the quad
                if (w0 > 0) a = *reinterpret_cast<const float4*>(xr - 4);
                const float4 b = *reinterpret_cast<const float4*>(xr);
                const float vv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
                for (int d = 0; d < K; ++d)
#pragma unroll
                    for (int px = 0; px < 4; ++px) acc[dh][d] = fmaf(gg[px], vv[4 + px - d], acc[dh][d]);
            }
        }
    }
    // let the next kernel on the stream be scheduled only now: its CTAs would otherwise sit on the SMs (and
    // hold their registers and shared memory) for this kernel's whole run, which measured slower
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // lanes -> warp -> CTA
    {
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = i < KK ? acc[(i < KK ? i : 0) / K][(i < KK ? i : 0) % K] : 0.f;
        const float tot = transpose_reduce32(v, lane);
        if (lane < KK) red[warp * KK + lane] = tot;
    }
    __syncthreads();
    float* part = p.partials + (size_t)blockIdx.x * NAP;
    for (int e = tid; e < NA; e += NT) {           // e = (co*C + ci)*K*K + dh*K + dw
        const int cb = e / KK, tap = e - cb * KK;
        float s = 0.f;
#pragma unroll
        for (int sub = 0; sub < WPC; ++sub) s += red[(cb * WPC + sub) * KK + tap];
        __stcg(part + tap * C * C + cb, s);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) ticket = atomicAdd(p.counter, 1u);
    __syncthreads();
    if (ticket != gridDim.x - 1) return;

    // last CTA: add the CTAs' sums in CTA order, staged through shared memory sixteen bytes at a time
    __threadfence();
    const int G = (int)gridDim.x;
    const int chunk = min(G, p.stage / NAP);
    for (int b0 = 0; b0 < G; b0 += chunk) {
        const int nbk = min(chunk, G - b0);
        const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)b0 * NAP);
        float4* dst = reinterpret_cast<float4*>(smem);
        const int tot4 = nbk * (NAP / 4);
        for (int i0 = tid; i0 < tot4; i0 += NT * 8) {
            float4 tv[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) tv[q] = __ldcg(src + min(i0 + q * NT, tot4 - 1));     // clamped: no branch
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (i0 + q * NT < tot4) dst[i0 + q * NT] = tv[q];
        }
        __syncthreads();
        for (int e = tid; e < NA; e += NT) {
            float s = b0 == 0 ? 0.f : red[e];
#pragma unroll 8
            for (int b = 0; b < nbk; ++b) s += smem[b * NAP + e];
            red[e] = s;
        }
        __syncthreads();
    }
    for (int e = tid; e < NA; e += NT) {
        const int ci_ = e % C, co_ = (e / C) % C, tap = e / (C * C);
        const int dh_ = tap / K, dw_ = tap % K;
        p.grad_w[((co_ * C + ci_) * K + (K - 1 - dh_)) * K + (K - 1 - dw_)] = finish_grad_w(red[e], co_, ci_, tap, C, K, p.ld);
    }
    if (tid == 0) *p.counter = 0u;
}

struct GradWSmallPlan {
    bool ok = false;
    int RB = 0, nbands = 0, gst = 0, xst = 0, grid = 0;
    size_t smem = 0;
};

// Bands are sized so that about one CTA per SM gets an item; a band never has fewer than four rows (the K-1
// halo rows are loaded once per band).
inline GradWSmallPlan plan_gradw_small(int B, int C, int H, int W, int K, size_t max_smem, size_t stage_smem, int sm_count)
{
    GradWSmallPlan pl;
    if (B < 1 || C > 4 || K > 5) return pl;
    const int Wq = (W + 3) & ~3;
    pl.gst = Wq;
    pl.xst = Wq;
    int nbands = sm_count / B;
    if (nbands > (H + 3) / 4) nbands = (H + 3) / 4;
    if (nbands < 1) nbands = 1;
    for (;; ++nbands) {
        const int RB = (H + nbands - 1) / nbands;
        const size_t bytes = sizeof(float) * (size_t)C * ((size_t)RB * pl.gst + (size_t)(RB + K - 1) * pl.xst);
        if (bytes <= max_smem) { pl.RB = RB; pl.smem = bytes; break; }
        if (RB == 1) return pl;
    }
    pl.nbands = (H + pl.RB - 1) / pl.RB;
    const int items = B * pl.nbands;
    const int rounds = (items + sm_count - 1) / sm_count;
    pl.grid = (items + rounds - 1) / rounds;           // every CTA takes `rounds` items (the last ones one fewer)
    // the last CTA stages the CTAs' sums in the same shared memory: all of them at once where that fits
    const size_t nap = (size_t)((C * C * K * K + 3) & ~3);
    size_t want = sizeof(float) * nap * (size_t)pl.grid;
    if (want > stage_smem) want = stage_smem - stage_smem % (sizeof(float) * nap);
    if (pl.smem < want) pl.smem = want;
    pl.ok = true;
    return pl;
}

}  // namespace invconv

// Warp-shuffle wavefront for few channels (C <= 4).
//
// One warp owns a block of 32 image rows: lane l solves row 32*j + l and, at
// local step s, the pixel in column s - l, so a warp walks one anti-diagonal
// per step (Section 3: pixels on one anti-diagonal are unordered and solved in
// parallel; the diagonals follow one another).  The k-1 already-solved
// neighbours in the lane's own row live in its registers; the rows above
// arrive from the lanes above by one shuffle per row and channel, so a step
// needs no barrier.  The whole image sits in shared memory, brought in by one
// bulk (TMA) copy and solved in place, then written back by one bulk copy, so
// every HBM access is a full contiguous transfer.
//
// Images taller than 32 rows use several warps: row block j starts a column as
// soon as block j-1 has published it (a progress counter in shared memory,
// polled every 8 steps with a bounded spin), i.e. the blocks run as a skewed
// pipeline instead of a global lock-step.
//
// The channel solve of the centre tap is folded into the taps once per call:
// with L = w[:, :, k-1, k-1] (lower triangular) the recurrence
//     L x_p = y_p - sum_{delta != 0} W_delta x_{p-delta}
// is solved as  x_p = L^-1 y_p - sum (L^-1 W_delta) x_{p-delta},
// which is the paper's own unit-diagonal form (Section 3) for the transformed
// kernel.  The transposed solve (grad_y, Theorem 1) is the same walk on the
// image rotated by 180 degrees with  L^-T W_delta^T.
//
// grad_w (Theorem 2): up to 81 partial sums ride along in the reverse wavefront
// (the solved neighbour grad_y[q + delta] is already in registers when x[q] is
// loaded); warp partials are combined per CTA and the last CTA to finish sums
// the CTA partials in a fixed order.  Larger kernels and images that stay in
// global memory get grad_w from the pixel-parallel kernel of gradw_kernels.cuh
// after the wavefront; a post-pass over the two resident images (lane =
// column, k x k window of x in registers) remains as the fallback for shapes
// that kernel's plan does not serve.
//
// Two variants of the walk serve shapes where one lane per row is not enough:
// the ring mode (images larger than shared memory stream through a per-warp
// ring of 128 columns) and the channel-split walk (lane = row x output
// channel, for C >= 3 with 5x5 kernels); both are described at their code.
#pragma once

#include <cstdio>
#include <cuda_bf16.h>

#include "common.cuh"
#include "tma.cuh"

#ifndef INVCONV_UNROLL_K5
#define INVCONV_UNROLL_K5 4      // unroll factor (in units of K-1 steps) of the one-channel 5x5 step loop
#endif

namespace invconv {

struct WarpParams {
    const float* rhs;      // y (forward) or grad_x (backward)
    const float* w;        // [C][C][K][K]
    float* out;            // x (forward) or grad_y (backward)
    const float* xsaved;   // backward: the saved forward output x
    float* grad_w;         // backward: may be nullptr
    float* partials;       // backward: [gridDim.x][K*K*C*C] scratch
    unsigned* counter;     // backward: one control word, zero on entry and on exit
    int B, H, W;
    int nb;                // row blocks (warps) per image
    int ipc;               // images per CTA
    int bulk;              // images are 16-byte aligned multiples of 16 bytes
    int glb;               // images stay in global memory (too large for shared memory)
    int vec;               // image rows are 16-byte aligned multiples of 16 bytes (ring mode: 16-byte copies)
    // The per-pixel neighbours of the layer in a flow step (Actnorm z = s*x + b, then the 1x1 convolution
    // u = V z), applied while the image is on chip; all nullptr = the plain layer.
    const float* mix_V = nullptr;   // [C][C]
    const float* mix_s = nullptr;   // [C]
    const float* mix_b = nullptr;   // [C] (forward only)
    float* mix_out = nullptr;       // forward: u [B][C][H][W], written beside x
    int mix_in = 0;                 // backward: rhs holds grad_u; grad_x = s * (V^T grad_u) is formed after the load
    float* logdet_out = nullptr;    // forward: CTA 0 also writes the layer's log-det (one float)
    LogdetFuse ld;                  // backward: the log-det's term on the diagonal of grad_w
    // Reduced-precision storage: rhs, out and xsaved point to bfloat16 images (C*H*W a multiple of 8, bulk copies,
    // images resident in shared memory, no flow-step neighbours).  They are widened to fp32 once they have
    // arrived in shared memory and narrowed again on the way out; every sum in between is fp32 as without it.
    int bf16 = 0;
};

template <int C> struct ColVec;
template <> struct ColVec<1> { using type = float;  static constexpr int CP = 1; };
template <> struct ColVec<2> { using type = float2; static constexpr int CP = 2; };
template <> struct ColVec<3> { using type = float4; static constexpr int CP = 4; };
template <> struct ColVec<4> { using type = float4; static constexpr int CP = 4; };

template <int C, int K>
struct WarpShape {
    static constexpr int KK = K * K;
    static constexpr int CP = ColVec<C>::CP;
    static constexpr int NA = KK * C * C;           // kernel entries
    static constexpr int NAP = KK * C * CP;         // padded copy in shared memory
    static constexpr bool WREG = NA <= 144;         // transformed kernel held in registers
    static constexpr int COB = (NA <= 100) ? C : 1; // output channels per grad_w pass
};

// Column a = 0..C-1 of the transformed kernel for (tap, input channel b).
template <int C>
__device__ __forceinline__ void load_col(const float* As, int idx, float (&col)[C])
{
    using V = typename ColVec<C>::type;
    const V v = reinterpret_cast<const V*>(As)[idx];
    if constexpr (C == 1) { col[0] = v; }
    else if constexpr (C == 2) { col[0] = v.x; col[1] = v.y; }
    else if constexpr (C == 3) { col[0] = v.x; col[1] = v.y; col[2] = v.z; }
    else { col[0] = v.x; col[1] = v.y; col[2] = v.z; col[3] = v.w; }
}

// Transformed kernel into shared memory: As[(tap*C + b)*CP + a], tap = dh*K + dw,
//   forward : tap 0 -> L^-1[a][b];          tap != 0 -> (L^-1 W_delta)[a][b]
//   backward: tap 0 -> L^-1[b][a];          tap != 0 -> sum_m L^-1[m][a] w[b][m][delta]
// where W_delta[co][ci] = w[co][ci][K-1-dh][K-1-dw].
template <int C, int K, bool BWD>
__device__ void build_transformed_kernel(const float* __restrict__ w, float* As)
{
    constexpr int KK = K * K, CP = ColVec<C>::CP;
    constexpr int ctr = KK - 1;
    // the taps of this thread's first entry are requested before the centre tap, so that one memory latency
    // covers both (the entry needs L^-1, which needs the centre tap)
    float wpre[C];
    {
        const int e = threadIdx.x;
        const int b = (e / C) % C, tap = e / (C * C);
        const int t = (K - 1 - tap / K) * K + (K - 1 - tap % K);
#pragma unroll
        for (int m = 0; m < C; ++m) {
            wpre[m] = 0.f;
            if (e < KK * C * C && tap != 0) wpre[m] = BWD ? __ldg(w + (b * C + m) * KK + t) : __ldg(w + (m * C + b) * KK + t);
        }
    }
    float L[C][C], Li[C][C];
#pragma unroll
    for (int i = 0; i < C; ++i)
#pragma unroll
        for (int j = 0; j < C; ++j) {
            L[i][j] = (j <= i) ? __ldg(w + (i * C + j) * KK + ctr) : 0.f;
            Li[i][j] = 0.f;
        }
#pragma unroll
    for (int j = 0; j < C; ++j) {
        Li[j][j] = 1.0f / L[j][j];
#pragma unroll
        for (int i = j + 1; i < C; ++i) {
            float s = 0.f;
#pragma unroll
            for (int m = j; m < i; ++m) s += L[i][m] * Li[m][j];
            Li[i][j] = -s / L[i][i];
        }
    }
    for (int e = threadIdx.x; e < KK * C * C; e += blockDim.x) {
        const int a = e % C, b = (e / C) % C, tap = e / (C * C);
        const int dh = tap / K, dw = tap % K;
        const int t = (K - 1 - dh) * K + (K - 1 - dw);
        float v = 0.f;
        if (tap == 0) {
#pragma unroll
            for (int i = 0; i < C; ++i)
#pragma unroll
                for (int j = 0; j < C; ++j)
                    if (i == (BWD ? b : a) && j == (BWD ? a : b)) v = Li[i][j];
        } else {
#pragma unroll
            for (int m = 0; m < C; ++m) {
                float li = 0.f;
#pragma unroll
                for (int i = 0; i < C; ++i)
#pragma unroll
                    for (int j = 0; j < C; ++j)
                        if (i == (BWD ? m : a) && j == (BWD ? a : m)) li = Li[i][j];
                const float wv = e == (int)threadIdx.x ? wpre[m]
                                                       : (BWD ? __ldg(w + (b * C + m) * KK + t) : __ldg(w + (m * C + b) * KK + t));
                v += li * wv;
            }
        }
        As[(tap * C + b) * CP + a] = v;
    }
}

// The wavefront over one block of up to 32 rows.  Logical pixel (lh, lw) of
// channel c lives at img[c*HW + origin + sgn*(lh*W + lw)] (sgn = -1 walks the
// rotated image of the transposed solve).  Returns false if a wait gave up.
//
// The step loop is unrolled by K-1 so that the sliding windows of solved
// neighbours rotate through registers by renaming instead of moves: the value
// produced at step s lives in slot s mod (K-1).  Lanes that have no row above
// inside the block (lane <= d for the row d+1 above) get zeroed copies of the
// taps that read those rows when the block is the image's first, so the
// shuffle result feeds the FMA directly with no select on the dependent chain.
//
// GW = true (transposed solve only) also accumulates this block's share of
// grad_w (Theorem 2 in closed form) on the fly:  with q the lane's pixel,
//   part[tap][co][ci] += grad_y[co][q + delta] * x[ci][q],
// where grad_y[q + delta] is exactly the solved neighbour the step already
// holds in registers; it costs one shared-memory load of x[q] and K*K*C*C FMAs
// off the dependent chain.  The partial sums go to gw_dst[(tap*C + co)*C + ci].
//
// GLB = true serves images too large for shared memory: the right-hand side is read from, and the solution
// written to, global memory directly (each lane walks its own row, so a 32-byte sector is fetched once and
// then hit in L1 for eight steps; sectors are prefetched two ahead), and the K-1 bottom rows of every row
// block go to a small shared-memory buffer `bnd` ([block][channel][row][W]) for the block below.
//
// RING = true (with GLB and MULTI, never GW) streams such images through shared memory instead: every warp
// owns a ring of 128 physical columns of its 32 rows (four tiles of 32 columns; per channel kRingCh floats,
// row stride 128, slot = physical column & 127, so the skewed accesses of the lanes stay conflict-free).
// Every 32 steps the warp (a) waits for the tile it asked for 32 steps earlier, (b) writes the tile that all
// of its lanes have finished (two tiles back) to global memory with coalesced stores, and (c) asks for the
// tile two ahead with asynchronous copies into the slot just freed.  The step itself is the shared-memory
// step: no global access on the dependent chain.  `vec` says whether rows are 16-byte aligned multiples of
// 16 bytes (16-byte copies and stores), else single floats are moved.
constexpr int kRingCh = 32 * 128 + 32;       // floats per channel of one warp's ring; the tail is a scratch slot

// Tile t of the ring (logical columns 32t .. 32t+31 of the walk) as physical columns: first column and count.
__device__ __forceinline__ void ring_tile_cols(int t, int W, int sgn, int& base, int& lo, int& hi)
{
    base = sgn > 0 ? 32 * t : W - 32 * (t + 1);      // may be negative for the last tile of a reversed walk
    lo = max(base, 0);
    hi = min(base + 32, W);
}

template <int C>
__device__ __forceinline__ void ring_load_tile(float* ring, const float* rin, int t, int H, int W, int sgn, int j,
                                               int rows, int lane, bool vec)
{
    int base, lo, hi;
    ring_tile_cols(t, W, sgn, base, lo, hi);
    const int HW = H * W;
    if (vec) {
#pragma unroll
        for (int c = 0; c < C; ++c)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = i * 32 + lane, row = v >> 3, col = base + 4 * (v & 7);
                const int pr = sgn > 0 ? 32 * j + row : H - 1 - (32 * j + row);
                const bool ok = row < rows && col >= lo && col < hi;
                cp_async_f32x4(ring + c * kRingCh + row * 128 + (col & 127), rin + (ok ? c * HW + pr * W + col : 0), ok);
            }
    } else {
        const int col = base + lane;
        const bool okc = col >= lo && col < hi;
#pragma unroll
        for (int c = 0; c < C; ++c)
#pragma unroll 8
            for (int row = 0; row < 32; ++row) {
                const int pr = sgn > 0 ? 32 * j + row : H - 1 - (32 * j + row);
                const bool ok = okc && row < rows;
                cp_async_f32(ring + c * kRingCh + row * 128 + (col & 127), rin + (ok ? c * HW + pr * W + col : 0), ok);
            }
    }
}

template <int C>
__device__ __forceinline__ void ring_store_tile(const float* ring, float* out, int t, int H, int W, int sgn, int j,
                                                int rows, int lane, bool vec)
{
    int base, lo, hi;
    ring_tile_cols(t, W, sgn, base, lo, hi);
    const int HW = H * W;
    if (vec) {
#pragma unroll
        for (int c = 0; c < C; ++c)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = i * 32 + lane, row = v >> 3, col = base + 4 * (v & 7);
                const int pr = sgn > 0 ? 32 * j + row : H - 1 - (32 * j + row);
                const float4 val = *reinterpret_cast<const float4*>(ring + c * kRingCh + row * 128 + (col & 127));
                if (row < rows && col >= lo && col < hi) *reinterpret_cast<float4*>(out + c * HW + pr * W + col) = val;
            }
    } else {
        const int col = base + lane;
        const bool okc = col >= lo && col < hi;
#pragma unroll
        for (int c = 0; c < C; ++c)
#pragma unroll 8
            for (int row = 0; row < 32; ++row) {
                const int pr = sgn > 0 ? 32 * j + row : H - 1 - (32 * j + row);
                const float val = ring[c * kRingCh + row * 128 + (col & 127)];
                if (okc && row < rows) out[c * HW + pr * W + col] = val;
            }
    }
}

template <int C, int K, bool MULTI, bool GW, bool GLB = false, bool RING = false>
__device__ __forceinline__ bool wavefront_block(float* img, const float* As, int H, int W, int origin, int sgn,
                                                int j, volatile int* progress, int lane,
                                                const float* xs = nullptr, float* gw_dst = nullptr,
                                                const float* rin = nullptr, float* bnd = nullptr, int nb = 1,
                                                int dummy_idx = 0, float* ring = nullptr, bool vec = false)
{
    static_assert(!RING || (GLB && MULTI && !GW), "the ring serves the global-memory mode without fused grad_w");
    if (!GLB) rin = img;
    using S = WarpShape<C, K>;
    constexpr int KM = K - 1;
    const int HW = H * W;
    const int rows = min(32, H - 32 * j);
    const int nsteps = W + rows - 1;
    const int nsteps_up = (nsteps + KM - 1) / KM * KM;
    const int prod_steps = (W + 31 + KM - 1) / KM * KM;
    const unsigned Wl = lane < rows ? (unsigned)W : 0u;     // active  <=>  (unsigned)lw < Wl
    const bool first_block = !MULTI || j == 0;

    float Ar[S::WREG ? S::NA : 1];
    if constexpr (S::WREG) {
#pragma unroll
        for (int t = 0; t < S::KK * C; ++t) {
            float col[C];
            load_col<C>(As, t, col);
            const int dh = t / (C * K);
            const bool dead = first_block && dh >= 1 && lane < dh;   // the row dh above lies outside the image
#pragma unroll
            for (int a = 0; a < C; ++a) Ar[t * C + a] = dead ? 0.f : col[a];
        }
    }
    float own[C][KM];          // slot (s mod KM) <- x[b][lh][lw] of step s
    float up[KM][C][KM];       // slot (s mod KM) <- x[b][lh-1-d][lw] of step s
#pragma unroll
    for (int b = 0; b < C; ++b)
#pragma unroll
        for (int q = 0; q < KM; ++q) {
            own[b][q] = 0.f;
#pragma unroll
            for (int d = 0; d < KM; ++d) up[d][b][q] = 0.f;
        }
    float gacc[GW ? S::NA : 1];
#pragma unroll
    for (int i = 0; i < (GW ? S::NA : 1); ++i) gacc[i] = 0.f;
    int p = origin + sgn * ((32 * j + lane) * W - lane);    // offset of (lh, lw) at step 0
    int pcol = sgn > 0 ? -lane : W - 1 + lane;              // RING: physical column of (lh, lw) at step 0
    const int rbase = lane * 128;
    const int ntiles = (W + 31) >> 5;
    int next_flush = 0;
    if constexpr (RING) {
        ring_load_tile<C>(ring, rin, 0, H, W, sgn, j, rows, lane, vec);
        if (ntiles > 1) ring_load_tile<C>(ring, rin, 1, H, W, sgn, j, rows, lane, vec);
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
    }
    float rnext[C];
#pragma unroll
    for (int c = 0; c < C; ++c) {
        if constexpr (RING) rnext[c] = (lane == 0 && Wl > 0) ? ring[c * kRingCh + rbase + (pcol & 127)] : 0.f;
        else rnext[c] = (lane == 0 && Wl > 0) ? rin[c * HW + p] : 0.f;
    }

    constexpr int UNR = C >= 3 ? 2 : (K == 5 ? INVCONV_UNROLL_K5 : 4);
#pragma unroll(UNR)
    for (int s0 = 0; s0 < nsteps_up; s0 += KM) {
        if constexpr (RING) {
            if ((s0 & 31) == 0) {
                const int t = s0 >> 5;
                cp_async_wait<0>();                      // tile t+1, asked for 32 steps ago
                __syncwarp();
                if (t >= 2 && t - 2 < ntiles) { ring_store_tile<C>(ring, img, t - 2, H, W, sgn, j, rows, lane, vec); next_flush = t - 1; }
                __syncwarp();
                if (t + 2 < ntiles) ring_load_tile<C>(ring, rin, t + 2, H, W, sgn, j, rows, lane, vec);
                cp_async_commit();
            }
        }
        if constexpr (MULTI) {
            if (j > 0 && (s0 & 7) == 0) {
                const int need = min(s0 + 39, prod_steps);
                unsigned spins = 0;
                bool ok = true;
                while (progress[j - 1] < need) {
                    if (++spins > kMaxSpins) { ok = false; break; }
                }
                if (!__all_sync(0xffffffffu, ok)) {
                    if constexpr (RING) cp_async_wait<0>();
                    return false;
                }
                __threadfence_block();
            }
        }
#pragma unroll
        for (int u = 0; u < KM; ++u) {
            const unsigned ulw = (unsigned)(s0 + u - lane);
            const bool active = ulw < Wl;
            float r[C];
#pragma unroll
            for (int c = 0; c < C; ++c) r[c] = rnext[c];
            float xq[GW ? C : 1];
            if constexpr (GW) {
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    if constexpr (GLB) xq[c] = active ? xs[c * HW + p] : 0.f;
                    else { const float t = xs[c * HW + (active ? p : origin)]; xq[c] = active ? t : 0.f; }
                }
            }
            {
                const bool act1 = (ulw + 1u) < Wl;
                if constexpr (RING) {
                    const int rn = act1 ? rbase + ((pcol + sgn) & 127) : 32 * 128;   // inactive lanes: the scratch slot
#pragma unroll
                    for (int c = 0; c < C; ++c) { const float t = ring[c * kRingCh + rn]; rnext[c] = act1 ? t : 0.f; }
                } else if constexpr (GLB) {
#pragma unroll
                    for (int c = 0; c < C; ++c) rnext[c] = act1 ? rin[c * HW + p + sgn] : 0.f;
                } else {
                    const int pn = act1 ? p + sgn : origin;  // inactive lanes read a valid dummy location: no branch
#pragma unroll
                    for (int c = 0; c < C; ++c) { const float t = rin[c * HW + pn]; rnext[c] = act1 ? t : 0.f; }
                }
                if constexpr (GLB && !RING) {
                    if (((ulw + 1u) & 7u) == 0u && (ulw + 17u) < Wl) {
#pragma unroll
                        for (int c = 0; c < C; ++c) {
                            asm volatile("prefetch.global.L1 [%0];" ::"l"(rin + c * HW + p + sgn * 17));
                            if constexpr (GW) asm volatile("prefetch.global.L1 [%0];" ::"l"(xs + c * HW + p + sgn * 17));
                        }
                    }
                }
            }
            // newest column of the rows above: by shuffle inside the block, from shared memory across blocks
            float nu[KM][C];
#pragma unroll
            for (int d = 0; d < KM; ++d)
#pragma unroll
                for (int b = 0; b < C; ++b) {
                    float v = __shfl_up_sync(0xffffffffu, own[b][(u - 1 - d + 2 * KM) % KM], d + 1);
                    if constexpr (MULTI) {
                        // lanes whose row above lies in the previous block read it from shared memory; every lane
                        // issues the (clamped) load so that the step stays branch-free
                        const bool edge = lane <= d;
                        const bool take = edge && j > 0 && active;
                        float vb;
                        if constexpr (GLB) vb = bnd[take ? (((j - 1) * C + b) * KM + (lane - d - 1 + KM)) * W + (int)ulw : 0];
                        else vb = img[take ? b * HW + p - sgn * (d + 1) * W : dummy_idx];
                        v = edge ? (take ? vb : 0.f) : v;
                    } else if constexpr (!S::WREG) {
                        if (lane <= d) v = 0.f;
                    }
                    nu[d][b] = v;
                }
            // everything that does not depend on the previous step's result
            float acc[C], acc2[C];
#pragma unroll
            for (int a = 0; a < C; ++a) { acc[a] = 0.f; acc2[a] = 0.f; }
#pragma unroll
            for (int b = 0; b < C; ++b) {
                float col[C];
                if constexpr (S::WREG) {
#pragma unroll
                    for (int a = 0; a < C; ++a) col[a] = Ar[b * C + a];
                } else load_col<C>(As, b, col);
#pragma unroll
                for (int a = 0; a < C; ++a) acc[a] = fmaf(col[a], r[b], acc[a]);
            }
#pragma unroll
            for (int dh = 0; dh < K; ++dh)
#pragma unroll
                for (int dw = (dh == 0 ? 2 : 1); dw < K; ++dw)
#pragma unroll
                    for (int b = 0; b < C; ++b) {
                        const int slot = (u - dw + 2 * KM) % KM;      // produced at step s - dw
                        const float v = dh == 0 ? own[b][slot] : up[dh - 1][b][slot];
                        float col[C];
                        if constexpr (S::WREG) {
#pragma unroll
                            for (int a = 0; a < C; ++a) col[a] = Ar[((dh * K + dw) * C + b) * C + a];
                        } else load_col<C>(As, (dh * K + dw) * C + b, col);
                        if (((dh * K + dw) & 1) == 0) {
#pragma unroll
                            for (int a = 0; a < C; ++a) acc[a] = fmaf(-col[a], v, acc[a]);
                        } else {
#pragma unroll
                            for (int a = 0; a < C; ++a) acc2[a] = fmaf(-col[a], v, acc2[a]);
                        }
                    }
#pragma unroll
            for (int a = 0; a < C; ++a) acc[a] += acc2[a];
            // rows two and more above (their shuffles were fed by older results)
#pragma unroll
            for (int d = KM - 1; d >= 1; --d)
#pragma unroll
                for (int b = 0; b < C; ++b) {
                    float col[C];
                    if constexpr (S::WREG) {
#pragma unroll
                        for (int a = 0; a < C; ++a) col[a] = Ar[(((d + 1) * K) * C + b) * C + a];
                    } else load_col<C>(As, ((d + 1) * K) * C + b, col);
#pragma unroll
                    for (int a = 0; a < C; ++a) acc[a] = fmaf(-col[a], nu[d][b], acc[a]);
                }
            // the two taps on the true critical path: left neighbour, then the row above
#pragma unroll
            for (int b = 0; b < C; ++b) {
                float col[C];
                if constexpr (S::WREG) {
#pragma unroll
                    for (int a = 0; a < C; ++a) col[a] = Ar[(1 * C + b) * C + a];
                } else load_col<C>(As, 1 * C + b, col);
#pragma unroll
                for (int a = 0; a < C; ++a) acc[a] = fmaf(-col[a], own[b][(u - 1 + 2 * KM) % KM], acc[a]);
            }
#pragma unroll
            for (int b = 0; b < C; ++b) {
                float col[C];
                if constexpr (S::WREG) {
#pragma unroll
                    for (int a = 0; a < C; ++a) col[a] = Ar[(K * C + b) * C + a];
                } else load_col<C>(As, K * C + b, col);
#pragma unroll
                for (int a = 0; a < C; ++a) acc[a] = fmaf(-col[a], nu[0][b], acc[a]);
            }
            if constexpr (!GLB) {
                // branch-free: lanes outside the image store to a scratch slot
#pragma unroll
                for (int a = 0; a < C; ++a) img[active ? a * HW + p : dummy_idx] = acc[a];
            }
            if constexpr (RING) {
                const int ro = active ? rbase + (pcol & 127) : 32 * 128;
#pragma unroll
                for (int a = 0; a < C; ++a) ring[a * kRingCh + ro] = acc[a];
                // the K-1 bottom rows also go to the boundary buffer of the block below (its last float is scratch)
                const bool pub = active && lane >= 32 - KM && j + 1 < nb;
#pragma unroll
                for (int a = 0; a < C; ++a)
                    bnd[pub ? ((j * C + a) * KM + (lane - (32 - KM))) * W + (int)ulw : nb * C * KM * W] = acc[a];
            }
            if (GLB && !RING && active) {
#pragma unroll
                for (int a = 0; a < C; ++a) img[a * HW + p] = acc[a];
                if constexpr (GLB && MULTI) {
                    if (lane >= 32 - KM && j + 1 < nb) {
#pragma unroll
                        for (int a = 0; a < C; ++a) bnd[((j * C + a) * KM + (lane - (32 - KM))) * W + (int)ulw] = acc[a];
                    }
                }
            }
            if constexpr (GW) {
#pragma unroll
                for (int dh = 0; dh < K; ++dh)
#pragma unroll
                    for (int dw = 0; dw < K; ++dw)
#pragma unroll
                        for (int b = 0; b < C; ++b) {
                            const int slot = (u - dw + 2 * KM) % KM;
                            const float nbr = dh == 0 ? (dw == 0 ? acc[b] : own[b][slot])
                                                      : (dw == 0 ? nu[dh - 1][b] : up[dh - 1][b][slot]);
#pragma unroll
                            for (int c = 0; c < C; ++c)
                                gacc[((dh * K + dw) * C + b) * C + c] =
                                    fmaf(nbr, xq[c], gacc[((dh * K + dw) * C + b) * C + c]);
                        }
            }
#pragma unroll
            for (int b = 0; b < C; ++b) {
                own[b][u] = acc[b];      // lanes before their first column produce exact zeros (zero inputs), lanes past
                                         // their last column only feed lanes that are past theirs too: no select needed
#pragma unroll
                for (int d = 0; d < KM; ++d) up[d][b][u] = nu[d][b];
            }
            p += sgn;
            pcol += sgn;
        }
        if constexpr (MULTI) {
            if (((s0 + KM) & 7) == 0) {
                __threadfence_block();
                __syncwarp();
                if (lane == 0) progress[j] = s0 + KM;
            }
        }
    }
    if constexpr (MULTI) {
        __threadfence_block();
        __syncwarp();
        if (lane == 0) progress[j] = prod_steps;
    }
    if constexpr (RING) {
        cp_async_wait<0>();
        __syncwarp();
        for (int t = next_flush; t < ntiles; ++t) ring_store_tile<C>(ring, img, t, H, W, sgn, j, rows, lane, vec);
    }
    if constexpr (GW) {
        // rows above the image never existed for the first lanes of the first block: drop what they gathered
#pragma unroll
        for (int dh = 1; dh < K; ++dh)
            if (first_block && lane < dh) {
#pragma unroll
                for (int i = 0; i < K * C * C; ++i) gacc[dh * K * C * C + i] = 0.f;
            }
#pragma unroll
        for (int base = 0; base < S::NA; base += 32) {
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = (base + i < S::NA) ? gacc[base + i] : 0.f;
            const float tot = transpose_reduce32(v, lane);
            if (base + lane < S::NA) gw_dst[base + lane] = tot;
        }
    }
    return true;
}

// Channel-split wavefront for kernels whose transformed taps do not fit one lane's registers (C >= 3 with
// K = 5): lane = (row r, output channel a), 32 / C rows per warp.  A lane keeps only column a of every
// (tap, input channel) -- K*K*C registers -- and computes one output channel of its row's pixel per step
// (K*K*C FMAs instead of K*K*C*C).  The solved neighbours of ALL input channels are still needed: the C lanes
// of a row exchange their new values by shuffles (so every lane of the row holds the row's C newest values),
// and the rows above come by shuffles over C*(d+1) lanes.  Row blocks are RPW rows high, so an image needs
// more warps and the skew between consecutive blocks is RPW steps instead of 32.
// Images resident in shared memory only; grad_w never rides along here.
template <int C, int K, bool MULTI>
__device__ __forceinline__ bool wavefront_block_cs(float* img, const float* As, int H, int W, int origin, int sgn,
                                                   int j, volatile int* progress, int lane, int dummy_idx)
{
    using S = WarpShape<C, K>;
    constexpr int KM = K - 1, RPW = 32 / C;
    constexpr int PUB = KM >= 4 ? KM : 4;                   // steps between progress checks / publications
    const int HW = H * W;
    const int r = lane / C, a = lane - r * C;
    const int row0 = RPW * j;
    const int rows = min(RPW, H - row0);
    const int nsteps = W + rows - 1;
    const int nsteps_up = (nsteps + PUB - 1) / PUB * PUB;
    const int prod_steps = (W + RPW - 1 + PUB - 1) / PUB * PUB;
    const unsigned Wl = r < rows ? (unsigned)W : 0u;        // active  <=>  (unsigned)lw < Wl
    const bool first_block = !MULTI || j == 0;

    float Ar[S::KK * C];                                    // column a of (tap, input channel b)
#pragma unroll
    for (int t = 0; t < S::KK * C; ++t) {
        float col[C];
        load_col<C>(As, t, col);
        float v = col[0];
#pragma unroll
        for (int q = 1; q < C; ++q) v = a == q ? col[q] : v;
        const int dh = t / (C * K);
        const bool dead = first_block && dh >= 1 && r < dh;  // the row dh above lies outside the image
        Ar[t] = dead ? 0.f : v;
    }
    float own[C][KM];          // slot (s mod KM) <- x[b][lh][lw] of step s, all input channels b
    float up[KM][C][KM];       // slot (s mod KM) <- x[b][lh-1-d][lw] of step s
#pragma unroll
    for (int b = 0; b < C; ++b)
#pragma unroll
        for (int q = 0; q < KM; ++q) {
            own[b][q] = 0.f;
#pragma unroll
            for (int d = 0; d < KM; ++d) up[d][b][q] = 0.f;
        }
    int p = origin + sgn * ((row0 + r) * W - r);            // offset of (lh, lw) at step 0
    float rnext[C];
#pragma unroll
    for (int c = 0; c < C; ++c) rnext[c] = (r == 0 && Wl > 0) ? img[c * HW + p] : 0.f;

#pragma unroll 1
    for (int s0 = 0; s0 < nsteps_up; s0 += KM) {
        if constexpr (MULTI) {
            if (j > 0 && (s0 % PUB) == 0) {
                const int need = min(s0 + PUB - 1 + RPW, prod_steps);
                unsigned spins = 0;
                bool ok = true;
                while (progress[j - 1] < need) {
                    if (++spins > kMaxSpins) { ok = false; break; }
                }
                if (!__all_sync(0xffffffffu, ok)) return false;
                __threadfence_block();
            }
        }
#pragma unroll
        for (int u = 0; u < KM; ++u) {
            const unsigned ulw = (unsigned)(s0 + u - r);
            const bool active = ulw < Wl;
            float rr[C];
#pragma unroll
            for (int c = 0; c < C; ++c) rr[c] = rnext[c];
            {
                const bool act1 = (ulw + 1u) < Wl;
                const int pn = act1 ? p + sgn : origin;      // inactive lanes read a valid dummy location: no branch
#pragma unroll
                for (int c = 0; c < C; ++c) { const float t = img[c * HW + pn]; rnext[c] = act1 ? t : 0.f; }
            }
            // newest column of the rows above.  Row lh-1 (on the dependent chain): by shuffle inside the block,
            // from shared memory across blocks.  Rows lh-2 and further were solved at least two steps ago and are
            // read back from the image in shared memory (this warp's own stores of earlier steps, or the block
            // above, which the progress counter covers); lanes outside the image or not yet started get zeros.
            float nu[KM][C];
            __syncwarp();
#pragma unroll
            for (int b = 0; b < C; ++b) {
                float v = __shfl_up_sync(0xffffffffu, own[b][(u - 1 + 2 * KM) % KM], C);
                if constexpr (MULTI) {
                    const bool edge = r == 0;
                    const bool take = edge && j > 0 && active;
                    const float vb = img[take ? b * HW + p - sgn * W : dummy_idx];
                    v = edge ? (take ? vb : 0.f) : v;
                }
                nu[0][b] = v;
            }
#pragma unroll
            for (int d = 1; d < KM; ++d) {
                const bool have = active && (row0 + r - d - 1 >= 0);
#pragma unroll
                for (int b = 0; b < C; ++b) {
                    const float t = img[have ? b * HW + p - sgn * (d + 1) * W : dummy_idx];
                    nu[d][b] = have ? t : 0.f;
                }
            }
            // everything off the dependent chain, on six independent accumulators (a lone accumulator would make
            // every FMA wait four cycles for the one before it)
            float pa[4] = {0.f, 0.f, 0.f, 0.f}, pn = 0.f, py = 0.f;
#pragma unroll
            for (int b = 0; b < C; ++b) py = fmaf(Ar[b], rr[b], py);
            {
                int q = 0;
#pragma unroll
                for (int dh = 0; dh < K; ++dh)
#pragma unroll
                    for (int dw = (dh == 0 ? 2 : 1); dw < K; ++dw)
#pragma unroll
                        for (int b = 0; b < C; ++b) {
                            const int slot = (u - dw + 2 * KM) % KM;      // produced at step s - dw
                            const float v = dh == 0 ? own[b][slot] : up[dh - 1][b][slot];
                            pa[q & 3] = fmaf(-Ar[(dh * K + dw) * C + b], v, pa[q & 3]);
                            ++q;
                        }
            }
#pragma unroll
            for (int d = KM - 1; d >= 1; --d)
#pragma unroll
                for (int b = 0; b < C; ++b) pn = fmaf(-Ar[((d + 1) * K) * C + b], nu[d][b], pn);
            float acc = ((pa[0] + pa[1]) + (pa[2] + pa[3])) + (pn + py);
            // the two taps on the true critical path: left neighbour, then the row above
#pragma unroll
            for (int b = 0; b < C; ++b) acc = fmaf(-Ar[1 * C + b], own[b][(u - 1 + 2 * KM) % KM], acc);
#pragma unroll
            for (int b = 0; b < C; ++b) acc = fmaf(-Ar[K * C + b], nu[0][b], acc);
            img[active ? a * HW + p : dummy_idx] = acc;
            // every lane of the row gets the row's C new values
#pragma unroll
            for (int b = 0; b < C; ++b) {
                own[b][u] = __shfl_sync(0xffffffffu, acc, (r * C + b) & 31);
#pragma unroll
                for (int d = 0; d < KM; ++d) up[d][b][u] = nu[d][b];
            }
            p += sgn;
        }
        if constexpr (MULTI) {
            if (((s0 + KM) % PUB) == 0) {
                __threadfence_block();
                __syncwarp();
                if (lane == 0) progress[j] = s0 + KM;
            }
        }
    }
    if constexpr (MULTI) {
        __threadfence_block();
        __syncwarp();
        if (lane == 0) progress[j] = prod_steps;
    }
    return true;
}

// grad_w partial of one row block, lane = column (Theorem 2 in closed form):
//   part[((dh*K+dw)*C + co)*C + ci] = sum_{h in block, w} gy[co][h][w] * x[ci][h-dh][w-dw]
// written to `dst` (shared memory, NA floats) by the lanes that end up owning each entry.
template <int C, int K>
__device__ __forceinline__ void grad_w_block(const float* gy, const float* xs, int H, int W, int j, int lane, float* dst)
{
    using S = WarpShape<C, K>;
    constexpr int COB = S::COB;
    constexpr int NACC = COB * C * K * K;
    const int HW = H * W;
    const int h0 = 32 * j, h1 = min(H, h0 + 32);
    for (int co0 = 0; co0 < C; co0 += COB) {
        float acc[NACC];
#pragma unroll
        for (int i = 0; i < NACC; ++i) acc[i] = 0.f;
        for (int w0 = 0; w0 < W; w0 += 32) {
            const int w = w0 + lane;
            const bool col_ok = w < W;
            float xr[K][C][K];       // [row slot][ci][dw] = x[ci][row][w-dw]
#pragma unroll
            for (int q = 1; q < K; ++q) {
                const int row = h0 - q;
#pragma unroll
                for (int ci = 0; ci < C; ++ci)
#pragma unroll
                    for (int dw = 0; dw < K; ++dw)
                        xr[(K - q) % K][ci][dw] = (row >= 0 && col_ok && w - dw >= 0) ? xs[ci * HW + row * W + w - dw] : 0.f;
            }
            for (int hb = h0; hb < h1; hb += K) {
#pragma unroll
                for (int r = 0; r < K; ++r) {
                    const int h = hb + r;
                    if (h < h1) {
#pragma unroll
                        for (int ci = 0; ci < C; ++ci)
#pragma unroll
                            for (int dw = 0; dw < K; ++dw)
                                xr[r][ci][dw] = (col_ok && w - dw >= 0) ? xs[ci * HW + h * W + w - dw] : 0.f;
                        float g[COB];
#pragma unroll
                        for (int c = 0; c < COB; ++c) g[c] = col_ok ? gy[(co0 + c) * HW + h * W + w] : 0.f;
#pragma unroll
                        for (int dh = 0; dh < K; ++dh)
#pragma unroll
                            for (int dw = 0; dw < K; ++dw)
#pragma unroll
                                for (int c = 0; c < COB; ++c)
#pragma unroll
                                    for (int ci = 0; ci < C; ++ci)
                                        acc[((dh * K + dw) * COB + c) * C + ci] =
                                            fmaf(g[c], xr[(r - dh + K) % K][ci][dw], acc[((dh * K + dw) * COB + c) * C + ci]);
                    }
                }
            }
        }
        // cross-lane sums, 32 entries at a time
#pragma unroll
        for (int base = 0; base < NACC; base += 32) {
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = (base + i < NACC) ? acc[base + i] : 0.f;
            const float tot = transpose_reduce32(v, lane);
            const int i = base + lane;
            if (i < NACC) {
                const int ci = i % C, c = (i / C) % COB, tap = i / (C * COB);
                dst[(tap * C + co0 + c) * C + ci] = tot;
            }
        }
    }
}

// Float offsets of the kernel's shared-memory regions (all multiples of 32 floats = 128 bytes).
template <int C, int K>
struct WarpSmem {
    using S = WarpShape<C, K>;
    int as_off, bar_off, prog_off, red_off, img_off, imgf, bnd_off, dummy_off, ring_off, total;
    // Hg > 0: the images stay in global memory (H = 0 is passed) and only the boundary rows between the row
    // blocks of one image live here; ring: every warp also owns a ring of 128 columns of its rows.
    __host__ __device__ WarpSmem(int H, int W, int nb, int ipc, bool bwd, int Hg = 0, bool ring = false)
    {
        auto up32 = [](int v) { return (v + 31) & ~31; };
        as_off = 0;
        bar_off = as_off + up32(S::NAP);
        prog_off = bar_off + up32(2 * ipc);
        red_off = prog_off + up32(ipc * nb);
        img_off = red_off + (bwd ? up32(nb * ipc * S::NA) : 0);
        imgf = up32(C * H * W);
        bnd_off = img_off + imgf * ipc * (bwd ? 2 : 1);
        dummy_off = bnd_off + (Hg > 0 ? up32(nb * C * (K - 1) * W + 1) : 0);
        ring_off = dummy_off + 32;
        total = ring_off + (ring ? nb * ipc * C * kRingCh : 0);
    }
};

// bfloat16 images that arrived in the upper half of their fp32 regions, widened in place by the whole CTA.
// Unit u = 8 consecutive values: 16 bytes of bfloat16 at byte 2*CHW + 16u become 32 bytes of fp32 at byte 32u,
// which overwrites the bfloat16 units 2u - CHW/8 and 2u - CHW/8 + 1.  Units are taken in ascending passes of
// blockDim.x, every pass reading all of its units before the barrier and writing after it: what a pass
// overwrites has either been widened by an earlier pass or is read by this one before the barrier.
__device__ __forceinline__ void widen_bf16_in_place(float* regions, int region_floats, int nregions, int CHW)
{
    const int units = CHW >> 3;
    for (int u0 = 0; u0 < units; u0 += (int)blockDim.x) {
        const int u = u0 + (int)threadIdx.x;
        for (int r0 = 0; r0 < nregions; r0 += 4) {
            uint4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                v[q] = make_uint4(0u, 0u, 0u, 0u);
                if (r0 + q < nregions && u < units)
                    v[q] = *reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(regions + (size_t)(r0 + q) * region_floats) +
                                                           2 * (size_t)CHW + 16 * (size_t)u);
            }
            __syncthreads();
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (r0 + q < nregions && u < units) {
                    // a bfloat16 is the upper half of the fp32 with the same value
                    float4* d = reinterpret_cast<float4*>(regions + (size_t)(r0 + q) * region_floats) + 2 * u;
                    d[0] = make_float4(__uint_as_float(v[q].x << 16), __uint_as_float(v[q].x & 0xffff0000u),
                                       __uint_as_float(v[q].y << 16), __uint_as_float(v[q].y & 0xffff0000u));
                    d[1] = make_float4(__uint_as_float(v[q].z << 16), __uint_as_float(v[q].z & 0xffff0000u),
                                       __uint_as_float(v[q].w << 16), __uint_as_float(v[q].w & 0xffff0000u));
                }
            }
        }
    }
    __syncthreads();
}

// The same for one image (and, with `second`, the saved image beside it) by the one warp that owns it: passes of
// 128 units, four per lane, with a warp barrier between a pass's reads and its writes.
__device__ __forceinline__ void widen_bf16_warp(float* region, float* second, int CHW, int lane)
{
    const int units = CHW >> 3;
    for (int u0 = 0; u0 < units; u0 += 128) {
        uint4 v[2][4];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const unsigned char* src = reinterpret_cast<const unsigned char*>(r == 0 ? region : second) + 2 * (size_t)CHW;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int u = u0 + q * 32 + lane;
                v[r][q] = make_uint4(0u, 0u, 0u, 0u);
                if ((r == 0 || second != nullptr) && u < units) v[r][q] = *reinterpret_cast<const uint4*>(src + 16 * (size_t)u);
            }
        }
        __syncwarp();
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float4* dst = reinterpret_cast<float4*>(r == 0 ? region : second);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int u = u0 + q * 32 + lane;
                if ((r == 0 || second != nullptr) && u < units) {
                    dst[2 * u] = make_float4(__uint_as_float(v[r][q].x << 16), __uint_as_float(v[r][q].x & 0xffff0000u),
                                             __uint_as_float(v[r][q].y << 16), __uint_as_float(v[r][q].y & 0xffff0000u));
                    dst[2 * u + 1] = make_float4(__uint_as_float(v[r][q].z << 16), __uint_as_float(v[r][q].z & 0xffff0000u),
                                                 __uint_as_float(v[r][q].w << 16), __uint_as_float(v[r][q].w & 0xffff0000u));
                }
            }
        }
        __syncwarp();
    }
}

__device__ __forceinline__ unsigned pack2_bf16(float lo, float hi)
{
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);     // .x = lo in the low half
    return *reinterpret_cast<const unsigned*>(&t);
}

template <int C, int K, bool BWD, bool MULTI, bool GLB = false, bool RING = false, bool CS = false>
__global__ void __launch_bounds__(256) warp_wavefront_kernel(WarpParams p)
{
    static_assert(!CS || (!GLB && !RING), "the channel-split walk serves images resident in shared memory");
    using S = WarpShape<C, K>;
    extern __shared__ __align__(128) float smem[];
    const int H = p.H, W = p.W, HW = H * W, CHW = C * HW;
    const int nwarps = blockDim.x >> 5;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int li = warp / p.nb, j = warp - li * p.nb;  // image within the CTA, row block within the image
    const int n = blockIdx.x * p.ipc + li;             // image index
    const bool has_img = n < p.B;
    const WarpSmem<C, K> lay(GLB ? 0 : H, W, p.nb, p.ipc, BWD, GLB ? H : 0, RING);

    float* As = smem + lay.as_off;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + lay.bar_off);
    int* progress = reinterpret_cast<int*>(smem + lay.prog_off);               // [ipc][nb]
    float* red = smem + lay.red_off;                                           // [nwarps][NA] (backward)
    float* img = smem + lay.img_off + li * lay.imgf;                           // rhs -> solution, in place
    float* xs_all = smem + lay.img_off + p.ipc * lay.imgf;                     // backward: the saved x images
    float* xs = xs_all + li * lay.imgf;
    float* bnd = smem + lay.bnd_off;                                           // GLB: boundary rows between row blocks
    const float* rin = img;
    const int dummy_idx = GLB ? 0 : (int)((smem + lay.dummy_off) - img);      // scratch slot for lanes outside the image
    if constexpr (GLB) {                                                        // operands stay in global memory
        const size_t base = (size_t)(n < p.B ? n : 0) * CHW;
        img = p.out + base;
        rin = p.rhs + base;
        xs = const_cast<float*>(p.xsaved ? p.xsaved + base : p.rhs + base);
    }

    constexpr bool FUSE_GW = (S::NA <= 81);   // few enough partial sums to ride along in the wavefront's registers
    const bool want_gw = BWD && !RING && !CS && p.grad_w != nullptr;     // ring and channel-split modes never carry grad_w
    const bool leader = has_img && j == 0 && lane == 0;
    // everything above touched no global memory; from here on the predecessor kernel's results are needed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // let the next kernel on the stream be scheduled now; it waits at its own griddepcontrol.wait until this
    // kernel has completed, so only its launch latency overlaps
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // the image's bulk copy goes out first; the kernel transform below overlaps its latency
    const bool narrow = !GLB && p.bf16 != 0;
    if (!GLB && leader && p.bulk) {
        mbar_init(&bars[li], 1);
        fence_mbar_init();
        const unsigned bytes = (unsigned)CHW * (narrow ? 2u : 4u);
        mbar_expect_tx(&bars[li], want_gw ? 2 * bytes : bytes);
        if (narrow) {
            // bfloat16 images land in the upper half of their regions (see widen_bf16_in_place)
            bulk_g2s(img + (CHW >> 1), reinterpret_cast<const __nv_bfloat16*>(p.rhs) + (size_t)n * CHW, bytes, &bars[li]);
            if (want_gw) bulk_g2s(xs + (CHW >> 1), reinterpret_cast<const __nv_bfloat16*>(p.xsaved) + (size_t)n * CHW, bytes, &bars[li]);
        } else {
            bulk_g2s(img, p.rhs + (size_t)n * CHW, bytes, &bars[li]);
            if (want_gw) bulk_g2s(xs, p.xsaved + (size_t)n * CHW, bytes, &bars[li]);
        }
    }
    if (!GLB && has_img && !p.bulk) {
        const float* src = p.rhs + (size_t)n * CHW;
        for (int i = j * 32 + lane; i < CHW; i += p.nb * 32) img[i] = __ldg(src + i);
        if (want_gw) {
            const float* xsrc = p.xsaved + (size_t)n * CHW;
            for (int i = j * 32 + lane; i < CHW; i += p.nb * 32) xs[i] = __ldg(xsrc + i);
        }
    }
    if (threadIdx.x < p.ipc * p.nb) progress[threadIdx.x] = 0;
    if constexpr (!BWD) {
        // the log-det rides in the shadow of the image's arrival: one warp of one CTA, C double-precision logarithms
        if (p.logdet_out != nullptr && blockIdx.x == 0 && warp == 0) warp_logdet(p.w, p.logdet_out, C, HW, K, lane);
    }
    build_transformed_kernel<C, K, BWD>(p.w, As);
    __syncthreads();

    bool ok = true;
    if (has_img) {
        if (!GLB && p.bulk) ok = mbar_wait_bounded(&bars[li], 0);
        ok = __all_sync(0xffffffffu, ok);
    }
    if constexpr (!GLB) {
        if (narrow && p.nb == 1) {
            // one warp per image: it widens its own image as soon as that has arrived
            if (has_img && ok) widen_bf16_warp(img, want_gw ? xs : nullptr, CHW, lane);
        } else if (narrow) {
            // every image of the CTA has to be there before the CTA-wide widening passes; a wait that gave up
            // fails the whole CTA (its images are left unsolved, the status says so)
            for (int l2 = 0; l2 < p.ipc; ++l2)
                if (l2 != li && blockIdx.x * p.ipc + l2 < p.B && !mbar_wait_bounded(&bars[l2], 0)) ok = false;
            ok = __syncthreads_and(ok ? 1 : 0) != 0;
            if (ok) widen_bf16_in_place(smem + lay.img_off, lay.imgf, (want_gw ? 2 : 1) * p.ipc, CHW);
        }
    }
    if constexpr (BWD && !GLB) {
        if (p.mix_in) {
            // load prologue of the transposed solve: the incoming gradient of the 1x1 convolution's output becomes
            // the gradient of x, pixel by pixel and in place: grad_x[c] = s[c] * sum_o V[o][c] * grad_u[o]
            if (has_img && ok) {
                float A[C][C];
#pragma unroll
                for (int c = 0; c < C; ++c)
#pragma unroll
                    for (int o = 0; o < C; ++o) A[c][o] = __ldg(p.mix_s + c) * __ldg(p.mix_V + o * C + c);
                for (int i = j * 32 + lane; i < HW; i += p.nb * 32) {
                    float g[C], r[C];
#pragma unroll
                    for (int o = 0; o < C; ++o) g[o] = img[o * HW + i];
#pragma unroll
                    for (int c = 0; c < C; ++c) {
                        r[c] = 0.f;
#pragma unroll
                        for (int o = 0; o < C; ++o) r[c] = fmaf(A[c][o], g[o], r[c]);
                    }
#pragma unroll
                    for (int c = 0; c < C; ++c) img[c * HW + i] = r[c];
                }
            }
            __syncthreads();
        }
    }
    if (has_img) {
        if (ok) {
            if constexpr (CS)
                ok = wavefront_block_cs<C, K, MULTI>(img, As, H, W, BWD ? HW - 1 : 0, BWD ? -1 : 1, j, progress + li * p.nb,
                                                     lane, dummy_idx);
            else if constexpr (RING)
                ok = wavefront_block<C, K, MULTI, false, GLB, true>(img, As, H, W, BWD ? HW - 1 : 0, BWD ? -1 : 1, j,
                                                                    progress + li * p.nb, lane, nullptr, nullptr, rin, bnd, p.nb,
                                                                    dummy_idx, smem + lay.ring_off + warp * C * kRingCh, p.vec != 0);
            else if (BWD && FUSE_GW && want_gw)
                ok = wavefront_block<C, K, MULTI, BWD && FUSE_GW, GLB>(img, As, H, W, HW - 1, -1, j, progress + li * p.nb,
                                                                       lane, xs, red + warp * S::NA, rin, bnd, p.nb, dummy_idx);
            else
                ok = wavefront_block<C, K, MULTI, false, GLB>(img, As, H, W, BWD ? HW - 1 : 0, BWD ? -1 : 1, j,
                                                              progress + li * p.nb, lane, nullptr, nullptr, rin, bnd, p.nb, dummy_idx);
        }
        if (!ok && lane == 0) raise_status(INVCONV_TIMEOUT);
    }
    __syncthreads();

    if (narrow && has_img) {
        // narrow on the way out: eight values per 16-byte store
        uint4* d16 = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + (size_t)n * CHW);
        const float4* s4 = reinterpret_cast<const float4*>(img);
        for (int u = j * 32 + lane; u < (CHW >> 3); u += p.nb * 32) {
            const float4 a = s4[2 * u], b = s4[2 * u + 1];
            d16[u] = make_uint4(pack2_bf16(a.x, a.y), pack2_bf16(a.z, a.w), pack2_bf16(b.x, b.y), pack2_bf16(b.z, b.w));
        }
    }
    if (!GLB && has_img && !narrow) {
        float* dst = p.out + (size_t)n * CHW;
        if (p.bulk && CHW * 4 <= 16384) {
            // small image: plain 16-byte stores retire without a completion wait at the end of the kernel
            const float4* s4 = reinterpret_cast<const float4*>(img);
            float4* d4 = reinterpret_cast<float4*>(dst);
            for (int i = j * 32 + lane; i < (CHW >> 2); i += p.nb * 32) d4[i] = s4[i];
        } else if (p.bulk) {
            if (leader) {
                fence_proxy_async();
                bulk_s2g(dst, img, (unsigned)CHW * 4u);
                bulk_commit();
            }
        } else {
            for (int i = j * 32 + lane; i < CHW; i += p.nb * 32) dst[i] = img[i];
        }
    }

    if constexpr (!BWD && !GLB) {
        if (p.mix_out != nullptr && has_img) {
            // store epilogue of the forward solve: Actnorm and the 1x1 convolution act on one pixel at a time, so
            // u = V (s * x + b) is formed from the solved image while it is still in shared memory
            float A[C][C], cb[C];
#pragma unroll
            for (int o = 0; o < C; ++o) {
                cb[o] = 0.f;
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    const float v = __ldg(p.mix_V + o * C + c);
                    A[o][c] = v * __ldg(p.mix_s + c);
                    cb[o] = fmaf(v, __ldg(p.mix_b + c), cb[o]);
                }
            }
            float* dst2 = p.mix_out + (size_t)n * CHW;
            for (int i = j * 32 + lane; i < HW; i += p.nb * 32) {
                float xin[C];
#pragma unroll
                for (int c = 0; c < C; ++c) xin[c] = img[c * HW + i];
#pragma unroll
                for (int o = 0; o < C; ++o) {
                    float u = cb[o];
#pragma unroll
                    for (int c = 0; c < C; ++c) u = fmaf(A[o][c], xin[c], u);
                    dst2[o * HW + i] = u;
                }
            }
        }
    }

    if constexpr (BWD) {
        if (want_gw) {
            float* mine = red + warp * S::NA;
            if (!has_img || !ok) { for (int i = lane; i < S::NA; i += 32) mine[i] = 0.f; }
            else if (!FUSE_GW) grad_w_block<C, K>(img, xs, H, W, j, lane, mine);
            __syncthreads();
            float* cta_part = p.partials + (size_t)blockIdx.x * S::NA;
            for (int i = threadIdx.x; i < S::NA; i += blockDim.x) {
                float s = 0.f;
                for (int wq = 0; wq < nwarps; ++wq) s += red[wq * S::NA + i];
                __stcg(cta_part + i, s);
            }
            __threadfence();
            __syncthreads();
            __shared__ unsigned ticket;
            if (threadIdx.x == 0) ticket = atomicAdd(p.counter, 1u);
            __syncthreads();
            if (ticket == gridDim.x - 1) {
                // last CTA: sum the CTA partials in CTA order.  They are staged through the (now idle) shared
                // memory of the saved-x images so that all threads have loads in flight at once.
                __threadfence();
                const int G = (int)gridDim.x;
                const int chunk = GLB ? 0 : min(G, (p.ipc * lay.imgf) / S::NA);
                for (int b0 = 0; chunk > 0 && b0 < G; b0 += chunk) {
                    const int nbk = min(chunk, G - b0);
                    const float* part = p.partials + (size_t)b0 * S::NA;
                    const int tot = nbk * S::NA, nt = (int)blockDim.x;
                    for (int i0 = threadIdx.x; i0 < tot; i0 += nt * 8) {       // eight loads in flight per thread
                        float tv[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) tv[q] = (i0 + q * nt < tot) ? __ldcg(part + i0 + q * nt) : 0.f;
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            if (i0 + q * nt < tot) xs_all[i0 + q * nt] = tv[q];
                    }
                    __syncthreads();
                    for (int i = threadIdx.x; i < S::NA; i += blockDim.x) {
                        float s = b0 == 0 ? 0.f : red[i];
                        for (int b = 0; b < nbk; ++b) s += xs_all[b * S::NA + i];
                        red[i] = s;
                    }
                    __syncthreads();
                }
                for (int i = threadIdx.x; i < S::NA; i += blockDim.x) {
                    float s = 0.f;
                    if (chunk > 0) s = red[i];
                    else for (int b = 0; b < G; ++b) s += __ldcg(p.partials + (size_t)b * S::NA + i);
                    const int ci = i % C, co = (i / C) % C, tap = i / (C * C);
                    const int dh = tap / K, dw = tap % K;
                    p.grad_w[((co * C + ci) * K + (K - 1 - dh)) * K + (K - 1 - dw)] = finish_grad_w(s, co, ci, tap, C, K, p.ld);
                }
                if (threadIdx.x == 0) *p.counter = 0u;
            }
        }
    }
    if (!GLB && p.bulk && leader && CHW * 4 > 16384 && !narrow) bulk_wait_read0();
}

// Dynamic shared memory the kernel needs for a launch shape.
template <int C, int K>
inline size_t warp_kernel_smem(int H, int W, int nb, int ipc, bool bwd, bool glb = false, bool ring = false)
{
    if (glb) return sizeof(float) * (size_t)WarpSmem<C, K>(0, W, nb, ipc, bwd, H, ring).total;
    return sizeof(float) * (size_t)WarpSmem<C, K>(H, W, nb, ipc, bwd).total;
}

}  // namespace invconv

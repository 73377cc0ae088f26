// Wide-channel wavefront: one CTA -- or one thread-block cluster -- per image.
//
// With many channels the per-diagonal update is a contraction
//     u[p][a] = sum_b A0[a][b] rhs[p][b] - sum_{delta != 0, b} A_delta[a][b] u[p - delta][b]
// of length C*k^2 for each of (pixels on the diagonal) x C outputs, and the fp32
// FMA pipe is the bound (Section 3.3: k^2 work per diagonal, here times C^2).
// The transformed kernel A (see team_prep_kernel) is the stationary operand: it
// is distributed once over the REGISTERS of the CTA -- thread (slice s, lane l)
// keeps the entries for its share of the contraction range (a few groups of
// four input channels of one tap) and its TA output channels -- and stays
// there for every image the CTA processes.  Solved pixels live in shared
// memory as [pixel][channel], so the four input channels of a group arrive
// as one broadcast 16-byte load feeding 4*TA FMAs.
//
// When C*C*k^2 floats outgrow one SM's register file the output channels are
// split over the CTAs of a cluster: each CTA finishes its C/R channels of the
// diagonal's pixels and stores them into every peer's shared-memory image
// (distributed shared memory), then one cluster barrier closes the step.
// Every CTA therefore always reads only its own shared memory.
//
// The transposed solve (grad_y = M^-T grad_x, Theorem 1) runs the same kernel:
// the image is rotated by 180 degrees while it is loaded and stored, and
// team_prep_kernel supplies L^-T W_delta^T.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace invconv {
namespace cg = cooperative_groups;

// ---------------------------------------------------------------------------
// Transformed kernel, one CTA per tap:  A[tap][b][a], tap = dh*K + dw,
//   forward : tap 0 -> L^-1[a][b];   tap != 0 -> sum_m L^-1[a][m] w[m][b][K-1-dh][K-1-dw]
//   backward: tap 0 -> L^-1[b][a];   tap != 0 -> sum_m L^-1[m][a] w[b][m][K-1-dh][K-1-dw]
// L = w[:, :, K-1, K-1] restricted to ci <= co.  L^-1 is built by blocked
// recursion: 12x12 diagonal blocks by column-parallel substitution, then pairs
// of blocks are merged,  [[X11, 0], [-X22 L21 X11, X22]],  doubling the block
// size each level, so the depth is logarithmic in C.
// Shared memory: three C x C matrices (rows padded to 16 bytes).
// ---------------------------------------------------------------------------
template <bool BWD>
__global__ void __launch_bounds__(512) team_prep_kernel(const float* __restrict__ w, float* __restrict__ A, int C, int K)
{
    extern __shared__ __align__(16) float sm[];
    const int CP = (C + 3) & ~3;  // row pitch (16-byte rows)
    float* Lm = sm;               // [C][CP] masked centre tap; later the tap's kernel slice T
    float* Li = sm + C * CP;      // [C][CP] inverse, row-major
    float* Sc = sm + 2 * C * CP;  // [C][CP] scratch of the merge steps; later the inverse transposed
    const int KK = K * K, ctr = KK - 1;
    const int tid = threadIdx.x, NT = blockDim.x;
    const int tap = blockIdx.x;
    const int dh = tap / K, dw = tap % K;
    const int t = (K - 1 - dh) * K + (K - 1 - dw);

    for (int i = tid / 32; i < C; i += NT / 32)
        for (int j = tid % 32; j < CP; j += 32) {
            Lm[i * CP + j] = (j <= i && j < C) ? __ldg(w + (size_t)(i * C + j) * KK + ctr) : 0.f;
            Li[i * CP + j] = 0.f;
        }
    __syncthreads();
    constexpr int NB0 = 12;
    for (int col = tid; col < C; col += NT) {       // diagonal blocks, one thread per column
        const int o = col / NB0 * NB0, e1 = min(C, o + NB0);
        Li[col * CP + col] = 1.0f / Lm[col * CP + col];
        for (int i = col + 1; i < e1; ++i) {
            float s = 0.f;
            for (int m = col; m < i; ++m) s = fmaf(Lm[i * CP + m], Li[m * CP + col], s);
            Li[i * CP + col] = -s / Lm[i * CP + i];
        }
    }
    __syncthreads();
    for (int sz = NB0; sz < C; sz *= 2) {
        // every pair of neighbouring blocks (o, o+sz): X21 = -X22 * (L21 * X11)
        const int npairs = (C + 2 * sz - 1) / (2 * sz);
        const int per = sz * sz;
        for (int idx = tid; idx < npairs * per; idx += NT) {
            const int pr = idx / per, rem = idx - pr * per;
            const int ii = rem / sz, jj = rem - ii * sz;
            const int o = pr * 2 * sz, i = o + sz + ii, j = o + jj;
            if (i < C) {
                float s = 0.f;
                for (int m = j; m < o + sz; ++m) s = fmaf(Lm[i * CP + m], Li[m * CP + j], s);
                Sc[i * CP + j] = s;
            }
        }
        __syncthreads();
        for (int idx = tid; idx < npairs * per; idx += NT) {
            const int pr = idx / per, rem = idx - pr * per;
            const int ii = rem / sz, jj = rem - ii * sz;
            const int o = pr * 2 * sz, i = o + sz + ii, j = o + jj;
            if (i < C) {
                float s = 0.f;
                for (int m = o + sz; m <= i; ++m) s = fmaf(Li[i * CP + m], Sc[m * CP + j], s);
                Li[i * CP + j] = -s;
            }
        }
        __syncthreads();
    }
    float* out = A + (size_t)tap * C * C;
    if (tap == 0) {
        for (int e = tid; e < C * C; e += NT) {
            const int b = e / C, a = e - b * C;
            out[e] = BWD ? Li[b * CP + a] : Li[a * CP + b];
        }
        return;
    }
    // T[m][b] = w[m][b][tap]  (over Lm, which is no longer needed); the forward product wants L^-1 transposed
    for (int i = tid / 32; i < C; i += NT / 32)
        for (int j = tid % 32; j < CP; j += 32) {
            Lm[i * CP + j] = j < C ? __ldg(w + (size_t)(i * C + j) * KK + t) : 0.f;
            if (!BWD && j < C) Sc[j * CP + i] = Li[i * CP + j];
        }
    __syncthreads();
    const float* T = Lm;
    const int nq = CP / 4;
    // thread -> (output channel a, quad of input channels b): conflict-free column reads, broadcast quads
    for (int task = tid; task < C * nq; task += NT) {
        const int bq = task / C, a = task - bq * C;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!BWD) {
            // A[b][a] = sum_{m <= a} Li[a][m] * T[m][b]
            for (int m = 0; m <= a; ++m) {
                const float l = Sc[m * CP + a];
                const float4 tv = *reinterpret_cast<const float4*>(T + m * CP + bq * 4);
                acc.x = fmaf(l, tv.x, acc.x); acc.y = fmaf(l, tv.y, acc.y);
                acc.z = fmaf(l, tv.z, acc.z); acc.w = fmaf(l, tv.w, acc.w);
            }
        } else {
            // A[b][a] = sum_{m >= a} Li[m][a] * T[b][m]
            for (int m = a; m < C; ++m) {
                const float l = Li[m * CP + a];
                acc.x = fmaf(l, T[(bq * 4 + 0) * CP + m], acc.x);
                acc.y = fmaf(l, (bq * 4 + 1 < C) ? T[(bq * 4 + 1) * CP + m] : 0.f, acc.y);
                acc.z = fmaf(l, (bq * 4 + 2 < C) ? T[(bq * 4 + 2) * CP + m] : 0.f, acc.z);
                acc.w = fmaf(l, (bq * 4 + 3 < C) ? T[(bq * 4 + 3) * CP + m] : 0.f, acc.w);
            }
        }
        const float v[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (bq * 4 + q < C) out[(size_t)(bq * 4 + q) * C + a] = v[q];
    }
}

inline size_t team_prep_smem(int C) { return sizeof(float) * 3 * (size_t)C * ((C + 3) & ~3); }

// ---------------------------------------------------------------------------
struct TeamParams {
    const float* rhs;   // y (forward) or grad_x (backward), [B][C][H][W]
    const float* A;     // transformed kernel [K*K][C(b)][C(a)]
    float* out;         // x or grad_y
    int B, C, H, W, K;
    int R;              // CTAs per image (cluster size)
    int CA;             // output channels per CTA (C / R)
    int LG;             // lanes per slice (power of two), LG*TA >= CA
    int NS;             // slices per pixel group (multiple of 32/LG)
    int NPG;            // pixel groups per CTA
    int CS;             // channel stride of the shared-memory images (multiple of 4)
    int PMAXS;          // pixel slots of one pixel group on the longest diagonal (multiple of 4)
    int rot;            // 1: walk the image rotated by 180 degrees (transposed solve)
    int ncl;            // clusters in the grid
};

// Thread (pixel group pg, slice s, lane l) owns NG groups of four input channels
// of one tap each and TA output channels.  Per diagonal it walks its pixels four
// at a time: one broadcast 16-byte load per pixel and group, 16*TA FMAs.  The
// slices' partial sums meet in shared memory; after one block barrier every
// (pixel, channel) of the diagonal is summed over the slices and stored into
// the image of every CTA of the cluster.
template <int TA, int NG>
__global__ void __launch_bounds__(256) team_wavefront_kernel(TeamParams p)
{
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) float smem[];
    const int C = p.C, H = p.H, W = p.W, K = p.K, CS = p.CS, R = p.R, CA = p.CA;
    const int HP = H + K - 1, WP = W + K - 1, HW = H * W;
    const int IMG = HP * WP * CS;
    float* U = smem;
    float* RH = smem + IMG;
    float* red = smem + 2 * IMG;
    const int r = R > 1 ? (int)cluster.block_rank() : 0;
    const int cl = blockIdx.x / R;
    const int tid = threadIdx.x, NT = blockDim.x;
    const int LG = p.LG, NS = p.NS, per_pg = NS * LG;
    const int pg = tid / per_pg, tq = tid - pg * per_pg;
    const int s = tq / LG, l = tq - s * LG;
    const int CAp = LG * TA;
    const int CB4 = CS >> 2;
    const int GT = K * K * CB4;

    // this thread's share of the transformed kernel, signs folded in
    float wt[NG][4][TA];
    int off[NG];
#pragma unroll
    for (int i = 0; i < NG; ++i) {
        const int g = s + i * NS;
        off[i] = 0;
        if (g < GT) {
            const int tap = g / CB4, b4 = g - tap * CB4;
            const int dh = tap / K, dw = tap - dh * K;
            off[i] = (tap == 0 ? IMG : 0) - (dh * WP + dw) * CS + b4 * 4;
        }
#pragma unroll
        for (int bb = 0; bb < 4; ++bb)
#pragma unroll
            for (int t = 0; t < TA; ++t) {
                float v = 0.f;
                if (g < GT) {
                    const int tap = g / CB4, b = (g - tap * CB4) * 4 + bb, al = l * TA + t;
                    if (b < C && al < CA) v = __ldg(p.A + ((size_t)tap * C + b) * C + r * CA + al);
                    if (tap != 0) v = -v;
                }
                wt[i][bb][t] = v;
            }
    }
    float* Urem[8];
#pragma unroll
    for (int rr = 0; rr < 8; ++rr) Urem[rr] = (R > 1 && rr < R) ? cluster.map_shared_rank(U, rr) : U;

    for (int i = tid; i < 2 * IMG; i += NT) smem[i] = 0.f;     // zero padding (and the channel padding) once
    __syncthreads();

    // finalize items of this thread walk (pixel, channel) pairs in steps of NT without divisions
    const int fin_i0 = tid / CA, fin_a0 = tid - fin_i0 * CA;
    const int fin_di = NT / CA, fin_da = NT - fin_di * CA;

    const int ND = H + W - 1;
    for (int n = cl; n < p.B; n += p.ncl) {
        // right-hand side of this image, all channels, rotated for the transposed solve
        const float* src = p.rhs + (size_t)n * C * HW;
        for (int c = tid / 32; c < C; c += NT / 32) {
            for (int pp = tid % 32; pp < HW; pp += 32) {
                int h = pp / W, w = pp - h * W;
                if (p.rot) { h = H - 1 - h; w = W - 1 - w; }
                RH[((h + K - 1) * WP + (w + K - 1)) * CS + c] = __ldg(src + c * HW + pp);
            }
        }
        if (R > 1) cluster.sync(); else __syncthreads();

        for (int d = 0; d < ND; ++d) {
            const int hlo = max(0, d - (W - 1));
            const int npix = min(H - 1, d) - hlo + 1;
            for (int q0 = 0; pg + p.NPG * q0 < npix; q0 += 4) {
                const float* up[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    int i = pg + p.NPG * (q0 + x);
                    if (i >= npix) i = pg;                    // padding slot: recompute a valid pixel, result unused
                    const int h = hlo + i;
                    up[x] = U + ((h + K - 1) * WP + (d - h) + K - 1) * CS;
                }
                float acc[4][TA];
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int t = 0; t < TA; ++t) acc[x][t] = 0.f;
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    float4 u[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) u[x] = *reinterpret_cast<const float4*>(up[x] + off[g]);
#pragma unroll
                    for (int x = 0; x < 4; ++x)
#pragma unroll
                        for (int t = 0; t < TA; ++t) {
                            acc[x][t] = fmaf(wt[g][0][t], u[x].x, acc[x][t]);
                            acc[x][t] = fmaf(wt[g][1][t], u[x].y, acc[x][t]);
                            acc[x][t] = fmaf(wt[g][2][t], u[x].z, acc[x][t]);
                            acc[x][t] = fmaf(wt[g][3][t], u[x].w, acc[x][t]);
                        }
                }
                float* dst = red + ((size_t)((pg * p.PMAXS + q0) * NS + s)) * CAp + l * TA;
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int t = 0; t < TA; ++t) dst[x * NS * CAp + t] = acc[x][t];
            }
            __syncthreads();
            // finish the diagonal: sum the slices' partial sums, publish to every CTA of the cluster
            for (int i = fin_i0, al = fin_a0; i < npix; ) {
                const int pgi = i % p.NPG, q = i / p.NPG;
                const float* src2 = red + ((size_t)((pgi * p.PMAXS + q) * NS)) * CAp + al;
                float v0 = 0.f, v1 = 0.f;
                int ss = 0;
                for (; ss + 1 < NS; ss += 2) { v0 += src2[ss * CAp]; v1 += src2[(ss + 1) * CAp]; }
                if (ss < NS) v0 += src2[ss * CAp];
                const float v = v0 + v1;
                const int h = hlo + i;
                const int o = ((h + K - 1) * WP + (d - h) + K - 1) * CS + r * CA + al;
                if (R > 1) {
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr)
                        if (rr < R) Urem[rr][o] = v;
                } else {
                    U[o] = v;
                }
                i += fin_di; al += fin_da;
                if (al >= CA) { al -= CA; ++i; }
            }
            if (R > 1) cluster.sync(); else __syncthreads();
        }
        // write back this CTA's channels
        float* dst = p.out + (size_t)n * C * HW + (size_t)r * CA * HW;
        for (int al = tid / 32; al < CA; al += NT / 32) {
            for (int pp = tid % 32; pp < HW; pp += 32) {
                int h = pp / W, w = pp - h * W;
                if (p.rot) { h = H - 1 - h; w = W - 1 - w; }
                dst[al * HW + pp] = U[((h + K - 1) * WP + (w + K - 1)) * CS + r * CA + al];
            }
        }
        if (R > 1) cluster.sync(); else __syncthreads();
    }
}

// ---------------------------------------------------------------------------
// Host-side launch plan.
// ---------------------------------------------------------------------------
struct TeamPlan {
    bool ok = false;
    int R = 1, CA = 0, TA = 3, LG = 0, NS = 0, NPG = 1, CS = 0, PMAXS = 0, NG = 0;
    int threads = 0, ncl = 0;
    size_t smem = 0;
};

inline TeamPlan plan_team(int B, int C, int H, int W, int K, size_t max_smem, int sm_count)
{
    TeamPlan best;
    if (C < 1 || K < 1) return best;
    // cluster size: enough CTAs that the kernel's share fits one CTA's registers, then fill the SMs
    int R = 1;
    auto divisible = [&](int rr) { return C % rr == 0 && (C / rr) >= 3; };
    while (R < 8 && (long long)C * C * K * K / R > 30000 && divisible(R * 2)) R *= 2;
    if ((long long)C * C * K * K / R > 30000) return best;
    while (R < 8 && (long long)B * R * 2 <= sm_count && divisible(R * 2)) R *= 2;
    const int CA = C / R;
    const int CS = (C + 3) & ~3;
    const int GT = K * K * (CS / 4);
    const int maxdiag = H < W ? H : W;
    const size_t img = (size_t)(H + K - 1) * (W + K - 1) * CS;
    // candidates (TA, NG), cheapest register footprint first within each TA; prefer wide TA (more FMAs per load)
    const int ta_opts[3] = {6, 3, 4};
    const int ng_opts[4] = {2, 4, 7, 10};
    for (int ti = 0; ti < 3 && !best.ok; ++ti) {
        const int TA = ta_opts[ti];
        if (TA == 6 && CA % 6 != 0) continue;
        if (TA == 3 && CA % 3 != 0) continue;
        int LG = 1;
        while (LG * TA < CA) LG *= 2;
        if (LG > 32) continue;
        const int SPW = 32 / LG;
        for (int ni = 0; ni < 4; ++ni) {
            const int NG = ng_opts[ni];
            if (NG * 4 * TA > 170) continue;                 // weights + accumulators must fit the register file
            int NS = (GT + NG - 1) / NG;
            NS = (NS + SPW - 1) / SPW * SPW;
            if (NS * LG > 256) continue;
            TeamPlan pl;
            pl.R = R; pl.CA = CA; pl.TA = TA; pl.LG = LG; pl.NS = NS; pl.CS = CS; pl.NG = NG;
            int NPG = 256 / (NS * LG);
            const int want = (maxdiag + 3) / 4;               // no more pixel groups than batches of four pixels
            if (NPG > want) NPG = want;
            if (NPG < 1) NPG = 1;
            pl.NPG = NPG;
            pl.threads = NPG * NS * LG;
            pl.PMAXS = (((maxdiag + NPG - 1) / NPG) + 3) & ~3;
            const size_t red = (size_t)NPG * pl.PMAXS * NS * LG * TA;
            pl.smem = sizeof(float) * (2 * img + red);
            if (pl.smem > max_smem) continue;
            int ncl = sm_count / R;
            if (B * 2 > ncl * 3) ncl = (2 * sm_count) / R;   // many images: two resident clusters per SM hide barrier latency
            if (ncl > B) ncl = B;
            if (ncl < 1) ncl = 1;
            pl.ncl = ncl;
            pl.ok = true;
            best = pl;
            break;
        }
    }
    return best;
}

}  // namespace invconv

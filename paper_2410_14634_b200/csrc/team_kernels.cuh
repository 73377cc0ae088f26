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
// Shared memory: 3*C*C floats.
// ---------------------------------------------------------------------------
template <bool BWD>
__global__ void __launch_bounds__(256) team_prep_kernel(const float* __restrict__ w, float* __restrict__ A, int C, int K)
{
    extern __shared__ float sm[];
    float* Lm = sm;               // [C][C] masked centre tap
    float* Li = sm + C * C;       // [C][C] its inverse
    float* T = sm + 2 * C * C;    // scratch of the inversion, then the tap's kernel slice
    const int KK = K * K, ctr = KK - 1;
    const int tid = threadIdx.x, NT = blockDim.x;
    const int tap = blockIdx.x;
    const int dh = tap / K, dw = tap % K;
    const int t = (K - 1 - dh) * K + (K - 1 - dw);

    for (int e = tid; e < C * C; e += NT) {
        const int i = e / C, j = e % C;
        Lm[e] = (j <= i) ? __ldg(w + (size_t)e * KK + ctr) : 0.f;
        Li[e] = 0.f;
    }
    __syncthreads();
    constexpr int NB0 = 12;
    // diagonal blocks: thread -> (block, column)
    for (int col = tid; col < C; col += NT) {
        const int o = col / NB0 * NB0, e1 = min(C, o + NB0);
        Li[col * C + col] = 1.0f / Lm[col * C + col];
        for (int i = col + 1; i < e1; ++i) {
            float s = 0.f;
            for (int m = col; m < i; ++m) s += Lm[i * C + m] * Li[m * C + col];
            Li[i * C + col] = -s / Lm[i * C + i];
        }
    }
    __syncthreads();
    for (int sz = NB0; sz < C; sz *= 2) {
        // pairs (o, o+sz): rows [o+sz, min(o+2sz, C)), cols [o, o+sz)
        // step 1: Tm = L21 * X11        (Tm stored at the X21 position of a scratch C x C matrix)
        float* Tm = T;
        for (int e = tid; e < C * C; e += NT) {
            const int i = e / C, j = e % C;
            const int o = i / (2 * sz) * (2 * sz);
            if (i >= o + sz && j >= o && j < o + sz) {
                float s = 0.f;
                for (int m = j; m < o + sz; ++m) s += Lm[i * C + m] * Li[m * C + j];
                Tm[e] = s;
            }
        }
        __syncthreads();
        // step 2: X21 = -X22 * Tm
        for (int e = tid; e < C * C; e += NT) {
            const int i = e / C, j = e % C;
            const int o = i / (2 * sz) * (2 * sz);
            if (i >= o + sz && j >= o && j < o + sz) {
                float s = 0.f;
                for (int m = o + sz; m <= i; ++m) s += Li[i * C + m] * Tm[m * C + j];
                Li[e] = -s;
            }
        }
        __syncthreads();
    }
    if (tap != 0) {
        for (int e = tid; e < C * C; e += NT) T[e] = __ldg(w + (size_t)e * KK + t);     // T[m][b] = w[m][b][tap]
        __syncthreads();
    }
    float* out = A + (size_t)tap * C * C;
    for (int e = tid; e < C * C; e += NT) {
        const int b = e / C, a = e % C;
        float v = 0.f;
        if (tap == 0) {
            v = BWD ? Li[b * C + a] : Li[a * C + b];
        } else if (!BWD) {
            for (int m = 0; m <= a; ++m) v += Li[a * C + m] * T[m * C + b];
        } else {
            for (int m = a; m < C; ++m) v += Li[m * C + a] * T[b * C + m];
        }
        out[e] = v;
    }
}

inline size_t team_prep_smem(int C) { return sizeof(float) * 3 * (size_t)C * C; }

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
    int PMAXS;          // pixels one pixel group handles on the longest diagonal
    int rot;            // 1: walk the image rotated by 180 degrees (transposed solve)
    int ncl;            // clusters in the grid
};

template <int TA, int NGN, int NGC>
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
    const int r = (int)cluster.block_rank();
    const int cl = blockIdx.x / R;
    const int tid = threadIdx.x, NT = blockDim.x;
    const int LG = p.LG, per_pg = p.NS * LG, NWP = per_pg >> 5;
    const int pg = tid / per_pg, tq = tid - pg * per_pg;
    const int s = tq / LG, l = tq - s * LG;
    const int wq = tq >> 5;
    const int CAp = LG * TA;
    const int CB4 = CS >> 2;
    const int GN = (K > 1 ? K * K - 2 : 1) * CB4, GC = (K > 1 ? 2 : 0) * CB4;

    // this thread's share of the transformed kernel, signs folded in
    float wn[NGN][4][TA], wc[NGC][4][TA];
    int offn[NGN], offc[NGC];
    auto fetch = [&](int tap, int b4, float (&dst)[4][TA], int& off) {
        const int dh = tap / K, dw = tap - dh * K;
        off = (tap == 0 ? IMG : 0) - (dh * WP + dw) * CS + b4 * 4;
#pragma unroll
        for (int bb = 0; bb < 4; ++bb)
#pragma unroll
            for (int t = 0; t < TA; ++t) {
                const int b = b4 * 4 + bb, al = l * TA + t;
                float v = 0.f;
                if (b < C && al < CA) v = __ldg(p.A + ((size_t)tap * C + b) * C + r * CA + al);
                dst[bb][t] = tap == 0 ? v : -v;
            }
    };
#pragma unroll
    for (int i = 0; i < NGN; ++i) {
        const int g = s + i * p.NS;
        if (g < GN) {
            const int tnc = g / CB4, b4 = g - tnc * CB4;
            const int tap = tnc == 0 ? 0 : (tnc <= K - 2 ? tnc + 1 : tnc + 2);   // skips taps 1 and K
            fetch(tap, b4, wn[i], offn[i]);
        } else {
            offn[i] = 0;
#pragma unroll
            for (int bb = 0; bb < 4; ++bb)
#pragma unroll
                for (int t = 0; t < TA; ++t) wn[i][bb][t] = 0.f;
        }
    }
#pragma unroll
    for (int i = 0; i < NGC; ++i) {
        const int g = s + i * p.NS;
        if (g < GC) {
            const int tcr = g / CB4, b4 = g - tcr * CB4;
            fetch(tcr == 0 ? 1 : K, b4, wc[i], offc[i]);
        } else {
            offc[i] = 0;
#pragma unroll
            for (int bb = 0; bb < 4; ++bb)
#pragma unroll
                for (int t = 0; t < TA; ++t) wc[i][bb][t] = 0.f;
        }
    }
    float* Urem[8];
#pragma unroll
    for (int rr = 0; rr < 8; ++rr) Urem[rr] = rr < R ? cluster.map_shared_rank(U, rr) : U;

    for (int i = tid; i < 2 * IMG; i += NT) smem[i] = 0.f;     // zero padding (and the channel padding) once
    __syncthreads();

    const int ND = H + W - 1;
    for (int n = cl; n < p.B; n += p.ncl) {
        // right-hand side of this image, all channels, rotated for the transposed solve
        const float* src = p.rhs + (size_t)n * C * HW;
        for (int idx = tid; idx < C * HW; idx += NT) {
            const int c = idx / HW, pp = idx - c * HW;
            int h = pp / W, w = pp - h * W;
            if (p.rot) { h = H - 1 - h; w = W - 1 - w; }
            RH[((h + K - 1) * WP + (w + K - 1)) * CS + c] = __ldg(src + idx);
        }
        cluster.sync();

        for (int d = 0; d < ND; ++d) {
            const int hlo = max(0, d - (W - 1));
            const int npix = min(H - 1, d) - hlo + 1;
            for (int q = 0; pg + p.NPG * q < npix; q += 2) {
                const int i1 = pg + p.NPG * q, i2 = i1 + p.NPG;
                const bool has2 = i2 < npix;
                const int h1 = hlo + i1, h2 = has2 ? hlo + i2 : h1;
                const float* u1 = U + ((h1 + K - 1) * WP + (d - h1) + K - 1) * CS;
                const float* u2 = U + ((h2 + K - 1) * WP + (d - h2) + K - 1) * CS;
                float acc1[TA], acc2[TA];
#pragma unroll
                for (int t = 0; t < TA; ++t) { acc1[t] = 0.f; acc2[t] = 0.f; }
#pragma unroll
                for (int g = 0; g < NGN; ++g) {
                    const float4 x1 = *reinterpret_cast<const float4*>(u1 + offn[g]);
                    const float4 x2 = *reinterpret_cast<const float4*>(u2 + offn[g]);
#pragma unroll
                    for (int t = 0; t < TA; ++t) {
                        acc1[t] = fmaf(wn[g][0][t], x1.x, acc1[t]); acc2[t] = fmaf(wn[g][0][t], x2.x, acc2[t]);
                        acc1[t] = fmaf(wn[g][1][t], x1.y, acc1[t]); acc2[t] = fmaf(wn[g][1][t], x2.y, acc2[t]);
                        acc1[t] = fmaf(wn[g][2][t], x1.z, acc1[t]); acc2[t] = fmaf(wn[g][2][t], x2.z, acc2[t]);
                        acc1[t] = fmaf(wn[g][3][t], x1.w, acc1[t]); acc2[t] = fmaf(wn[g][3][t], x2.w, acc2[t]);
                    }
                }
#pragma unroll
                for (int g = 0; g < NGC; ++g) {
                    const float4 x1 = *reinterpret_cast<const float4*>(u1 + offc[g]);
                    const float4 x2 = *reinterpret_cast<const float4*>(u2 + offc[g]);
#pragma unroll
                    for (int t = 0; t < TA; ++t) {
                        acc1[t] = fmaf(wc[g][0][t], x1.x, acc1[t]); acc2[t] = fmaf(wc[g][0][t], x2.x, acc2[t]);
                        acc1[t] = fmaf(wc[g][1][t], x1.y, acc1[t]); acc2[t] = fmaf(wc[g][1][t], x2.y, acc2[t]);
                        acc1[t] = fmaf(wc[g][2][t], x1.z, acc1[t]); acc2[t] = fmaf(wc[g][2][t], x2.z, acc2[t]);
                        acc1[t] = fmaf(wc[g][3][t], x1.w, acc1[t]); acc2[t] = fmaf(wc[g][3][t], x2.w, acc2[t]);
                    }
                }
                // sum over the slices that share this warp
                for (int o = LG; o < 32; o <<= 1) {
#pragma unroll
                    for (int t = 0; t < TA; ++t) {
                        acc1[t] += __shfl_xor_sync(0xffffffffu, acc1[t], o);
                        acc2[t] += __shfl_xor_sync(0xffffffffu, acc2[t], o);
                    }
                }
                if ((tq & 31) < LG) {
                    float* d1 = red + ((pg * NWP + wq) * p.PMAXS + q) * CAp + l * TA;
#pragma unroll
                    for (int t = 0; t < TA; ++t) d1[t] = acc1[t];
                    if (has2) {
#pragma unroll
                        for (int t = 0; t < TA; ++t) d1[CAp + t] = acc2[t];
                    }
                }
            }
            __syncthreads();
            // finish the diagonal: sum the warps' partial sums, publish to every CTA of the cluster
            for (int idx = tid; idx < npix * CA; idx += NT) {
                const int i = idx / CA, al = idx - i * CA;
                const int pgi = i % p.NPG, q = i / p.NPG;
                const float* src2 = red + ((pgi * NWP) * p.PMAXS + q) * CAp + al;
                float v = 0.f;
                for (int ww = 0; ww < NWP; ++ww) v += src2[ww * p.PMAXS * CAp];
                const int h = hlo + i;
                const int off = ((h + K - 1) * WP + (d - h) + K - 1) * CS + r * CA + al;
#pragma unroll
                for (int rr = 0; rr < 8; ++rr)
                    if (rr < R) Urem[rr][off] = v;
            }
            cluster.sync();
        }
        // write back this CTA's channels
        float* dst = p.out + (size_t)n * C * HW + (size_t)r * CA * HW;
        for (int idx = tid; idx < CA * HW; idx += NT) {
            const int al = idx / HW, pp = idx - al * HW;
            int h = pp / W, w = pp - h * W;
            if (p.rot) { h = H - 1 - h; w = W - 1 - w; }
            dst[idx] = U[((h + K - 1) * WP + (w + K - 1)) * CS + r * CA + al];
        }
        cluster.sync();
    }
}

// ---------------------------------------------------------------------------
// Host-side launch plan.
// ---------------------------------------------------------------------------
struct TeamPlan {
    bool ok = false;
    int R = 1, CA = 0, TA = 3, LG = 0, NS = 0, NPG = 1, CS = 0, PMAXS = 0, NGN = 0, NGC = 0;
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
    const int TA = (CA % 3 == 0) ? 3 : 4;
    int LG = 1;
    while (LG * TA < CA) LG *= 2;
    if (LG > 32) return best;
    const int SPW = 32 / LG;
    const int CS = (C + 3) & ~3;
    const int CB4 = CS / 4;
    const int GN = (K > 1 ? K * K - 2 : 1) * CB4, GC = (K > 1 ? 2 : 0) * CB4;
    const int menu[3][2] = {{3, 1}, {6, 2}, {9, 1}};
    for (int m = 0; m < 3; ++m) {
        const int NGN = menu[m][0], NGC = menu[m][1];
        int NS = (GN + NGN - 1) / NGN;
        if (GC > 0) NS = NS > (GC + NGC - 1) / NGC ? NS : (GC + NGC - 1) / NGC;
        NS = (NS + SPW - 1) / SPW * SPW;
        if (NS * LG > 256) continue;
        TeamPlan pl;
        pl.R = R; pl.CA = CA; pl.TA = TA; pl.LG = LG; pl.NS = NS; pl.CS = CS; pl.NGN = NGN; pl.NGC = NGC;
        const int maxdiag = H < W ? H : W;
        int NPG = 256 / (NS * LG);
        if (NPG > maxdiag) NPG = maxdiag;
        if (NPG < 1) NPG = 1;
        pl.NPG = NPG;
        pl.threads = NPG * NS * LG;
        pl.PMAXS = ((maxdiag + NPG - 1) / NPG + 1) & ~1;       // pixel pairs: keep the slot count even
        const size_t img = (size_t)(H + K - 1) * (W + K - 1) * CS;
        const size_t red = (size_t)NPG * (NS * LG / 32) * pl.PMAXS * LG * TA;
        pl.smem = sizeof(float) * (2 * img + red);
        if (pl.smem > max_smem) continue;
        int ncl = sm_count / R;
        if (ncl > B) ncl = B;
        if (ncl < 1) ncl = 1;
        pl.ncl = ncl;
        pl.ok = true;
        best = pl;
        break;
    }
    return best;
}

}  // namespace invconv

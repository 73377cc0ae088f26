// Launch geometry of the tensor-core wavefront (host side; see tensor_kernels.cuh for the kernel).
#pragma once

#include <stddef.h>

namespace invconv {

struct TensorPlan {
    bool ok = false;
    int R = 0;          // CTAs per cluster = C / (8 * NCH)
    int NCH = 0;        // 8-channel chunks of the contraction per CTA
    int I = 0;          // images per group (128 lanes / HP)
    int HP = 0;         // image rows padded to 8 or 16
    int S = 0;          // accumulator slots
    int ngroups = 0, ncl = 0;
    unsigned tmem_cols = 0;
    unsigned wbytes = 0;            // packed kernel bytes per CTA
    unsigned off_stage = 0, off_x = 0, off_y = 0, off_recv = 0, off_bar = 0;
    unsigned stage_img = 0;         // floats between the images of the staged slice
    size_t smem = 0;
    size_t wop_bytes = 0;           // packed kernel, all CTAs
};

constexpr int kTensorThreads = 416;     // warps 0-7: accumulators -> solved pixels; warp 8: MMA issue; warps 9-12: right-hand side

inline TensorPlan plan_tensor(int B, int C, int H, int W, int K, size_t max_smem, int sms)
{
    TensorPlan pl;
    if (K < 2 || K > 5 || H > 16 || C % 16 != 0 || C > 64 || (H * W) % 4 != 0 || B < 1) return pl;
    pl.NCH = 1;
    pl.R = C / 8;
    if (pl.R < 2 || pl.R > 8) return pl;
    pl.HP = H <= 8 ? 8 : 16;
    pl.I = 128 / pl.HP;
    pl.S = 2 * (K - 1);
    if (pl.S * C > 512) return pl;
    unsigned cols = 32;
    while (cols < (unsigned)(pl.S * C)) cols *= 2;
    pl.tmem_cols = cols;
    const int CS = 8 * pl.NCH, KC = K * C, ROWS = (K - 1) * pl.I + 128;
    auto up = [](size_t v) { return (v + 127) & ~(size_t)127; };
    pl.wbytes = (unsigned)(K * pl.NCH * KC * 64);
    pl.stage_img = (unsigned)(CS * H * W + 4);
    size_t off = up(pl.wbytes);
    pl.off_stage = (unsigned)off;  off = up(off + sizeof(float) * (size_t)pl.I * pl.stage_img);
    pl.off_x = (unsigned)off;      off = up(off + 2 * (size_t)pl.NCH * 4 * ROWS * 16);
    pl.off_y = (unsigned)off;      off = up(off + 2 * (size_t)pl.NCH * 4 * 128 * 16);
    pl.off_recv = (unsigned)off;   off = up(off + 2 * (size_t)(pl.R - 1) * 128 * CS * sizeof(float));
    pl.off_bar = (unsigned)off;    off += 256;
    pl.smem = off;
    if (pl.smem > max_smem) return pl;
    pl.ngroups = (B + pl.I - 1) / pl.I;
    int ncl = sms / pl.R;
    if (ncl < 1) return pl;
    pl.ncl = pl.ngroups < ncl ? pl.ngroups : ncl;
    pl.wop_bytes = (size_t)pl.R * pl.wbytes;
    pl.ok = true;
    return pl;
}

struct GradWTensorPlan {
    bool ok = false;
    int RB = 0, Wp = 0, nbands = 0, S = 0, grid = 0, nk = 0;
    unsigned tmem_cols = 0, planeA = 0, planeB = 0, stage_bytes = 0;
    size_t smem = 0;
};

constexpr int kGradWTensorIssuers = 4;        // MMA-issuing warps at most (a fifth accumulator shares the first warp)
constexpr int kGradWTensorProducers = 256;    // warps 0-7 stage the operands (0-3 also write the result); warps 8.. issue the MMAs, one per kernel column

inline GradWTensorPlan plan_gradw_tensor(int B, int C, int H, int W, int K, size_t max_smem, int sms)
{
    GradWTensorPlan pl;
    if (C % 16 != 0 || C < 16 || C > 128 || K * C > 512 || B < 1 || K > 5 || W % 4 != 0) return pl;
    pl.Wp = W;
    // Rows per unit: four, or more where few channels leave room (a unit then carries a thread's full four
    // items, and its fixed cost -- one L2 round trip, barrier hand-offs -- is paid less often), as long as every
    // CTA still gets at least two units to double-buffer.
    const int cand[4] = {16, 8, 4, 2};
    pl.RB = 0;
    for (int i = 0; i < 4; ++i) {
        const int rb = cand[i];
        if (rb > 4 && (rb > H || C * rb * (W / 4) > 4 * kGradWTensorProducers || (long long)B * ((H + rb - 1) / rb) < 2LL * (sms / K))) continue;
        if (rb == 4 && H < 4) continue;
        // one stage: grad_y and K shifted copies of x, [quad][channel][4 pixels] each, plus room for the rows
        // C..127 that the MMA reads (and ignores) behind the last quad plane
        pl.stage_bytes = (unsigned)(((size_t)(K + 1) * (rb * W / 4) * (C + 1) * 16 + 128 * 16 + 127) & ~(size_t)127);
        pl.smem = 2 * (size_t)pl.stage_bytes + 256;
        if (pl.smem <= max_smem) { pl.RB = rb; break; }
    }
    if (pl.RB < 2 || (pl.RB * W) % 8 != 0 || C * pl.RB * (W / 4) > 8 * kGradWTensorProducers) return pl;
    pl.nbands = (H + pl.RB - 1) / pl.RB;
    pl.nk = pl.RB * W / 8;
    pl.planeA = pl.planeB = (unsigned)(C + 1) * 16;
    pl.S = sms / K;
    if (pl.S < 1) return pl;
    const int units = B * pl.nbands;
    if (pl.S > units) pl.S = units;
    pl.grid = pl.S * K;
    unsigned cols = 32;
    while (cols < (unsigned)(K * C)) cols *= 2;
    pl.tmem_cols = cols;
    pl.ok = true;
    return pl;
}

// Masked convolution y = f(x) on the tensor cores (conv_tensor.cuh): lanes are the padded pixel slots of a band of
// rows of one image, taps are row offsets of the staged x operand, weights stream through a ring of stages.
struct ConvTensorPlan {
    bool ok = false;
    int RB = 0, Wp = 0, nbands = 0, ntiles = 0, grid = 0, slots = 0;
    int spi = 0;                    // weight stages per issuing warp (ring depth)
    unsigned tmem_cols = 0, x_bytes = 0, wstage_bytes = 0, off_w = 0, off_bar = 0;
    size_t smem = 0, pack_bytes = 0;
};

constexpr int kConvTensorThreads = 352;       // warps 0-7 stage x (0-3 also write y); warps 8, 9 issue MMAs; warp 10 loads weights
constexpr int kConvTensorMaxSpi = 4;            // at most 4 weight stages per issuing warp

inline ConvTensorPlan plan_conv_tensor(int B, int C, int H, int W, int K, size_t max_smem, int sms)
{
    ConvTensorPlan pl;
    if (C % 16 != 0 || C < 16 || C > 64 || K < 2 || K > 5 || B < 1) return pl;
    pl.Wp = W + K - 1;
    if (pl.Wp > 128) return pl;
    pl.wstage_bytes = (unsigned)((C / 8) * 4 * C * 16);
    for (pl.RB = 128 / pl.Wp < H ? 128 / pl.Wp : H; pl.RB >= 1; --pl.RB) {
        pl.slots = (K - 1) + (K - 1) * pl.Wp + 128 + pl.Wp;                 // every tap's 128 rows stay inside the buffer
        const int need = (K - 1) + (pl.RB + K - 1) * pl.Wp;
        if (need > pl.slots) pl.slots = need;
        pl.x_bytes = (unsigned)(((size_t)(C / 8) * 4 * pl.slots * 16 + 127) & ~(size_t)127);
        pl.off_w = pl.x_bytes;
        // as many weight stages as fit (the bytes in flight from L2 set the streaming rate), at least two per warp
        for (pl.spi = kConvTensorMaxSpi; pl.spi >= 2; --pl.spi) {
            pl.off_bar = pl.off_w + 2 * pl.spi * pl.wstage_bytes;
            pl.smem = (size_t)pl.off_bar + 256;
            if (pl.smem <= max_smem) break;
        }
        if (pl.spi >= 2) break;
    }
    if (pl.RB < 1) return pl;
    pl.nbands = (H + pl.RB - 1) / pl.RB;
    pl.ntiles = B * pl.nbands;
    pl.grid = pl.ntiles < sms ? pl.ntiles : sms;
    unsigned cols = 32;
    while (cols < (unsigned)(2 * C)) cols *= 2;
    pl.tmem_cols = cols;
    pl.pack_bytes = (size_t)K * K * pl.wstage_bytes;
    pl.ok = true;
    return pl;
}

}  // namespace invconv

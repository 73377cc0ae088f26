// C ABI of the inverse-convolution library: argument checks, kernel-family
// dispatch and launches.  Every step of the path runs in the kernels included
// below; nothing here computes.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "invconv.h"

#include "common.cuh"
#include "generic_kernels.cuh"
#include "probe_kernels.cuh"
#include "warp_kernels.cuh"
#include "team_kernels.cuh"
#include "tensor_plan.h"
#include "lib_internal.h"
#include "gradw_kernels.cuh"
#include "conv_kernels.cuh"

using namespace invconv;
using invconv_internal::set_smem_limit;
using invconv_internal::kMaxDynSmem;

namespace {

std::atomic<int> g_forced_path{INVCONV_PATH_AUTO};
std::atomic<unsigned long long> g_kernel_launches{0};
// development and test controls (invconv_set_option); defaults as documented in the header
std::atomic<int> g_opt[INVCONV_OPT_COUNT] = {{1}, {1}, {-1}, {1}, {0}, {0}, {1}};
inline int opt(int o) { return g_opt[o].load(std::memory_order_relaxed); }

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

}  // namespace

namespace invconv_internal {
// Called once after every kernel launch of the library.
int check_launch()
{
    g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: CUDA error: %s\n", cudaGetErrorString(e));
        return INVCONV_CUDA_ERROR;
    }
    return INVCONV_OK;
}
}  // namespace invconv_internal
using invconv_internal::check_launch;

namespace {

int check_shape(int B, int C, int H, int W, int k)
{
    if (B < 0 || C < 1 || H < 1 || W < 1 || k < 1) return INVCONV_BAD_ARG;
    if (k > INVCONV_MAX_K || C > INVCONV_MAX_C) return INVCONV_UNSUPPORTED;
    const long long e = (long long)B * C * H * W;
    if (e >= (1LL << 31)) return INVCONV_UNSUPPORTED;
    return INVCONV_OK;
}


// ---------------------------------------------------------------- warp family
#define INVCONV_WARP_CASES(X) \
    X(1, 2) X(1, 3) X(1, 5) X(2, 2) X(2, 3) X(2, 5) X(3, 2) X(3, 3) X(3, 5) X(4, 2) X(4, 3) X(4, 5)

struct WarpPlan {
    bool ok = false;
    bool glb = false;      // image too large for shared memory: operands stay in global memory
    bool ring = false;     // ... and a ring of 128 columns per warp fits: streamed through shared memory
    bool cs = false;       // channel-split walk available (lane = (row, output channel)); its own geometry below
    int nb = 0, ipc = 0, grid = 0;
    int nb_cs = 0, ipc_cs = 0, grid_cs = 0;
    size_t smem = 0, smem_ring = 0, smem_cs = 0;
};

template <int C, int K>
WarpPlan plan_warp_ck(int B, int H, int W, bool bwd)
{
    WarpPlan pl;
    pl.nb = (H + 31) / 32;
    if (pl.nb > 8) return pl;
    int ipc = 4 / pl.nb;
    if (ipc < 1) ipc = 1;
    if (ipc > B) ipc = B > 0 ? B : 1;
    while (ipc > 1 && warp_kernel_smem<C, K>(H, W, pl.nb, ipc, bwd) > kMaxDynSmem) --ipc;
    pl.smem = warp_kernel_smem<C, K>(H, W, pl.nb, ipc, bwd);
    if (pl.smem > kMaxDynSmem) {
        if (pl.nb < 2) return pl;
        ipc = 1;
        pl.glb = true;
        pl.smem = warp_kernel_smem<C, K>(H, W, pl.nb, 1, bwd, true);
        if (pl.smem > kMaxDynSmem) return pl;
        pl.smem_ring = warp_kernel_smem<C, K>(H, W, pl.nb, 1, bwd, true, true);
        pl.ring = pl.smem_ring <= kMaxDynSmem;
    }
    pl.ipc = ipc;
    pl.grid = (B + ipc - 1) / ipc;
    pl.ok = true;
    // channel-split walk: where the transformed kernel does not fit one lane's registers (C >= 3, 5x5)
    if (C >= 3 && K == 5 && !pl.glb) {
        const int rpw = 32 / C;
        const int nbc = (H + rpw - 1) / rpw;
        if (nbc <= 8) {
            int ic = 8 / nbc;
            if (ic < 1) ic = 1;
            if (ic > B) ic = B > 0 ? B : 1;
            while (ic > 1 && warp_kernel_smem<C, K>(H, W, nbc, ic, bwd) > kMaxDynSmem) --ic;
            const size_t sm = warp_kernel_smem<C, K>(H, W, nbc, ic, bwd);
            if (sm <= kMaxDynSmem) {
                pl.cs = true; pl.nb_cs = nbc; pl.ipc_cs = ic; pl.grid_cs = (B + ic - 1) / ic; pl.smem_cs = sm;
            }
        }
    }
    return pl;
}

WarpPlan plan_warp(int B, int C, int H, int W, int k, bool bwd)
{
#define X(CC, KK) if (C == CC && k == KK) return plan_warp_ck<CC, KK>(B, H, W, bwd);
    INVCONV_WARP_CASES(X)
#undef X
    return WarpPlan{};
}

template <int C, int K, bool BWD>
int launch_warp_ck(const WarpPlan& pl, WarpParams prm, cudaStream_t st)
{
    // global-memory mode: streamed through a shared-memory ring unless grad_w rides along in the wavefront
    const bool ring = pl.glb && pl.ring && prm.grad_w == nullptr && opt(INVCONV_OPT_WARP_RING) != 0;
    // channel-split walk (its own row-block geometry) unless grad_w rides along in the wavefront
    bool cs = false;
    if constexpr (C >= 3 && K == 5) cs = pl.cs && prm.grad_w == nullptr && opt(INVCONV_OPT_WARP_CHANNEL_SPLIT) != 0;
    auto kern = ring ? warp_wavefront_kernel<C, K, BWD, true, true, true>
                     : (pl.glb ? warp_wavefront_kernel<C, K, BWD, true, true>
                               : (pl.nb > 1 ? warp_wavefront_kernel<C, K, BWD, true> : warp_wavefront_kernel<C, K, BWD, false>));
    size_t smem = ring ? pl.smem_ring : pl.smem;
    int nb = pl.nb, ipc = pl.ipc, grid = pl.grid;
    if constexpr (C >= 3 && K == 5) {
        if (cs) {
            kern = pl.nb_cs > 1 ? warp_wavefront_kernel<C, K, BWD, true, false, false, true>
                                : warp_wavefront_kernel<C, K, BWD, false, false, false, true>;
            smem = pl.smem_cs; nb = pl.nb_cs; ipc = pl.ipc_cs; grid = pl.grid_cs;
            prm.nb = nb; prm.ipc = ipc;
        }
    }
    const int rc = set_smem_limit(kern, smem);
    if (rc) return rc;
    // Programmatic dependent launch: the kernel may be scheduled while its predecessor on the stream drains;
    // it touches no global memory before griddepcontrol.wait, which waits for that predecessor to complete.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(nb * ipc * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = opt(INVCONV_OPT_DEPENDENT_LAUNCH) ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: warp launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return check_launch();
}

constexpr size_t kGradWSmallSmem = 96 * 1024;

using invconv_internal::sm_count;

GradWSmallPlan gradw_small_plan(int B, int C, int H, int W, int k)
{
    return plan_gradw_small(B, C, H, W, k, kGradWSmallSmem, kMaxDynSmem - 8 * 1024, sm_count());
}

// Whether grad_w comes from the pixel-parallel kernel after the wavefront instead of riding along in it.
// Riding along costs every diagonal step C*C*k*k extra multiply-adds on the one warp that owns the rows; the
// separate kernel costs a launch and a second read of grad_y and x from L2.  Measured on B200, added time of
// the separate kernel against riding along: 18 us against 10 us (C=3, 32x32, k=3, batch 128), 11 us against
// 4 us (C=1, 28x28, k=3, batch 256), 13 us against 118 us (C=3, 64x64, k=5, batch 16, where the sums do not
// fit the wavefront's registers), 24 us against 75 us (C=1, 256x256, k=5, batch 4, images in global memory).
// So it is used where the sums do not fit the registers or the images stay in global memory (INVCONV_OPT_GRADW_SEPARATE overrides).
bool gradw_separate(const WarpPlan& pl, const GradWSmallPlan& gs, int C, int k)
{
    if (!gs.ok) return false;
    const int knob = opt(INVCONV_OPT_GRADW_SEPARATE);
    if (knob == 0) return false;
    if (knob == 1) return true;
    return pl.glb || C * C * k * k > 81;
}

template <int C, int K>
int launch_gradw_small_ck(const GradWSmallPlan& gs, const GradWSmallParams& prm, cudaStream_t st)
{
    auto kern = gradw_small_kernel<C, K>;
    const int rc = set_smem_limit(kern, gs.smem);
    if (rc) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(gs.grid);
    cfg.blockDim = dim3(GradWSmallShape<C, K>::NT);
    cfg.dynamicSmemBytes = gs.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = opt(INVCONV_OPT_DEPENDENT_LAUNCH) ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: grad_w launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return check_launch();
}

int launch_gradw_small(const GradWSmallPlan& gs, const float* gy, const float* x, float* gw, Geom g, void* ws, cudaStream_t st,
                       const LogdetFuse& ld)
{
    GradWSmallParams prm;
    prm.gy = gy; prm.x = x; prm.grad_w = gw; prm.ld = ld;
    prm.counter = static_cast<unsigned*>(ws);
    prm.partials = reinterpret_cast<float*>(static_cast<char*>(ws) + INVCONV_WS_CONTROL_BYTES);
    prm.B = g.B; prm.H = g.H; prm.W = g.W;
    prm.RB = gs.RB; prm.nbands = gs.nbands; prm.gst = gs.gst; prm.xst = gs.xst;
    prm.stage = (int)(gs.smem / sizeof(float));
    prm.bulk = (((reinterpret_cast<uintptr_t>(gy) | reinterpret_cast<uintptr_t>(x)) & 15) == 0 && g.W % 4 == 0) ? 1 : 0;
    prm.div_bands = make_fast_div((unsigned)gs.nbands);
    prm.div_gcpr = make_fast_div((unsigned)((gs.gst + 31) / 32));
    prm.div_xcpr = make_fast_div((unsigned)((gs.xst + 31) / 32));
    prm.div_rb = make_fast_div((unsigned)gs.RB);
    prm.div_xr = make_fast_div((unsigned)(gs.RB + g.k - 1));
    prm.div_qpr = make_fast_div((unsigned)(gs.gst / 4));
#define X(CC, KK) if (g.C == CC && g.k == KK) return launch_gradw_small_ck<CC, KK>(gs, prm, st);
    INVCONV_WARP_CASES(X)
#undef X
    return INVCONV_UNSUPPORTED;
}

// The per-pixel neighbours of the layer in a flow step, applied inside the wavefront kernel (see WarpParams).
struct WarpMix {
    const float* V = nullptr; const float* s = nullptr; const float* b = nullptr;
    float* u_out = nullptr;     // forward
    bool grad_in = false;       // backward
};

// `bf16`: rhs, out and xsaved are bfloat16 images (see WarpParams::bf16); INVCONV_UNSUPPORTED where the kernel
// cannot take them (images in global memory, grad_w from the separate kernel, sizes or pointers the bulk copies
// do not accept) -- the caller then converts around the fp32 path.
int launch_warp(bool bwd, const float* rhs, const float* w, float* out, const float* xsaved, float* gw, Geom g,
                void* ws, cudaStream_t st, const WarpMix* mix = nullptr, float* logdet_out = nullptr,
                const LogdetFuse& ld = LogdetFuse{}, bool bf16 = false)
{
    const WarpPlan pl = plan_warp(g.B, g.C, g.H, g.W, g.k, bwd);
    if (!pl.ok) return INVCONV_UNSUPPORTED;
    if (mix && pl.glb) return INVCONV_UNSUPPORTED;       // images in global memory: the caller composes the step
    const GradWSmallPlan gs = (bwd && gw) ? gradw_small_plan(g.B, g.C, g.H, g.W, g.k) : GradWSmallPlan{};
    const bool separate = bwd && gw && ws && gradw_separate(pl, gs, g.C, g.k);
    if (bf16 && (pl.glb || separate || mix)) return INVCONV_UNSUPPORTED;
    WarpParams prm;
    prm.rhs = rhs; prm.w = w; prm.out = out; prm.xsaved = xsaved; prm.grad_w = separate ? nullptr : gw;
    prm.counter = static_cast<unsigned*>(ws);
    prm.partials = ws ? reinterpret_cast<float*>(static_cast<char*>(ws) + INVCONV_WS_CONTROL_BYTES) : nullptr;
    prm.B = g.B; prm.H = g.H; prm.W = g.W; prm.nb = pl.nb; prm.ipc = pl.ipc;
    prm.logdet_out = bwd ? nullptr : logdet_out;
    prm.ld = ld;
    if (mix) {
        prm.mix_V = mix->V; prm.mix_s = mix->s; prm.mix_b = mix->b;
        prm.mix_out = bwd ? nullptr : mix->u_out;
        prm.mix_in = (bwd && mix->grad_in) ? 1 : 0;
    }
    const size_t chw = (size_t)g.C * g.H * g.W;
    const bool aligned = ((reinterpret_cast<uintptr_t>(rhs) | reinterpret_cast<uintptr_t>(out) |
                           reinterpret_cast<uintptr_t>(xsaved)) & 15) == 0;
    prm.bulk = (aligned && chw % 4 == 0) ? 1 : 0;
    if (bf16) {
        if (!aligned || chw % 8 != 0) return INVCONV_UNSUPPORTED;
        prm.bulk = 1; prm.bf16 = 1;
    }
    prm.glb = pl.glb ? 1 : 0;
    prm.vec = (aligned && g.W % 4 == 0) ? 1 : 0;
    int rc = INVCONV_UNSUPPORTED;
#define X(CC, KK)                                                                         \
    if (g.C == CC && g.k == KK)                                                           \
        rc = bwd ? launch_warp_ck<CC, KK, true>(pl, prm, st) : launch_warp_ck<CC, KK, false>(pl, prm, st);
    INVCONV_WARP_CASES(X)
#undef X
    if (rc || !separate) return rc;
    return launch_gradw_small(gs, out, xsaved, gw, g, ws, st, ld);
}

size_t warp_workspace_bytes(int B, int C, int H, int W, int k)
{
    const WarpPlan pl = plan_warp(B, C, H, W, k, true);
    if (!pl.ok) return 0;
    const size_t na = (size_t)C * C * k * k;
    size_t floats = (size_t)pl.grid * na;
    const GradWSmallPlan gs = gradw_small_plan(B > 0 ? B : 1, C, H, W, k);
    if (gs.ok && (size_t)gs.grid * ((na + 3) & ~(size_t)3) > floats) floats = (size_t)gs.grid * ((na + 3) & ~(size_t)3);
    return INVCONV_WS_CONTROL_BYTES + sizeof(float) * floats;
}

// ---------------------------------------------------------------- masked convolution, few channels
template <int C, int K>
int launch_masked_conv_ck(const float* x, const float* w, float* y, Geom g, cudaStream_t st)
{
    // warps per band of rows: one, or one per output channel where the kernel does not fit a lane's registers
    constexpr int wsplit = (C * C * K * K <= 108) ? 1 : C;
    constexpr int maxw = 8 / wsplit;             // eight warps per CTA
    int wpi = (g.H + 7) / 8;                     // about eight rows per warp
    if (wpi > maxw) wpi = maxw;
    if (wpi < 1) wpi = 1;
    int ipc = maxw / wpi;
    if (ipc > g.B) ipc = g.B;
    if (ipc < 1) ipc = 1;
    while (ipc > 1 && masked_conv_smem<C, K>(g.H, g.W, ipc) > kMaxDynSmem) --ipc;
    size_t smem = masked_conv_smem<C, K>(g.H, g.W, ipc);
    const size_t chw = (size_t)g.C * g.H * g.W;
    ConvParams prm;
    prm.x = x; prm.w = w; prm.y = y; prm.B = g.B; prm.H = g.H; prm.W = g.W;
    prm.bulk = ((reinterpret_cast<uintptr_t>(x) & 15) == 0 && chw % 4 == 0) ? 1 : 0;
    int grid = (g.B + ipc - 1) / ipc;
    // few (fewer CTAs than half the SMs) or very large images: one CTA per band of rows instead, about two CTAs per SM
    const bool rows_ok = (reinterpret_cast<uintptr_t>(x) & 15) == 0 && g.W % 4 == 0;
    if (rows_ok && g.H >= 16 && (smem > kMaxDynSmem || 2 * grid <= sm_count())) {
        int bands = (2 * sm_count() + g.B - 1) / g.B;
        if (bands > (g.H + 7) / 8) bands = (g.H + 7) / 8;             // at least eight rows per band
        int bh = (g.H + bands - 1) / bands;
        while (masked_conv_smem<C, K>(bh + K - 1, g.W, 1) > kMaxDynSmem && bh > 1) bh = (bh + 1) / 2;
        bands = (g.H + bh - 1) / bh;
        if (bands > 1 && masked_conv_smem<C, K>(bh + K - 1, g.W, 1) <= kMaxDynSmem) {
            prm.bands = bands; prm.bh = bh; prm.bulk = 1;
            ipc = 1;
            wpi = bh >= 16 ? 4 : (bh >= 8 ? 2 : 1);
            if (wpi > maxw) wpi = maxw;
            smem = masked_conv_smem<C, K>(bh + K - 1, g.W, 1);
            grid = g.B * bands;
        }
    }
    if (smem > kMaxDynSmem) return INVCONV_UNSUPPORTED;
    auto kern = masked_conv_warp_kernel<C, K>;
    const int rc = set_smem_limit(kern, smem);
    if (rc) return rc;
    prm.ipc = ipc; prm.wpi = wpi;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(ipc * wpi * wsplit * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // launch latency overlaps the kernel before
    attr[0].val.programmaticStreamSerializationAllowed = opt(INVCONV_OPT_DEPENDENT_LAUNCH) ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, prm) != cudaSuccess) {
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return check_launch();
}

template <int K>
int launch_masked_conv_tile_k(const ConvTilePlan& pl, const ConvTileParams& prm, cudaStream_t st)
{
    auto kern = masked_conv_tile_kernel<K>;
    const int rc = set_smem_limit(kern, pl.smem);
    if (rc) return rc;
    kern<<<pl.grid, pl.threads, pl.smem, st>>>(prm);
    return check_launch();
}

// Many channels: the register-tiled kernel; INVCONV_UNSUPPORTED where its plan does not fit.
int launch_masked_conv_tile(const float* x, const float* w, float* y, Geom g, cudaStream_t st)
{
    const ConvTilePlan pl = plan_conv_tile(g.B, g.C, g.H, g.W, g.k, kMaxDynSmem / 2, sm_count());
    if (!pl.ok) return INVCONV_UNSUPPORTED;
    ConvTileParams prm;
    prm.x = x; prm.w = w; prm.y = y; prm.B = g.B; prm.C = g.C; prm.H = g.H; prm.W = g.W;
    prm.RB = pl.RB; prm.nbands = pl.nbands; prm.Q = pl.Q; prm.IPC = pl.IPC; prm.PW = pl.PW; prm.PH = pl.PH;
    prm.cotiles = pl.cotiles;
    prm.vec = (((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15) == 0 && g.W % 4 == 0) ? 1 : 0;
    prm.div_q = make_fast_div((unsigned)pl.Q);
    prm.div_qpr = make_fast_div((unsigned)((pl.PW - 4) / 4));
    prm.div_bands = make_fast_div((unsigned)pl.nbands);
    prm.div_ph = make_fast_div((unsigned)pl.PH);
    switch (g.k) {
    case 1: return launch_masked_conv_tile_k<1>(pl, prm, st);
    case 2: return launch_masked_conv_tile_k<2>(pl, prm, st);
    case 3: return launch_masked_conv_tile_k<3>(pl, prm, st);
    case 4: return launch_masked_conv_tile_k<4>(pl, prm, st);
    case 5: return launch_masked_conv_tile_k<5>(pl, prm, st);
    default: return INVCONV_UNSUPPORTED;
    }
}

int launch_masked_conv_small(const float* x, const float* w, float* y, Geom g, cudaStream_t st)
{
#define X(CC, KK) if (g.C == CC && g.k == KK) return launch_masked_conv_ck<CC, KK>(x, w, y, g, st);
    INVCONV_WARP_CASES(X)
#undef X
    return INVCONV_UNSUPPORTED;
}

// ---------------------------------------------------------------- team family
}  // namespace
namespace invconv_internal {
// Scratch comes from a memory pool the library owns (one per device, created on first use) whose release
// threshold is unlimited: memory freed with cudaFreeAsync stays in the pool across synchronisations, so the
// steady state allocates nothing from the driver (the default pool would hand its memory back at every
// synchronisation and pay for a fresh allocation, about 200 us, on the next call).
int scratch_alloc(void** out, size_t bytes, cudaStream_t st)
{
    static std::mutex mu;
    static cudaMemPool_t pools[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    cudaMemPool_t pool;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!pools[dev]) {
            // a pool cannot be created while the stream is being captured into a graph: this call then takes the
            // device's default pool (make the first call of a process outside a capture to get the library's pool)
            cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
            if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
            if (cap != cudaStreamCaptureStatusNone) {
                if (cudaMallocAsync(out, bytes, st) != cudaSuccess) { cudaGetLastError(); *out = nullptr; return INVCONV_CUDA_ERROR; }
                return INVCONV_OK;
            }
            cudaMemPoolProps props = {};
            props.allocType = cudaMemAllocationTypePinned;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            if (cudaMemPoolCreate(&pools[dev], &props) != cudaSuccess) { cudaGetLastError(); pools[dev] = nullptr; return INVCONV_CUDA_ERROR; }
            unsigned long long keep = ~0ull;
            cudaMemPoolSetAttribute(pools[dev], cudaMemPoolAttrReleaseThreshold, &keep);
        }
        pool = pools[dev];
    }
    if (cudaMallocFromPoolAsync(out, bytes, pool, st) != cudaSuccess) { cudaGetLastError(); *out = nullptr; return INVCONV_CUDA_ERROR; }
    return INVCONV_OK;
}

int sm_count()
{
    static std::atomic<int> cached[64];
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    const int v = cached[dev].load();
    if (v > 0) return v;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return 148;            // B200; only used for planning when no device is present
    }
    cached[dev].store(n);
    return n;
}
}  // namespace invconv_internal
namespace {

TeamPlan team_plan(int B, int C, int H, int W, int k)
{
    if (team_solve_smem(C, k) > kMaxDynSmem) return TeamPlan{};
    return plan_team(B > 0 ? B : 1, C, H, W, k, kMaxDynSmem, sm_count(), opt(INVCONV_OPT_TEAM_VARIANT), opt(INVCONV_OPT_TEAM_CLUSTER));
}

GradWPlan gradw_plan(int B, int C, int H, int W, int k)
{
    return plan_gradw(B, C, H, W, k, kMaxDynSmem / 2, sm_count());      // two CTAs per SM
}

GradWTensorPlan gradw_tensor_plan(int B, int C, int H, int W, int k)
{
    return plan_gradw_tensor(B > 0 ? B : 1, C, H, W, k, kMaxDynSmem, sm_count());
}

// Workspace of the team family: control words, transformed kernel, C*C floats, then the partial sums of
// grad_w -- one set per batch share of whichever correlation kernel runs (the tcgen05 one included).
size_t team_workspace_bytes(int B, int C, int H, int W, int k)
{
    if (!team_plan(B, C, H, W, k).ok) return 0;
    const size_t na = sizeof(float) * (size_t)k * k * C * C;
    const GradWPlan gp = gradw_plan(B, C, H, W, k);
    const GradWTensorPlan gt = gradw_tensor_plan(B, C, H, W, k);
    int shares = gp.ok ? (gp.nbc > gp.nbc_all ? gp.nbc : gp.nbc_all) : 0;
    if (gt.ok && gt.S > shares) shares = gt.S;
    return INVCONV_WS_CONTROL_BYTES + na + sizeof(float) * (size_t)C * C + na * shares;
}

template <int TC, int K>
int launch_gradw_inst(const GradWPlan& gp, const GradWParams& prm, cudaStream_t st)
{
    auto kern = gradw_tile_kernel<TC, K>;
    const int rc = set_smem_limit(kern, gp.smem);
    if (rc) return rc;
    kern<<<gp.grid, 256, gp.smem, st>>>(prm);
    return check_launch();
}

template <int TC, int K>
int launch_gradw_mma_inst(const GradWPlan& gp, const GradWParams& prm, cudaStream_t st)
{
    auto kern = gradw_mma_kernel<TC, K>;
    const int rc = set_smem_limit(kern, gp.smem);
    if (rc) return rc;
    kern<<<gp.grid, 32 * TC * K, gp.smem, st>>>(prm);
    return check_launch();
}

template <int K>
int launch_gradw_mma_all_inst(const GradWPlan& gp, const GradWParams& prm, cudaStream_t st)
{
    auto kern = gradw_mma_kernel<1, K, true>;
    const int rc = set_smem_limit(kern, gp.smem);
    if (rc) return rc;
    kern<<<gp.grid_all, 32 * K * K, gp.smem, st>>>(prm);
    return check_launch();
}

// grad_w through the tiled correlation kernel; partial sums live behind the transformed kernel in the workspace.
int launch_gradw(const float* gy, const float* x, float* gw, Geom g, void* ws, cudaStream_t st, const LogdetFuse& ld)
{
    const GradWPlan gp = gradw_plan(g.B, g.C, g.H, g.W, g.k);
    const bool aligned = ((reinterpret_cast<uintptr_t>(gy) | reinterpret_cast<uintptr_t>(x)) & 15) == 0;
    if (!gp.ok || !aligned || g.B == 0) {
        generic_grad_w_kernel<<<g.C * g.C * g.k * g.k, 128, 0, st>>>(gy, x, gw, g, ld);
        return check_launch();
    }
    const size_t na = (size_t)g.k * g.k * g.C * g.C;
    GradWParams prm;
    prm.gy = gy; prm.x = x;
    prm.partials = reinterpret_cast<float*>(static_cast<char*>(ws) + INVCONV_WS_CONTROL_BYTES) + na + (size_t)g.C * g.C;
    prm.B = g.B; prm.C = g.C; prm.H = g.H; prm.W = g.W; prm.nbc = gp.nbc; prm.tiles = gp.tiles; prm.plane = gp.plane;
    int rc = INVCONV_UNSUPPORTED;
    // tensor pipe (TF32 inputs) where the fragments line up: rows of whole 8-pixel chunks, conflict-free planes
    // (measured, kernel + reduction: 31 / 58 us against 41 / 87 us for the FMA kernel on the 48-channel shapes,
    // k = 3 / 5; 19 us against 25 us on the 12-channel one with all taps in one CTA)
    // Not below 8 channels: with a handful of entries none of them is large against the cancellation in its own sum,
    // and TF32 rounding (2^-11 per operand) then shows at 1e-3 of the entry (seen at C = 1, 2 with k = 1).
    const bool mma = g.C >= 8 && g.W % 8 == 0 && gp.plane % 32 == 4 && opt(INVCONV_OPT_GRADW_TENSOR_PIPE) != 0;
    int shares = gp.nbc;
    if (mma && gp.TC == 1) {                 // tiles of 16 channels: one CTA covers all taps, its own share count
        shares = gp.nbc_all;
        prm.nbc = shares;
        if (g.k == 1) rc = launch_gradw_mma_all_inst<1>(gp, prm, st);
        if (g.k == 2) rc = launch_gradw_mma_all_inst<2>(gp, prm, st);
        if (g.k == 3) rc = launch_gradw_mma_all_inst<3>(gp, prm, st);
        if (g.k == 5) rc = launch_gradw_mma_all_inst<5>(gp, prm, st);
    } else {
#define X(TT, KK_)                                                                                    \
    if (gp.TC == TT && g.k == KK_) rc = (mma && TT == 3) ? launch_gradw_mma_inst<TT, KK_>(gp, prm, st) : launch_gradw_inst<TT, KK_>(gp, prm, st);
    X(1, 1) X(1, 2) X(1, 3) X(1, 5) X(3, 1) X(3, 2) X(3, 3) X(3, 5)
#undef X
    }
    if (rc) return rc;
    if (na < 16384) {       // few entries: four lanes per entry (64 entries per CTA)
        gradw_reduce_kernel<4><<<(int)((na + 63) / 64), 256, 0, st>>>(prm.partials, gw, shares, g.C, g.k, ld);
    } else {
        const int blocks = (int)((na + 255) / 256 < 4096 ? (na + 255) / 256 : 4096);
        gradw_reduce_kernel<1><<<blocks, 256, 0, st>>>(prm.partials, gw, shares, g.C, g.k, ld);
    }
    return check_launch();
}

template <int TA, int NGN, int NGC, int PM, int MAXT>
int launch_team_inst(const TeamPlan& pl, const TeamParams& prm, cudaStream_t st)
{
    auto kern = team_wavefront_kernel<TA, NGN, NGC, PM, MAXT>;
    const int rc = set_smem_limit(kern, pl.smem);
    if (rc) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.ncl * pl.R);
    cfg.blockDim = dim3(pl.threads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = pl.R; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = opt(INVCONV_OPT_DEPENDENT_LAUNCH) ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: team launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return check_launch();
}

template <int TA, int NGN, int NGC, int PJ>
int launch_pixel_inst(const TeamPlan& pl, const TeamParams& prm, cudaStream_t st)
{
    auto kern = team_pixel_kernel<TA, NGN, NGC, PJ>;
    const int rc = set_smem_limit(kern, pl.smem);
    if (rc) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.ncl * pl.R);
    cfg.blockDim = dim3(pl.threads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = pl.R; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = opt(INVCONV_OPT_DEPENDENT_LAUNCH) ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: pixel-team launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return check_launch();
}

// Transposed or plain solve through the team family; the transformed kernel goes to the workspace.
int launch_team(bool bwd, const float* rhs, const float* w, float* out, Geom g, void* ws, cudaStream_t st, float* logdet_out = nullptr)
{
    const TeamPlan pl = team_plan(g.B, g.C, g.H, g.W, g.k);
    if (!pl.ok) return INVCONV_UNSUPPORTED;
    float* A = reinterpret_cast<float*>(static_cast<char*>(ws) + INVCONV_WS_CONTROL_BYTES);
    {
        if (team_solve_launch(bwd, w, A, g.C, g.k, nullptr, 0, 0u, logdet_out, g.H * g.W, st) != cudaSuccess) {
            cudaGetLastError();
            return INVCONV_CUDA_ERROR;
        }
        const int rl = check_launch();
        if (rl) return rl;
    }
    TeamParams prm;
    prm.rhs = rhs; prm.A = A; prm.out = out;
    prm.B = g.B; prm.C = g.C; prm.H = g.H; prm.W = g.W; prm.K = g.k;
    prm.R = pl.R; prm.CA = pl.CA; prm.LG = pl.LG; prm.NS = pl.NS; prm.NPG = pl.NPG; prm.CS = pl.CS;
    prm.KW = pl.KW;
    prm.rot = bwd ? 1 : 0; prm.ncl = pl.ncl;
    prm.vec = (((reinterpret_cast<uintptr_t>(rhs) | reinterpret_cast<uintptr_t>(out)) & 15) == 0 && (g.H * g.W) % 4 == 0) ? 1 : 0;
    prm.div_w = make_fast_div((unsigned)g.W);
    prm.div_hw = make_fast_div((unsigned)(g.H * g.W));
    prm.div_q4 = make_fast_div((unsigned)(g.H * g.W / 4 > 0 ? g.H * g.W / 4 : 1));
    if (pl.pixel) {
#define XP(TT, GN_, GC_, PJ_) \
    if (pl.TA == TT && pl.NGN == GN_ && pl.NGC == GC_ && pl.PJ == PJ_) return launch_pixel_inst<TT, GN_, GC_, PJ_>(pl, prm, st);
        XP(3, 3, 1, 1) XP(3, 6, 2, 1) XP(3, 12, 3, 1) XP(3, 3, 1, 2) XP(3, 6, 2, 2) XP(3, 12, 3, 2)
        XP(4, 3, 1, 1) XP(4, 6, 2, 1) XP(4, 12, 3, 1) XP(4, 3, 1, 2) XP(4, 6, 2, 2) XP(4, 12, 3, 2)
#undef XP
        return INVCONV_UNSUPPORTED;
    }
#define X(TT, GN_, GC_, PM_, MT_)                                                              \
    if (pl.TA == TT && pl.NGN == GN_ && pl.NGC == GC_ && pl.PM == PM_ && pl.maxt == MT_)          \
        return launch_team_inst<TT, GN_, GC_, PM_, MT_>(pl, prm, st);
    X(3, 3, 1, 8, 256) X(3, 6, 2, 8, 256) X(3, 9, 1, 8, 256) X(3, 3, 1, 16, 256) X(3, 6, 2, 16, 256) X(3, 9, 1, 16, 256)
    X(4, 3, 1, 8, 256) X(4, 6, 2, 8, 256) X(4, 9, 1, 8, 256) X(4, 3, 1, 16, 256) X(4, 6, 2, 16, 256) X(4, 9, 1, 16, 256)
#undef X
    return INVCONV_UNSUPPORTED;
}

// ---------------------------------------------------------------- tensor family
TensorPlan tensor_plan(int B, int C, int H, int W, int k)
{
    if (team_solve_smem(C, k) > kMaxDynSmem) return TensorPlan{};
    return plan_tensor(B > 0 ? B : 1, C, H, W, k, kMaxDynSmem, sm_count());
}

// Workspace: control words, transformed kernel [k*k][C][C] (+ C*C floats of slack shared with the team
// family's layout), grad_w partial sums, then the packed tensor-core operands.
size_t tensor_wop_offset(int B, int C, int H, int W, int k)
{
    const size_t na = sizeof(float) * (size_t)k * k * C * C;
    const GradWPlan gp = gradw_plan(B, C, H, W, k);
    const int shares = gp.nbc > gp.nbc_all ? gp.nbc : gp.nbc_all;
    const size_t base = INVCONV_WS_CONTROL_BYTES + na + sizeof(float) * (size_t)C * C + (gp.ok ? na * shares : 0);
    return (base + 255) & ~(size_t)255;
}

size_t tensor_gradw_offset(int B, int C, int H, int W, int k)
{
    return (tensor_wop_offset(B, C, H, W, k) + tensor_plan(B, C, H, W, k).wop_bytes + 255) & ~(size_t)255;
}

size_t tensor_workspace_bytes(int B, int C, int H, int W, int k)
{
    const TensorPlan pl = tensor_plan(B, C, H, W, k);
    if (!pl.ok) return 0;
    const GradWTensorPlan gt = gradw_tensor_plan(B, C, H, W, k);
    const size_t na = sizeof(float) * (size_t)k * k * C * C;
    return tensor_gradw_offset(B, C, H, W, k) + (gt.ok ? na * gt.S : 0);
}

// grad_w through the tensor-core correlation kernel and the fixed-order reduction over its shares.
// `partials_offset`: where in the workspace the [shares][k*k][C][C] partial sums go.
int launch_gradw_tensor(const float* gy, const float* x, float* gw, Geom g, void* ws, size_t partials_offset, cudaStream_t st,
                        const LogdetFuse& ld)
{
    const GradWTensorPlan gt = gradw_tensor_plan(g.B, g.C, g.H, g.W, g.k);
    const bool aligned = ((reinterpret_cast<uintptr_t>(gy) | reinterpret_cast<uintptr_t>(x)) & 15) == 0;
    if (!gt.ok || !aligned || g.B == 0 || opt(INVCONV_OPT_GRADW_TENSOR_PIPE) == 0) return launch_gradw(gy, x, gw, g, ws, st, ld);
    float* partials = reinterpret_cast<float*>(static_cast<char*>(ws) + partials_offset);
    const int rc = invconv_internal::gradw_tensor_launch(gt, gy, x, partials, g, st);
    if (rc) return rc;
    const size_t na = (size_t)g.k * g.k * g.C * g.C;
    if (na < 16384) {
        gradw_reduce_kernel<4><<<(int)((na + 63) / 64), 256, 0, st>>>(partials, gw, gt.S, g.C, g.k, ld);
    } else {
        const int blocks = (int)((na + 255) / 256 < 4096 ? (na + 255) / 256 : 4096);
        gradw_reduce_kernel<1><<<blocks, 256, 0, st>>>(partials, gw, gt.S, g.C, g.k, ld);
    }
    return check_launch();
}

// Plain or transposed solve on the tensor cores: kernel transform, operand packing, wavefront.
int launch_tensor(bool bwd, const float* rhs, const float* w, float* out, Geom g, void* ws, cudaStream_t st, float* logdet_out = nullptr)
{
    const TensorPlan pl = tensor_plan(g.B, g.C, g.H, g.W, g.k);
    if (!pl.ok) return INVCONV_UNSUPPORTED;
    float* A = reinterpret_cast<float*>(static_cast<char*>(ws) + INVCONV_WS_CONTROL_BYTES);
    unsigned char* wop = static_cast<unsigned char*>(ws) + tensor_wop_offset(g.B, g.C, g.H, g.W, g.k);
    return invconv_internal::tensor_launch(pl, bwd, rhs, w, out, g, A, wop, st, logdet_out);
}

// ---------------------------------------------------------------- dispatch
int auto_path(int B, int C, int H, int W, int k)
{
    if (plan_warp(B > 0 ? B : 1, C, H, W, k, true).ok) return INVCONV_PATH_WARP;
    if (tensor_plan(B, C, H, W, k).ok) return INVCONV_PATH_TENSOR;
    if (team_plan(B, C, H, W, k).ok) return INVCONV_PATH_TEAM;
    return INVCONV_PATH_GENERIC;
}

int resolve_path(int B, int C, int H, int W, int k)
{
    const int forced = g_forced_path.load();
    return forced == INVCONV_PATH_AUTO ? auto_path(B, C, H, W, k) : forced;
}

size_t workspace_bytes_for(int path, int B, int C, int H, int W, int k)
{
    if (path == INVCONV_PATH_WARP) return warp_workspace_bytes(B, C, H, W, k);
    if (path == INVCONV_PATH_TEAM) return team_workspace_bytes(B, C, H, W, k);
    if (path == INVCONV_PATH_TENSOR) return tensor_workspace_bytes(B, C, H, W, k);
    return 0;
}

// `logdet_out` (optional): the layer's log-det, written by the forward kernels themselves where they have a
// warp to spare (warp family; the kernel transform of the team and tensor families), else by its own launch.
int launch_forward(int path, const float* y, const float* w, float* x, Geom g,
                   void* ws, size_t ws_bytes, cudaStream_t st, float* logdet_out = nullptr)
{
    (void)ws_bytes;
    auto separate_logdet = [&]() {
        if (!logdet_out) return (int)INVCONV_OK;
        logdet_kernel<<<1, 32, 0, st>>>(w, logdet_out, g.C, g.H, g.W, g.k);
        return check_launch();
    };
    if (g.B == 0) return separate_logdet();
    switch (path) {
    case INVCONV_PATH_GENERIC: {
        generic_wavefront_kernel<false><<<g.B, 256, 0, st>>>(y, w, x, g);
        const int rc = check_launch();
        return rc ? rc : separate_logdet();
    }
    case INVCONV_PATH_WARP:
        return launch_warp(false, y, w, x, nullptr, nullptr, g, ws, st, nullptr, logdet_out);
    case INVCONV_PATH_TEAM:
        return launch_team(false, y, w, x, g, ws, st, logdet_out);
    case INVCONV_PATH_TENSOR: {
        // buffers off a 16-byte boundary cannot use the bulk copies of the tensor family: the team family serves
        // them from the same workspace (its layout is a prefix of the tensor family's)
        const bool aligned = ((reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(x)) & 15) == 0;
        if (!aligned && g_forced_path.load() == INVCONV_PATH_AUTO) {
            if (team_plan(g.B, g.C, g.H, g.W, g.k).ok) return launch_team(false, y, w, x, g, ws, st, logdet_out);
            generic_wavefront_kernel<false><<<g.B, 256, 0, st>>>(y, w, x, g);      // neither family takes them: the generic one does
            const int rc = check_launch();
            return rc ? rc : separate_logdet();
        }
        return launch_tensor(false, y, w, x, g, ws, st, logdet_out);
    }
    default:
        return INVCONV_UNSUPPORTED;
    }
}

// `grad_logdet` (optional, one device float): the kernels that write the final grad_w add the log-det's term.
int launch_backward(int path, const float* gx, const float* x, const float* w, float* gy, float* gw, Geom g,
                    void* ws, size_t ws_bytes, cudaStream_t st, const float* grad_logdet = nullptr)
{
    (void)ws_bytes;
    LogdetFuse ld;
    ld.grad_logdet = grad_logdet; ld.w = w; ld.HW = g.H * g.W;
    switch (path) {
    case INVCONV_PATH_GENERIC: {
        if (g.B > 0) {
            generic_wavefront_kernel<true><<<g.B, 256, 0, st>>>(gx, w, gy, g);
            const int rc = check_launch();
            if (rc) return rc;
        }
        if (gw) {
            generic_grad_w_kernel<<<g.C * g.C * g.k * g.k, 128, 0, st>>>(gy, x, gw, g, ld);
            return check_launch();
        }
        return INVCONV_OK;
    }
    case INVCONV_PATH_WARP:
        return launch_warp(true, gx, w, gy, x, gw, g, ws, st, nullptr, nullptr, ld);
    case INVCONV_PATH_TEAM: {
        if (g.B > 0) {
            const int rc = launch_team(true, gx, w, gy, g, ws, st);
            if (rc) return rc;
        }
        if (gw) {
            const size_t na = sizeof(float) * (size_t)g.k * g.k * g.C * g.C;
            return launch_gradw_tensor(gy, x, gw, g, ws, INVCONV_WS_CONTROL_BYTES + na + sizeof(float) * (size_t)g.C * g.C, st, ld);
        }
        return INVCONV_OK;
    }
    case INVCONV_PATH_TENSOR: {
        if (g.B > 0) {
            const bool aligned = ((reinterpret_cast<uintptr_t>(gx) | reinterpret_cast<uintptr_t>(gy)) & 15) == 0;
            int rc;
            if (!aligned && g_forced_path.load() == INVCONV_PATH_AUTO) {
                if (team_plan(g.B, g.C, g.H, g.W, g.k).ok) {
                    rc = launch_team(true, gx, w, gy, g, ws, st);
                } else {
                    generic_wavefront_kernel<true><<<g.B, 256, 0, st>>>(gx, w, gy, g);
                    rc = check_launch();
                }
            } else {
                rc = launch_tensor(true, gx, w, gy, g, ws, st);
            }
            if (rc) return rc;
        }
        if (gw) return launch_gradw_tensor(gy, x, gw, g, ws, tensor_gradw_offset(g.B, g.C, g.H, g.W, g.k), st, ld);
        return INVCONV_OK;
    }
    default:
        return INVCONV_UNSUPPORTED;
    }
}

// Stream-ordered scratch for the entry points that take no workspace (see invconv_internal::scratch_alloc).
struct StreamScratch {
    void* p = nullptr;
    cudaStream_t st;
    int acquire(size_t bytes, cudaStream_t s) {
        st = s;
        if (bytes == 0) return INVCONV_OK;
        const int rc = invconv_internal::scratch_alloc(&p, bytes, st);
        if (rc) { p = nullptr; return rc; }
        if (cudaMemsetAsync(p, 0, INVCONV_WS_CONTROL_BYTES, st) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
        return INVCONV_OK;
    }
    ~StreamScratch() { if (p) cudaFreeAsync(p, st); }
};

// Side stream and events of invconv_step_host, one set per device, created on first use and kept.
struct StepSide {
    cudaStream_t side = nullptr;
    cudaEvent_t start = nullptr, gx_in = nullptr, x_ready = nullptr, x_out = nullptr;
    bool ok = false;
    std::mutex enqueue;     // one call at a time records and waits on the events (calls may come from several threads)
};

StepSide* step_side()
{
    static std::mutex mu;
    static StepSide sides[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return nullptr; }
    std::lock_guard<std::mutex> lock(mu);
    StepSide& s = sides[dev];
    if (!s.ok) {
        bool good = cudaStreamCreateWithFlags(&s.side, cudaStreamNonBlocking) == cudaSuccess;
        cudaEvent_t* evs[4] = {&s.start, &s.gx_in, &s.x_ready, &s.x_out};
        for (cudaEvent_t* e : evs) good = good && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
        if (!good) { cudaGetLastError(); return nullptr; }
        s.ok = true;
    }
    return &s;
}

// ---------------------------------------------------------------- bfloat16 storage around the fp32 path
// Where a kernel family cannot take bfloat16 images itself, the variant is composed: widen into fp32 scratch, run
// the fp32 path, narrow the result.  Eight values per thread where the buffers allow 16-byte accesses.
__global__ void widen_bf16_kernel(const __nv_bfloat16* __restrict__ in, float* __restrict__ out, size_t n, int vec)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    if (vec) {
        for (size_t u = (size_t)blockIdx.x * blockDim.x + threadIdx.x; u < n / 8; u += stride) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(in) + u);
            float4* d = reinterpret_cast<float4*>(out) + 2 * u;
            d[0] = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                               __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
            d[1] = make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u),
                               __uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
        }
    } else {
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) out[i] = __bfloat162float(in[i]);
    }
}

__global__ void narrow_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, size_t n, int vec)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    if (vec) {
        for (size_t u = (size_t)blockIdx.x * blockDim.x + threadIdx.x; u < n / 8; u += stride) {
            const float4 a = reinterpret_cast<const float4*>(in)[2 * u], b = reinterpret_cast<const float4*>(in)[2 * u + 1];
            reinterpret_cast<uint4*>(out)[u] =
                make_uint4(pack2_bf16(a.x, a.y), pack2_bf16(a.z, a.w), pack2_bf16(b.x, b.y), pack2_bf16(b.z, b.w));
        }
    } else {
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) out[i] = __float2bfloat16_rn(in[i]);
    }
}

int launch_widen(const void* in, float* out, size_t n, cudaStream_t st)
{
    const int vec = ((reinterpret_cast<uintptr_t>(in) & 15) == 0 && n % 8 == 0) ? 1 : 0;
    const size_t items = vec ? n / 8 : n;
    const int blocks = (int)std::min<size_t>((items + 255) / 256, (size_t)sm_count() * 8);
    widen_bf16_kernel<<<blocks > 0 ? blocks : 1, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(in), out, n, vec);
    return check_launch();
}

int launch_narrow(const float* in, void* out, size_t n, cudaStream_t st)
{
    const int vec = ((reinterpret_cast<uintptr_t>(out) & 15) == 0 && n % 8 == 0) ? 1 : 0;
    const size_t items = vec ? n / 8 : n;
    const int blocks = (int)std::min<size_t>((items + 255) / 256, (size_t)sm_count() * 8);
    narrow_bf16_kernel<<<blocks > 0 ? blocks : 1, 256, 0, st>>>(in, static_cast<__nv_bfloat16*>(out), n, vec);
    return check_launch();
}

// Whether the wavefront kernel itself reads and writes the bfloat16 images (no conversion pass, no fp32 copy).
bool bf16_in_kernel(int B, int C, int H, int W, int k, bool bwd, bool with_gw)
{
    if (resolve_path(B, C, H, W, k) != INVCONV_PATH_WARP) return false;
    const WarpPlan pl = plan_warp(B, C, H, W, k, bwd);
    if (!pl.ok || pl.glb || ((size_t)C * H * W) % 8 != 0) return false;
    if (bwd && with_gw) {
        const GradWSmallPlan gs = gradw_small_plan(B, C, H, W, k);
        if (gradw_separate(pl, gs, C, k)) return false;
    }
    return true;
}

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

// The path's own workspace inside the storage variant's workspace (what follows it are the fp32 copies of a composed call).
size_t bf16_ws_need(int path, int B, int C, int H, int W, int k)
{
    return up256(std::max<size_t>(workspace_bytes_for(path, B, C, H, W, k), INVCONV_WS_CONTROL_BYTES));
}

}  // namespace

namespace invconv_internal {

// The layer with its flow-step neighbours inside the warp-family kernel; INVCONV_UNSUPPORTED where that family
// (or its shared-memory mode) does not serve the shape -- the caller then composes the step from separate kernels.
int warp_step_forward(const float* y, const float* w, const float* s, const float* b, const float* V, float* x, float* u,
                      Geom g, void* ws, cudaStream_t st)
{
    if (resolve_path(g.B, g.C, g.H, g.W, g.k) != INVCONV_PATH_WARP) return INVCONV_UNSUPPORTED;
    WarpMix mix;
    mix.V = V; mix.s = s; mix.b = b; mix.u_out = u;
    return launch_warp(false, y, w, x, nullptr, nullptr, g, ws, st, &mix);
}

int warp_step_backward(const float* grad_u, const float* x, const float* w, const float* s, const float* V,
                       float* grad_y, float* grad_w, Geom g, void* ws, cudaStream_t st)
{
    if (resolve_path(g.B, g.C, g.H, g.W, g.k) != INVCONV_PATH_WARP) return INVCONV_UNSUPPORTED;
    WarpMix mix;
    mix.V = V; mix.s = s; mix.grad_in = true;
    return launch_warp(true, grad_u, w, grad_y, x, grad_w, g, ws, st, &mix);
}

}  // namespace invconv_internal

extern "C" {

size_t invconv_workspace_bytes(int B, int C, int H, int W, int k)
{
    if (check_shape(B, C, H, W, k) != INVCONV_OK) return 0;
    return workspace_bytes_for(resolve_path(B, C, H, W, k), B, C, H, W, k);
}

int invconv_forward_ws(const float* y, const float* w, float* x, int B, int C, int H, int W, int k,
                       void* workspace, size_t workspace_bytes, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B == 0) return w ? INVCONV_OK : INVCONV_BAD_ARG;
    if (!y || !w || !x || y == x) return INVCONV_BAD_ARG;
    const int path = resolve_path(B, C, H, W, k);
    const size_t need = workspace_bytes_for(path, B, C, H, W, k);
    if (need > 0 && (!workspace || workspace_bytes < need)) return INVCONV_WORKSPACE_TOO_SMALL;
    return launch_forward(path, y, w, x, Geom{B, C, H, W, k}, workspace, workspace_bytes, as_stream(stream));
}

int invconv_backward_ws(const float* grad_x, const float* x, const float* w, float* grad_y, float* grad_w,
                        int B, int C, int H, int W, int k, void* workspace, size_t workspace_bytes, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B == 0) {
        if (!w) return INVCONV_BAD_ARG;
        if (grad_w && cudaMemsetAsync(grad_w, 0, sizeof(float) * C * C * k * k, as_stream(stream)) != cudaSuccess) {
            cudaGetLastError();
            return INVCONV_CUDA_ERROR;
        }
        return INVCONV_OK;
    }
    if (!grad_x || !x || !w || !grad_y || grad_x == grad_y || x == grad_y) return INVCONV_BAD_ARG;
    const int path = resolve_path(B, C, H, W, k);
    const size_t need = workspace_bytes_for(path, B, C, H, W, k);
    if (need > 0 && (!workspace || workspace_bytes < need)) return INVCONV_WORKSPACE_TOO_SMALL;
    return launch_backward(path, grad_x, x, w, grad_y, grad_w, Geom{B, C, H, W, k}, workspace, workspace_bytes,
                           as_stream(stream));
}

int invconv_forward(const float* y, const float* w, float* x, int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B > 0 && (!y || !w || !x || y == x)) return INVCONV_BAD_ARG;
    StreamScratch sc;
    const size_t need = B > 0 ? workspace_bytes_for(resolve_path(B, C, H, W, k), B, C, H, W, k) : 0;
    const int ra = sc.acquire(need, as_stream(stream));
    if (ra) return ra;
    return invconv_forward_ws(y, w, x, B, C, H, W, k, sc.p, need, stream);
}

int invconv_backward(const float* grad_x, const float* x, const float* w, float* grad_y, float* grad_w,
                     int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B > 0 && (!grad_x || !x || !w || !grad_y || grad_x == grad_y || x == grad_y)) return INVCONV_BAD_ARG;
    StreamScratch sc;
    const size_t need = B > 0 ? workspace_bytes_for(resolve_path(B, C, H, W, k), B, C, H, W, k) : 0;
    const int ra = sc.acquire(need, as_stream(stream));
    if (ra) return ra;
    return invconv_backward_ws(grad_x, x, w, grad_y, grad_w, B, C, H, W, k, sc.p, need, stream);
}

int invconv_bf16_in_kernel(int B, int C, int H, int W, int k, int backward, int with_grad_w)
{
    if (check_shape(B, C, H, W, k) != INVCONV_OK || B == 0) return 0;
    return bf16_in_kernel(B, C, H, W, k, backward != 0, with_grad_w != 0) ? 1 : 0;
}

size_t invconv_bf16_workspace_bytes(int B, int C, int H, int W, int k)
{
    if (check_shape(B, C, H, W, k) != INVCONV_OK || B == 0) return 0;
    const size_t need = bf16_ws_need(resolve_path(B, C, H, W, k), B, C, H, W, k);
    const bool in_kernel = bf16_in_kernel(B, C, H, W, k, false, false) && bf16_in_kernel(B, C, H, W, k, true, true);
    return need + (in_kernel ? 0 : 3 * up256((size_t)B * C * H * W * sizeof(float)));
}

int invconv_forward_bf16_ws(const void* y, const float* w, void* x, int B, int C, int H, int W, int k,
                            void* workspace, size_t workspace_bytes, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B == 0) return w ? INVCONV_OK : INVCONV_BAD_ARG;
    if (!y || !w || !x || y == x) return INVCONV_BAD_ARG;
    const cudaStream_t st = as_stream(stream);
    const Geom g{B, C, H, W, k};
    const int path = resolve_path(B, C, H, W, k);
    const size_t need = bf16_ws_need(path, B, C, H, W, k);
    if (!workspace || workspace_bytes < need) return INVCONV_WORKSPACE_TOO_SMALL;
    if (path == INVCONV_PATH_WARP) {
        const int rw = launch_warp(false, static_cast<const float*>(y), w, static_cast<float*>(x), nullptr, nullptr, g, workspace, st,
                                   nullptr, nullptr, LogdetFuse{}, true);
        if (rw != INVCONV_UNSUPPORTED) return rw;
    }
    const size_t n = (size_t)B * C * H * W, act = up256(n * sizeof(float));
    if (workspace_bytes < need + 2 * act) return INVCONV_WORKSPACE_TOO_SMALL;
    float* y32 = reinterpret_cast<float*>(static_cast<char*>(workspace) + need);
    float* x32 = reinterpret_cast<float*>(static_cast<char*>(workspace) + need + act);
    int r = launch_widen(y, y32, n, st);
    if (!r) r = launch_forward(path, y32, w, x32, g, workspace, need, st);
    if (!r) r = launch_narrow(x32, x, n, st);
    return r;
}

int invconv_backward_bf16_ws(const void* grad_x, const void* x, const float* w, void* grad_y, float* grad_w,
                             int B, int C, int H, int W, int k, void* workspace, size_t workspace_bytes, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    const cudaStream_t st = as_stream(stream);
    if (B == 0) {
        if (!w) return INVCONV_BAD_ARG;
        if (grad_w && cudaMemsetAsync(grad_w, 0, sizeof(float) * C * C * k * k, st) != cudaSuccess) {
            cudaGetLastError();
            return INVCONV_CUDA_ERROR;
        }
        return INVCONV_OK;
    }
    if (!grad_x || !x || !w || !grad_y || grad_x == grad_y || x == grad_y) return INVCONV_BAD_ARG;
    const Geom g{B, C, H, W, k};
    const int path = resolve_path(B, C, H, W, k);
    const size_t need = bf16_ws_need(path, B, C, H, W, k);
    if (!workspace || workspace_bytes < need) return INVCONV_WORKSPACE_TOO_SMALL;
    if (path == INVCONV_PATH_WARP) {
        const int rw = launch_warp(true, static_cast<const float*>(grad_x), w, static_cast<float*>(grad_y),
                                   static_cast<const float*>(x), grad_w, g, workspace, st, nullptr, nullptr, LogdetFuse{}, true);
        if (rw != INVCONV_UNSUPPORTED) return rw;
    }
    const size_t n = (size_t)B * C * H * W, act = up256(n * sizeof(float));
    if (workspace_bytes < need + 3 * act) return INVCONV_WORKSPACE_TOO_SMALL;
    float* gx32 = reinterpret_cast<float*>(static_cast<char*>(workspace) + need);
    float* x32 = reinterpret_cast<float*>(static_cast<char*>(workspace) + need + act);
    float* gy32 = reinterpret_cast<float*>(static_cast<char*>(workspace) + need + 2 * act);
    int r = launch_widen(grad_x, gx32, n, st);
    if (!r && grad_w) r = launch_widen(x, x32, n, st);
    if (!r) r = launch_backward(path, gx32, x32, w, gy32, grad_w, g, workspace, need, st);
    if (!r) r = launch_narrow(gy32, grad_y, n, st);
    return r;
}

int invconv_forward_bf16(const void* y, const float* w, void* x, int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B == 0) return w ? INVCONV_OK : INVCONV_BAD_ARG;
    if (!y || !w || !x || y == x) return INVCONV_BAD_ARG;
    const bool aligned = ((reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(x)) & 15) == 0;
    const size_t bytes = bf16_ws_need(resolve_path(B, C, H, W, k), B, C, H, W, k) +
                         ((aligned && bf16_in_kernel(B, C, H, W, k, false, false)) ? 0 : 2 * up256((size_t)B * C * H * W * sizeof(float)));
    StreamScratch sc;
    const int ra = sc.acquire(bytes, as_stream(stream));
    if (ra) return ra;
    return invconv_forward_bf16_ws(y, w, x, B, C, H, W, k, sc.p, bytes, stream);
}

int invconv_backward_bf16(const void* grad_x, const void* x, const float* w, void* grad_y, float* grad_w,
                          int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B == 0 || !grad_x || !x || !w || !grad_y || grad_x == grad_y || x == grad_y)
        return invconv_backward_bf16_ws(grad_x, x, w, grad_y, grad_w, B, C, H, W, k, nullptr, 0, stream);
    const bool aligned = ((reinterpret_cast<uintptr_t>(grad_x) | reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(grad_y)) & 15) == 0;
    const size_t bytes = bf16_ws_need(resolve_path(B, C, H, W, k), B, C, H, W, k) +
                         ((aligned && bf16_in_kernel(B, C, H, W, k, true, grad_w != nullptr)) ? 0 : 3 * up256((size_t)B * C * H * W * sizeof(float)));
    StreamScratch sc;
    const int ra = sc.acquire(bytes, as_stream(stream));
    if (ra) return ra;
    return invconv_backward_bf16_ws(grad_x, x, w, grad_y, grad_w, B, C, H, W, k, sc.p, bytes, stream);
}

int masked_conv_forward(const float* x, const float* w, float* y, int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B == 0) return w ? INVCONV_OK : INVCONV_BAD_ARG;
    if (!x || !w || !y || x == y) return INVCONV_BAD_ARG;
    if (g_forced_path.load() != INVCONV_PATH_GENERIC) {
        const int rs = launch_masked_conv_small(x, w, y, Geom{B, C, H, W, k}, as_stream(stream));
        if (rs != INVCONV_UNSUPPORTED) return rs;
        // many channels: the tensor cores (forcing the team family keeps the FMA tile kernel, for comparison)
        const ConvTensorPlan ct = plan_conv_tensor(B, C, H, W, k, kMaxDynSmem, sm_count());
        if (ct.ok && g_forced_path.load() != INVCONV_PATH_TEAM) {
            StreamScratch sc;
            const int ra = sc.acquire(ct.pack_bytes, as_stream(stream));
            if (ra) return ra;
            return invconv_internal::conv_tensor_launch(ct, x, w, y, Geom{B, C, H, W, k}, static_cast<unsigned char*>(sc.p), as_stream(stream));
        }
        const int rt = launch_masked_conv_tile(x, w, y, Geom{B, C, H, W, k}, as_stream(stream));
        if (rt != INVCONV_UNSUPPORTED) return rt;
    }
    const long long total = (long long)B * C * H * W;
    const int blocks = (int)((total + 255) / 256 < 148LL * 16 ? (total + 255) / 256 : 148LL * 16);
    generic_masked_conv_kernel<<<blocks, 256, 0, as_stream(stream)>>>(x, w, y, Geom{B, C, H, W, k}, total);
    return check_launch();
}

int invconv_logdet(const float* w, float* logdet, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(1, C, H, W, k);
    if (rc) return rc;
    if (!w || !logdet) return INVCONV_BAD_ARG;
    logdet_kernel<<<1, 32, 0, as_stream(stream)>>>(w, logdet, C, H, W, k);
    return check_launch();
}

int invconv_forward_logdet(const float* y, const float* w, float* x, float* logdet,
                           int B, int C, int H, int W, int k, void* stream)
{
    if (!logdet) return INVCONV_BAD_ARG;
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (!w) return INVCONV_BAD_ARG;
    if (B > 0 && (!y || !x || y == x)) return INVCONV_BAD_ARG;
    StreamScratch sc;
    const int path = resolve_path(B > 0 ? B : 1, C, H, W, k);
    const size_t need = B > 0 ? workspace_bytes_for(path, B, C, H, W, k) : 0;
    const int ra = sc.acquire(need, as_stream(stream));
    if (ra) return ra;
    return launch_forward(path, y, w, x, Geom{B, C, H, W, k}, sc.p, need, as_stream(stream), logdet);
}

int invconv_backward_logdet(const float* grad_x, const float* x, const float* w, const float* grad_logdet,
                            float* grad_y, float* grad_w, int B, int C, int H, int W, int k, void* stream)
{
    if (!grad_logdet || !grad_w) return INVCONV_BAD_ARG;
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (!w) return INVCONV_BAD_ARG;
    if (B == 0) {
        // no image: grad_w is the log-det's term alone
        if (cudaMemsetAsync(grad_w, 0, sizeof(float) * C * C * k * k, as_stream(stream)) != cudaSuccess) {
            cudaGetLastError();
            return INVCONV_CUDA_ERROR;
        }
        logdet_grad_kernel<<<1, 128, 0, as_stream(stream)>>>(w, grad_logdet, grad_w, C, H, W, k);
        return check_launch();
    }
    if (!grad_x || !x || !grad_y || grad_x == grad_y || x == grad_y) return INVCONV_BAD_ARG;
    StreamScratch sc;
    const int path = resolve_path(B, C, H, W, k);
    const size_t need = workspace_bytes_for(path, B, C, H, W, k);
    const int ra = sc.acquire(need, as_stream(stream));
    if (ra) return ra;
    return launch_backward(path, grad_x, x, w, grad_y, grad_w, Geom{B, C, H, W, k}, sc.p, need, as_stream(stream), grad_logdet);
}

size_t invconv_step_scratch_bytes(int B, int C, int H, int W, int k)
{
    if (check_shape(B, C, H, W, k) != INVCONV_OK) return 0;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t act = up((size_t)B * C * H * W * sizeof(float));
    const size_t wb = up((size_t)C * C * k * k * sizeof(float));
    return up(invconv_workspace_bytes(B, C, H, W, k) + INVCONV_WS_CONTROL_BYTES) + 4 * act + 2 * wb + 256;
}

int invconv_step_host(const float* y_host, const float* w_host, const float* grad_x_host,
                      float* x_host, float* grad_y_host, float* grad_w_host, float* logdet_host,
                      int B, int C, int H, int W, int k,
                      void* device_scratch, size_t device_scratch_bytes, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (!y_host || !w_host || !grad_x_host || !x_host || !grad_y_host || !grad_w_host || !logdet_host || !device_scratch)
        return INVCONV_BAD_ARG;
    if (device_scratch_bytes < invconv_step_scratch_bytes(B, C, H, W, k)) return INVCONV_WORKSPACE_TOO_SMALL;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t act_b = (size_t)B * C * H * W * sizeof(float), act = up(act_b);
    const size_t w_b = (size_t)C * C * k * k * sizeof(float), wb = up(w_b);
    const size_t ws_b = up(invconv_workspace_bytes(B, C, H, W, k) + INVCONV_WS_CONTROL_BYTES);
    char* p = static_cast<char*>(device_scratch);
    void* ws = p;               p += ws_b;
    float* d_y = (float*)p;     p += act;
    float* d_gx = (float*)p;    p += act;
    float* d_x = (float*)p;     p += act;
    float* d_gy = (float*)p;    p += act;
    float* d_w = (float*)p;     p += wb;
    float* d_gw = (float*)p;    p += wb;
    float* d_ld = (float*)p;
    cudaStream_t st = as_stream(stream);
    // The copy of grad_x in and the copy of x out run on a side stream: the device has one copy engine per
    // direction, so x leaves while grad_x arrives and the backward kernels run.  Everything is joined back
    // into `stream` before the call returns, so the caller still synchronises that stream only.
    StepSide* side = act_b ? step_side() : nullptr;
    if (act_b && !side) return INVCONV_CUDA_ERROR;
    std::unique_lock<std::mutex> enqueue_lock;
    if (side) enqueue_lock = std::unique_lock<std::mutex>(side->enqueue);
    cudaMemcpyAsync(d_w, w_host, w_b, cudaMemcpyHostToDevice, st);
    if (act_b) {
        cudaEventRecord(side->start, st);                     // earlier work on `stream` may still use the scratch
        cudaStreamWaitEvent(side->side, side->start, 0);
        cudaMemcpyAsync(d_y, y_host, act_b, cudaMemcpyHostToDevice, st);
        cudaMemcpyAsync(d_gx, grad_x_host, act_b, cudaMemcpyHostToDevice, side->side);
        cudaEventRecord(side->gx_in, side->side);
    }
    // on an error the side stream is still joined back into `stream`, so the caller's stream orders everything
    auto fail = [&](int code) {
        if (act_b) {
            cudaEventRecord(side->x_out, side->side);
            cudaStreamWaitEvent(st, side->x_out, 0);
        }
        return code;
    };
    int r = invconv_forward_ws(d_y, d_w, d_x, B, C, H, W, k, ws, ws_b, stream);
    if (r) return fail(r);
    if (act_b) {
        cudaEventRecord(side->x_ready, st);
        cudaStreamWaitEvent(side->side, side->x_ready, 0);
        cudaMemcpyAsync(x_host, d_x, act_b, cudaMemcpyDeviceToHost, side->side);
        cudaEventRecord(side->x_out, side->side);
        cudaStreamWaitEvent(st, side->gx_in, 0);
    }
    r = invconv_backward_ws(d_gx, d_x, d_w, d_gy, d_gw, B, C, H, W, k, ws, ws_b, stream);
    if (r) return fail(r);
    r = invconv_logdet(d_w, d_ld, C, H, W, k, stream);
    if (r) return fail(r);
    if (act_b) cudaMemcpyAsync(grad_y_host, d_gy, act_b, cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(grad_w_host, d_gw, w_b, cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(logdet_host, d_ld, sizeof(float), cudaMemcpyDeviceToHost, st);
    if (act_b) cudaStreamWaitEvent(st, side->x_out, 0);
    if (cudaGetLastError() != cudaSuccess) return INVCONV_CUDA_ERROR;
    return INVCONV_OK;
}

// ---------------------------------------------------------------- no-allocation backward
// Scratch of invconv_backward_noalloc: part of the module image, one copy per device that loads it.
static __device__ __align__(256) unsigned char g_noalloc_scratch[INVCONV_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::atomic<void*> g_noalloc_ptr[kMaxDevices];

// Device address of the scratch array on the current device.  In host code the array's name is only a
// handle for the runtime, not an address a kernel could use, so the address is asked for once per device.
int noalloc_scratch(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    void* p = g_noalloc_ptr[dev].load();
    if (!p) {
        const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            std::fprintf(stderr, "invconv: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
            cudaGetLastError();
            return INVCONV_CUDA_ERROR;
        }
        g_noalloc_ptr[dev].store(p);
    }
    *out = p;
    return INVCONV_OK;
}
}  // namespace

int invconv_backward_noalloc(const float* grad_x, const float* x, const float* w, float* grad_y, float* grad_w,
                             int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (B == 0) return invconv_backward_ws(grad_x, x, w, grad_y, grad_w, B, C, H, W, k, nullptr, 0, stream);
    if (!grad_x || !x || !w || !grad_y || grad_x == grad_y || x == grad_y) return INVCONV_BAD_ARG;
    if (!plan_warp(B, C, H, W, k, true).ok) return INVCONV_UNSUPPORTED;
    const size_t need = warp_workspace_bytes(B, C, H, W, k);
    if (need > INVCONV_NOALLOC_SCRATCH_BYTES) return INVCONV_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    const int rs = noalloc_scratch(&scratch);
    if (rs) return rs;
    cudaStream_t st = as_stream(stream);
    if (cudaMemsetAsync(scratch, 0, INVCONV_WS_CONTROL_BYTES, st) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    return launch_warp(true, grad_x, w, grad_y, x, grad_w, Geom{B, C, H, W, k}, scratch, st);
}

int invconv_set_path(int path)
{
    if (path < INVCONV_PATH_AUTO || path > INVCONV_PATH_TENSOR) return -1;
    return g_forced_path.exchange(path);
}

int invconv_debug_bounds_info(int* info)
{
    if (!info) return INVCONV_BAD_ARG;
    return invconv_internal::tensor_bounds_info(info);
}

int invconv_selftest_bounds(void* stream)
{
    return invconv_internal::tensor_selftest_bounds(as_stream(stream));
}

int invconv_set_option(int option, int value)
{
    if (option < 0 || option >= INVCONV_OPT_COUNT) return -1;
    return g_opt[option].exchange(value);
}

int invconv_selftest_wait_timeout(unsigned limit_cycles, void* stream)
{
    if (limit_cycles < 1 || limit_cycles > (1u << 24)) return INVCONV_BAD_ARG;
    probe_wait_timeout<<<1, 64, 0, as_stream(stream)>>>(limit_cycles);
    return check_launch();
}

int invconv_path_for(int B, int C, int H, int W, int k)
{
    if (check_shape(B, C, H, W, k) != INVCONV_OK) return -1;
    return auto_path(B, C, H, W, k);
}

int invconv_cluster_size_for(int B, int C, int H, int W, int k)
{
    if (check_shape(B, C, H, W, k) != INVCONV_OK) return -1;
    switch (auto_path(B, C, H, W, k)) {
    case INVCONV_PATH_TENSOR: return tensor_plan(B, C, H, W, k).R;
    case INVCONV_PATH_TEAM: return team_plan(B, C, H, W, k).R;
    default: return 1;
    }
}

int invconv_get_status(void* stream, int* device_status_out)
{
    if (!device_status_out) return INVCONV_BAD_ARG;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    int v = 0, vt = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    if (v != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
    }
    if (invconv_internal::tensor_read_clear_status(&vt) != INVCONV_OK) return INVCONV_CUDA_ERROR;
    int vf = 0;
    if (invconv_internal::flow_read_clear_status(&vf) != INVCONV_OK) return INVCONV_CUDA_ERROR;
    if (vf > vt) vt = vf;
    *device_status_out = v > vt ? v : vt;
    return INVCONV_OK;
}

int invconv_probe_step_latency(int mechanism, int steps, unsigned long long* cycles_out, void* stream)
{
    if (!cycles_out || steps < 1 || steps > (1 << 20)) return INVCONV_BAD_ARG;
    cudaStream_t st = as_stream(stream);
    switch (mechanism) {
    case 0: probe_shuffle_chain<<<1, 32, 0, st>>>(steps, cycles_out); break;
    case 1: probe_smem_chain<<<1, 256, 0, st>>>(steps, cycles_out); break;
    case 2: {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2); cfg.blockDim = dim3(128); cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, probe_cluster_chain, steps, cycles_out) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
        break;
    }
    default: return INVCONV_BAD_ARG;
    }
    return check_launch();
}

const char* invconv_status_string(int status)
{
    switch (status) {
    case INVCONV_OK: return "ok";
    case INVCONV_BAD_ARG: return "bad argument";
    case INVCONV_UNSUPPORTED: return "unsupported shape or path";
    case INVCONV_CUDA_ERROR: return "CUDA error";
    case INVCONV_TIMEOUT: return "device-side wait timed out";
    case INVCONV_WORKSPACE_TOO_SMALL: return "workspace too small";
    case INVCONV_BOUNDS: return "checked accessor caught an index out of bounds (debug-bounds build)";
    default: return "unknown status";
    }
}

unsigned long long invconv_kernel_launch_count(void) { return g_kernel_launches.load(); }

int invconv_version(void) { return 100; }

}  // extern "C"

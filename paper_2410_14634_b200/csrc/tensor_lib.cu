// Launch side of the TENSOR family (tcgen05 wavefront): its own translation unit so that the tensor-core
// kernels build independently of the other families.
#include <cuda_runtime.h>

#include <cstdio>

#include "invconv.h"

#include "common.cuh"
#include "lib_internal.h"
#include "team_kernels.cuh"      // team_solve_kernel: the kernel transform L^-1 W_delta
#include "tensor_kernels.cuh"
#include "gradw_tensor.cuh"
#include "conv_tensor.cuh"

using namespace invconv;

namespace {

template <int CG, int K>
int launch_tensor_inst(const TensorPlan& pl, const TensorParams& prm, cudaStream_t st)
{
    auto kern = tensor_wavefront_kernel<CG, K>;
    const int rc = invconv_internal::set_smem_limit(kern, pl.smem);
    if (rc) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.ncl * pl.R);
    cfg.blockDim = dim3(kTensorThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    // Programmatic dependent launch: the CTAs set themselves up (barriers, tensor memory, the right-hand side)
    // while the kernel transform still runs; they wait for it (griddepcontrol.wait) before reading its output.
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = pl.R; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: tensor launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return invconv_internal::check_launch();
}

}  // namespace

namespace invconv_internal {

int tensor_launch(const TensorPlan& pl, bool bwd, const float* rhs, const float* w, float* out, Geom g,
                  float* A, unsigned char* wop, cudaStream_t st, float* logdet_out)
{
    if (((reinterpret_cast<uintptr_t>(rhs) | reinterpret_cast<uintptr_t>(out)) & 15) != 0) return INVCONV_UNSUPPORTED;
    {
        if (team_solve_launch(bwd, w, A, g.C, g.k, wop, pl.NCH, pl.wbytes, logdet_out, g.H * g.W, st) != cudaSuccess) {
            cudaGetLastError();
            return INVCONV_CUDA_ERROR;
        }
        const int rl = check_launch();
        if (rl) return rl;
    }
    TensorParams prm;
    prm.rhs = rhs; prm.out = out; prm.wop = wop;
    prm.B = g.B; prm.C = g.C; prm.H = g.H; prm.W = g.W; prm.K = g.k;
    prm.R = pl.R; prm.I = pl.I; prm.HP = pl.HP; prm.S = pl.S; prm.ngroups = pl.ngroups; prm.ncl = pl.ncl;
    prm.rot = bwd ? 1 : 0;
    prm.tmem_cols = pl.tmem_cols; prm.wbytes = pl.wbytes;
    prm.off_stage = pl.off_stage; prm.off_x = pl.off_x; prm.off_y = pl.off_y; prm.off_recv = pl.off_recv;
    prm.off_bar = pl.off_bar; prm.stage_img = pl.stage_img;
#define X(CG_, K_) if (g.C == 16 * CG_ && g.k == K_) return launch_tensor_inst<CG_, K_>(pl, prm, st);
    X(1, 2) X(1, 3) X(1, 4) X(1, 5) X(2, 2) X(2, 3) X(2, 4) X(2, 5)
    X(3, 2) X(3, 3) X(3, 4) X(3, 5) X(4, 2) X(4, 3) X(4, 4) X(4, 5)
#undef X
    return INVCONV_UNSUPPORTED;
}

int gradw_tensor_launch(const GradWTensorPlan& pl, const float* gy, const float* x, float* partials, Geom g, cudaStream_t st)
{
    auto kern = gradw_tensor_kernel;
    const int rc = set_smem_limit(kern, pl.smem);
    if (rc) return rc;
    GradWTensorParams prm;
    prm.gy = gy; prm.x = x; prm.partials = partials;
    prm.B = g.B; prm.C = g.C; prm.H = g.H; prm.W = g.W; prm.K = g.k;
    prm.RB = pl.RB; prm.Wp = pl.Wp; prm.nbands = pl.nbands; prm.S = pl.S; prm.nk = pl.nk;
    prm.tmem_cols = pl.tmem_cols; prm.planeA = pl.planeA; prm.planeB = pl.planeB; prm.stage_bytes = pl.stage_bytes;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.grid);
    cfg.blockDim = dim3(kGradWTensorProducers + 32 * (g.k < kGradWTensorIssuers ? g.k : kGradWTensorIssuers));
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // set-up overlaps the tail of the solve
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: grad_w tensor launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return check_launch();
}

int conv_tensor_launch(const ConvTensorPlan& pl, const float* x, const float* w, float* y, Geom g, unsigned char* pack, cudaStream_t st)
{
    const int total = g.k * g.k * (g.C / 8) * g.C;
    conv_pack_kernel<<<(total + 255) / 256, 256, 0, st>>>(w, pack, g.C, g.k);
    int rc = check_launch();
    if (rc) return rc;
    auto kern = conv_tensor_kernel;
    rc = set_smem_limit(kern, pl.smem);
    if (rc) return rc;
    ConvTensorParams prm;
    prm.x = x; prm.pack = pack; prm.y = y;
    prm.B = g.B; prm.C = g.C; prm.H = g.H; prm.W = g.W; prm.K = g.k;
    prm.RB = pl.RB; prm.Wp = pl.Wp; prm.nbands = pl.nbands; prm.ntiles = pl.ntiles; prm.slots = pl.slots; prm.spi = pl.spi;
    prm.tmem_cols = pl.tmem_cols; prm.x_bytes = pl.x_bytes; prm.wstage_bytes = pl.wstage_bytes;
    prm.off_w = pl.off_w; prm.off_bar = pl.off_bar;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.grid);
    cfg.blockDim = dim3(kConvTensorThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // x is staged while the kernel is being packed
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
    if (e != cudaSuccess) {
        std::fprintf(stderr, "invconv: tensor convolution launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return check_launch();
}

#ifdef INVCONV_DEBUG_BOUNDS
namespace { __global__ void bounds_selftest_kernel() { (void)INVCONV_CHECKED(5, 3, 999); } }
#endif

int tensor_selftest_bounds(cudaStream_t st)
{
#ifdef INVCONV_DEBUG_BOUNDS
    bounds_selftest_kernel<<<1, 1, 0, st>>>();
    return check_launch();
#else
    (void)st;
    return INVCONV_UNSUPPORTED;
#endif
}

int tensor_bounds_info(int* info)
{
#ifdef INVCONV_DEBUG_BOUNDS
    int a[4] = {0, 0, 0, 0}, b[4] = {0, 0, 0, 0};
    const int zero[4] = {0, 0, 0, 0};
    if (cudaMemcpyFromSymbol(a, g_bounds_record, sizeof(a)) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    cudaMemcpyToSymbol(g_bounds_record, zero, sizeof(zero));
    if (flow_bounds_info(b) != INVCONV_OK) return INVCONV_CUDA_ERROR;
    const int* first = a[0] ? a : b;
    info[0] = first[0]; info[1] = first[1]; info[2] = first[2]; info[3] = a[3] + b[3];
    return INVCONV_OK;
#else
    (void)info;
    return INVCONV_UNSUPPORTED;
#endif
}

int tensor_read_clear_status(int* status_out)
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

}  // namespace invconv_internal

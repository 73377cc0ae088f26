// C ABI of the inverse-convolution library: argument checks, kernel-family
// dispatch and launches.  Every step of the path runs in the kernels included
// below; nothing here computes.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>
#include <cstring>

#include "invconv.h"

#include "common.cuh"
#include "generic_kernels.cuh"
#include "probe_kernels.cuh"

using namespace invconv;

namespace {

std::atomic<int> g_forced_path{INVCONV_PATH_AUTO};
std::atomic<unsigned long long> g_kernel_launches{0};

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

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

int check_shape(int B, int C, int H, int W, int k)
{
    if (B < 0 || C < 1 || H < 1 || W < 1 || k < 1) return INVCONV_BAD_ARG;
    if (k > INVCONV_MAX_K || C > INVCONV_MAX_C) return INVCONV_UNSUPPORTED;
    const long long e = (long long)B * C * H * W;
    if (e >= (1LL << 31)) return INVCONV_UNSUPPORTED;
    return INVCONV_OK;
}

int auto_path(int B, int C, int H, int W, int k)
{
    (void)B; (void)C; (void)H; (void)W; (void)k;
    return INVCONV_PATH_GENERIC;
}

int resolve_path(int B, int C, int H, int W, int k)
{
    const int forced = g_forced_path.load();
    return forced == INVCONV_PATH_AUTO ? auto_path(B, C, H, W, k) : forced;
}

size_t workspace_bytes_for(int path, int B, int C, int H, int W, int k)
{
    (void)path; (void)B; (void)C; (void)H; (void)W; (void)k;
    return 0;
}

int launch_forward(int path, const float* y, const float* w, float* x, Geom g,
                   void* ws, size_t ws_bytes, cudaStream_t st)
{
    (void)ws; (void)ws_bytes;
    if (g.B == 0) return INVCONV_OK;
    switch (path) {
    case INVCONV_PATH_GENERIC:
        generic_wavefront_kernel<false><<<g.B, 256, 0, st>>>(y, w, x, g);
        return check_launch();
    default:
        return INVCONV_UNSUPPORTED;
    }
}

int launch_backward(int path, const float* gx, const float* x, const float* w, float* gy, float* gw, Geom g,
                    void* ws, size_t ws_bytes, cudaStream_t st)
{
    (void)ws; (void)ws_bytes;
    switch (path) {
    case INVCONV_PATH_GENERIC: {
        if (g.B > 0) {
            generic_wavefront_kernel<true><<<g.B, 256, 0, st>>>(gx, w, gy, g);
            const int rc = check_launch();
            if (rc) return rc;
        }
        if (gw) {
            generic_grad_w_kernel<<<g.C * g.C * g.k * g.k, 128, 0, st>>>(gy, x, gw, g);
            return check_launch();
        }
        return INVCONV_OK;
    }
    default:
        return INVCONV_UNSUPPORTED;
    }
}

// Stream-ordered scratch for the entry points that take no workspace.
struct StreamScratch {
    void* p = nullptr;
    cudaStream_t st;
    int acquire(size_t bytes, cudaStream_t s) {
        st = s;
        if (bytes == 0) return INVCONV_OK;
        if (cudaMallocAsync(&p, bytes, st) != cudaSuccess) { cudaGetLastError(); p = nullptr; return INVCONV_CUDA_ERROR; }
        if (cudaMemsetAsync(p, 0, INVCONV_WS_CONTROL_BYTES, st) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
        return INVCONV_OK;
    }
    ~StreamScratch() { if (p) cudaFreeAsync(p, st); }
};

}  // namespace

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
    StreamScratch sc;
    const size_t need = workspace_bytes_for(resolve_path(B, C, H, W, k), B, C, H, W, k);
    const int ra = sc.acquire(need, as_stream(stream));
    if (ra) return ra;
    return invconv_forward_ws(y, w, x, B, C, H, W, k, sc.p, need, stream);
}

int invconv_backward(const float* grad_x, const float* x, const float* w, float* grad_y, float* grad_w,
                     int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    StreamScratch sc;
    const size_t need = workspace_bytes_for(resolve_path(B, C, H, W, k), B, C, H, W, k);
    const int ra = sc.acquire(need, as_stream(stream));
    if (ra) return ra;
    return invconv_backward_ws(grad_x, x, w, grad_y, grad_w, B, C, H, W, k, sc.p, need, stream);
}

int masked_conv_forward(const float* x, const float* w, float* y, int B, int C, int H, int W, int k, void* stream)
{
    const int rc = check_shape(B, C, H, W, k);
    if (rc) return rc;
    if (!x || !w || !y || x == y) return INVCONV_BAD_ARG;
    if (B == 0) return INVCONV_OK;
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
    cudaMemcpyAsync(d_w, w_host, w_b, cudaMemcpyHostToDevice, st);
    if (act_b) {
        cudaMemcpyAsync(d_y, y_host, act_b, cudaMemcpyHostToDevice, st);
        cudaMemcpyAsync(d_gx, grad_x_host, act_b, cudaMemcpyHostToDevice, st);
    }
    int r = invconv_forward_ws(d_y, d_w, d_x, B, C, H, W, k, ws, ws_b, stream);
    if (r) return r;
    r = invconv_backward_ws(d_gx, d_x, d_w, d_gy, d_gw, B, C, H, W, k, ws, ws_b, stream);
    if (r) return r;
    r = invconv_logdet(d_w, d_ld, C, H, W, k, stream);
    if (r) return r;
    if (act_b) {
        cudaMemcpyAsync(x_host, d_x, act_b, cudaMemcpyDeviceToHost, st);
        cudaMemcpyAsync(grad_y_host, d_gy, act_b, cudaMemcpyDeviceToHost, st);
    }
    cudaMemcpyAsync(grad_w_host, d_gw, w_b, cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(logdet_host, d_ld, sizeof(float), cudaMemcpyDeviceToHost, st);
    if (cudaGetLastError() != cudaSuccess) return INVCONV_CUDA_ERROR;
    return INVCONV_OK;
}

int invconv_set_path(int path)
{
    if (path < INVCONV_PATH_AUTO || path > INVCONV_PATH_TEAM) return -1;
    return g_forced_path.exchange(path);
}

int invconv_path_for(int B, int C, int H, int W, int k)
{
    if (check_shape(B, C, H, W, k) != INVCONV_OK) return -1;
    return auto_path(B, C, H, W, k);
}

int invconv_get_status(void* stream, int* device_status_out)
{
    if (!device_status_out) return INVCONV_BAD_ARG;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return INVCONV_CUDA_ERROR; }
    if (v != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
    }
    *device_status_out = v;
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
    default: return "unknown status";
    }
}

unsigned long long invconv_kernel_launch_count(void) { return g_kernel_launches.load(); }

int invconv_version(void) { return 100; }

}  // extern "C"

// Host-side declarations shared by the translation units of the library (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>

#include <cstdio>

#include "common.cuh"
#include "tensor_plan.h"

namespace invconv_internal {

constexpr size_t kMaxDynSmem = 226 * 1024;   // 227 KiB per CTA minus the kernels' static shared memory

// Counts the launch and turns cudaGetLastError into a status code.
int check_launch();

// Stream-ordered device scratch from the library's own memory pool; release with cudaFreeAsync on the same stream.
int scratch_alloc(void** out, size_t bytes, cudaStream_t st);

// Multiprocessors of the current device (cached per device).
int sm_count();

template <typename Kern>
inline int set_smem_limit(Kern kern, size_t smem)
{
    // the 48 KB a kernel may use without opting in include its static shared memory (up to a few KB in some kernels)
    if (smem <= 40 * 1024) return INVCONV_OK;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return INVCONV_CUDA_ERROR;
    }
    return INVCONV_OK;
}

// invconv_lib.cu: forward / backward of the layer with Actnorm and the 1x1 convolution applied inside the warp-family
// kernel (see flow_step_lib.cu); INVCONV_UNSUPPORTED where that kernel does not serve the shape.
int warp_step_forward(const float* y, const float* w, const float* s, const float* b, const float* V, float* x, float* u,
                      invconv::Geom g, void* ws, cudaStream_t st);
int warp_step_backward(const float* grad_u, const float* x, const float* w, const float* s, const float* V,
                       float* grad_y, float* grad_w, invconv::Geom g, void* ws, cudaStream_t st);

// tensor_lib.cu: the tcgen05 wavefront (kernel transform into A, operand packing into wop, solve).
int tensor_launch(const invconv::TensorPlan& pl, bool bwd, const float* rhs, const float* w, float* out,
                  invconv::Geom g, float* A, unsigned char* wop, cudaStream_t st, float* logdet_out = nullptr);
int tensor_read_clear_status(int* status_out);
int flow_read_clear_status(int* status_out);              // flow_step_lib.cu's copy of the status word
int tensor_bounds_info(int* info);                        // debug-bounds build: first violation and count (both units)
int flow_bounds_info(int* info);
int tensor_selftest_bounds(cudaStream_t st);

// tensor_lib.cu: y = f(x) on the tensor cores; `pack` is device scratch of pl.pack_bytes bytes.
int conv_tensor_launch(const invconv::ConvTensorPlan& pl, const float* x, const float* w, float* y, invconv::Geom g,
                       unsigned char* pack, cudaStream_t st);

// tensor_lib.cu: the tcgen05 correlation kernel of grad_w; partial sums [pl.S][k*k][C][C] go to `partials`.
int gradw_tensor_launch(const invconv::GradWTensorPlan& pl, const float* gy, const float* x, float* partials,
                        invconv::Geom g, cudaStream_t st);

}  // namespace invconv_internal

// Shared declarations of the inverse-convolution kernels (device side).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "invconv.h"

namespace invconv {

// Problem geometry handed to every kernel.
struct Geom {
    int B, C, H, W, k;
};

// Device-side status word (one per device that loads the library and per translation unit).  Kernels
// only ever raise it (atomicMax) when a bounded wait gives up; invconv_get_status reads every copy.
static __device__ int g_device_status = 0;

__device__ __forceinline__ void raise_status(int code) { atomicMax(&g_device_status, code); }

// Checked accessors (development build, -DINVCONV_DEBUG_BOUNDS; stands in for a memory checker): an index
// that is about to be used goes through INVCONV_CHECKED(index, limit, site).  In the debug build an index outside
// [0, limit) is recorded (the first one with its site number, index and limit; a count of all), the status word
// is raised to INVCONV_BOUNDS and the macro yields false, so the caller skips the access instead of faulting.
// In the normal build the macro is the constant true and costs nothing.
#ifdef INVCONV_DEBUG_BOUNDS
static __device__ int g_bounds_record[4] = {0, 0, 0, 0};      // site, index, limit, count
__device__ __forceinline__ bool bounds_ok(long long i, long long n, int site)
{
    if (i >= 0 && i < n) return true;
    atomicAdd(&g_bounds_record[3], 1);
    if (atomicCAS(&g_bounds_record[0], 0, site) == 0) { g_bounds_record[1] = (int)i; g_bounds_record[2] = (int)n; }
    raise_status(INVCONV_BOUNDS);
    return false;
}
#define INVCONV_CHECKED(i, n, site) (::invconv::bounds_ok((long long)(i), (long long)(n), (site)))
#else
#define INVCONV_CHECKED(i, n, site) (true)
#endif

// Index helpers.  Activations are [B][C][H][W]; kernels [C][C][k][k].
__host__ __device__ __forceinline__ size_t act_index(int n, int c, int h, int w, int C, int H, int W) {
    return (((size_t)n * C + c) * H + h) * W + w;
}
__host__ __device__ __forceinline__ int w_index(int co, int ci, int a, int b, int C, int k) {
    return ((co * C + ci) * k + a) * k + b;
}

// Round to nearest tf32 (10 explicit mantissa bits; the low 13 bits of the result are zero).
__device__ __forceinline__ float tf32_hi(float v)
{
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
    return __uint_as_float(u);
}

// The log-det folded into the training step (Section 4: the layer's log-det enters the likelihood).
// Forward: kernels that are given `out` write H*W*sum_c log|w[c][c][k-1][k-1]|, accumulated in double by one warp.
// Backward: the kernels that write the final grad_w add  grad_logdet * H*W / w[c][c][k-1][k-1]  on the channel
// diagonal of the tap that multiplies the pixel itself (tap index 0 in (dh, dw) order).
struct LogdetFuse {
    const float* grad_logdet = nullptr;   // one float: upstream gradient with respect to the log-det (nullptr: none)
    const float* w = nullptr;             // [C][C][k][k]
    int HW = 0;
};

__device__ __forceinline__ void warp_logdet(const float* __restrict__ wgt, float* __restrict__ out, int C, int HW, int k, int lane)
{
    double s = 0.0;
    for (int c = lane; c < C; c += 32) s += log(fabs((double)__ldg(wgt + w_index(c, c, k - 1, k - 1, C, k))));
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) out[0] = (float)((double)HW * s);
}

// value of grad_w at (co, ci, tap) given the correlation sum `s` (grad_w = -s on the mask, 0 outside it)
__device__ __forceinline__ float finish_grad_w(float s, int co, int ci, int tap, int C, int k, const LogdetFuse& ld)
{
    if (tap == 0 && ci > co) return 0.f;
    float v = -s;
    if (tap == 0 && ci == co && ld.grad_logdet != nullptr)
        v += (__ldg(ld.grad_logdet) * (float)ld.HW) / __ldg(ld.w + w_index(co, co, k - 1, k - 1, C, k));
    return v;
}

// Upper bound on polls of any device-side wait before it gives up.
constexpr unsigned kMaxSpins = 1u << 22;

// Sum v[0..31] over the 32 lanes; lane i returns the total of entry i.
__device__ __forceinline__ float transpose_reduce32(float (&v)[32], int lane)
{
#pragma unroll
    for (int off = 16, n = 32; off >= 1; off >>= 1, n >>= 1) {
        const bool hi = (lane & off) != 0;
#pragma unroll
        for (int q = 0; q < n / 2; ++q) {
            const float send = hi ? v[q] : v[q + n / 2];
            const float keep = hi ? v[q + n / 2] : v[q];
            v[q] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    return v[0];
}

}  // namespace invconv

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

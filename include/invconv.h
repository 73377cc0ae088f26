/*
 * invconv.h -- C ABI of the B200 (sm_100a) library for the inverse of a masked,
 * top-left-padded k x k multi-channel convolution and its backpropagation
 * (Nagar & Varma, "Parallel Backpropagation for Inverse of a Convolution with
 * Application to Normalizing Flows").
 *
 * Conventions shared by every call
 * --------------------------------
 *  - Unless a parameter is named *_host, every pointer is a DEVICE pointer to
 *    contiguous fp32.  Activations x, y, grad_x, grad_y are [B][C][H][W];
 *    kernels w, grad_w are [C_out][C_in][k][k].
 *  - The kernel entry that multiplies pixel (h-dh, w-dw) in output pixel (h, w)
 *    is w[co][ci][k-1-dh][k-1-dw], 0 <= dh, dw < k (Eq. 1; Algorithm 1's index
 *    K[c, k_c, k_H-k_h-1, k_W-k_w-1]).  Pixels with a negative coordinate are
 *    the zero padding on the top and left (Section 3).
 *  - The bottom-right entry w[:, :, k-1, k-1] multiplies the output pixel
 *    itself.  It is masked to ci <= co; its channel diagonal must be non-zero
 *    (the paper fixes it to 1).  Values stored at ci > co on that tap are never
 *    read.  A zero diagonal yields inf/nan, as in the paper where invertibility
 *    is assumed.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Calls only enqueue work on `stream`: they never synchronise and
 *    never free or keep caller memory.  The library is re-entrant; calls that
 *    share a workspace must be ordered on one stream.
 *  - Ownership: the caller owns every buffer.  Outputs are overwritten, never
 *    accumulated into.  Inputs and outputs must not alias.
 *  - Return value: an invconv_status (0 = success).  Nothing throws or aborts.
 *    Pointers need no particular alignment: unaligned buffers take scalar
 *    loads.
 *  - Limits: 1 <= k <= INVCONV_MAX_K, 1 <= C <= INVCONV_MAX_C, B, H, W >= 1,
 *    B*C*H*W < 2^31.  B == 0 is a successful no-op (grad_w is still zeroed).
 */
#ifndef INVCONV_H_
#define INVCONV_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define INVCONV_MAX_K 11   /* largest kernel in the paper's ablation (Supplementary, kernel-size table) */
#define INVCONV_MAX_C 128

enum invconv_status {
    INVCONV_OK = 0,
    INVCONV_BAD_ARG = 1,          /* NULL pointer, non-positive size, aliasing in == out */
    INVCONV_UNSUPPORTED = 2,      /* k or C beyond the compiled limits, tensor too large */
    INVCONV_CUDA_ERROR = 3,       /* a launch or runtime call failed (cudaGetLastError) */
    INVCONV_TIMEOUT = 4,          /* a bounded device-side wait gave up (see invconv_get_status) */
    INVCONV_WORKSPACE_TOO_SMALL = 5,
    INVCONV_BOUNDS = 6            /* debug-bounds build only: a checked accessor caught an index outside its array */
};

/* Which kernel family serves a call.  AUTO picks by shape; the others force a
 * family (tests and measurements); a family that cannot serve the shape
 * returns INVCONV_UNSUPPORTED. */
enum invconv_path {
    INVCONV_PATH_AUTO = 0,
    INVCONV_PATH_GENERIC = 1,     /* one CTA per image, operands in global memory, any shape */
    INVCONV_PATH_WARP = 2,        /* warp-shuffle wavefront, image resident in shared memory, small C */
    INVCONV_PATH_TEAM = 3,        /* CTA / cluster per image, register-tiled channel contraction, wide C */
    INVCONV_PATH_TENSOR = 4       /* cluster per group of images, channel contraction on the tcgen05 tensor cores */
};

/* x = f^{-1}(y): the inverse of the masked convolution, by wavefront
 * substitution over the H+W-1 anti-diagonals (Section 3, Eq. 1 solved for
 * x_q; Supplementary "Input Padding and Kernel Masking").
 *   y [B,C,H,W] in, w [C,C,k,k] in, x [B,C,H,W] out.
 * Uses stream-ordered scratch when the shape needs a workspace (see
 * invconv_workspace_bytes), taken from a memory pool the library creates per
 * device on first use and keeps (freed blocks stay cached in it); use the _ws
 * form to supply the scratch yourself. */
int invconv_forward(const float* y, const float* w, float* x,
                    int B, int C, int H, int W, int k, void* stream);

/* Backpropagation through x = f^{-1}(y) (Section 3.1-3.3, Theorems 1 and 2,
 * Algorithm 1's schedule):
 *   grad_y = M^{-T} grad_x       reverse wavefront from the bottom-right corner,
 *   grad_w[co][ci][k-1-dh][k-1-dw] = -sum_{n,h,w} grad_y[n,co,h,w] * x[n,ci,h-dh,w-dw],
 *                                   summed over the batch; 0 outside the mask.
 *   grad_x [B,C,H,W] in, x [B,C,H,W] in (the saved forward output), w in,
 *   grad_y [B,C,H,W] out, grad_w [C,C,k,k] out.  grad_w may be NULL (skip it);
 *   grad_y must be non-NULL (grad_w is computed from it).
 * Precision: the solves accumulate in fp32 throughout (the tensor-core family splits every operand into a
 * tf32 part and a bf16 remainder, so its products carry about 19 bits).  For C >= 8 outside the warp-shuffle
 * family the sum over pixels of grad_w may run on the tensor pipe with its two operands rounded to tf32
 * (10-bit mantissa) and fp32 accumulation: each entry is then accurate to about 3e-4 of the LARGEST entry of
 * grad_w, not of itself; INVCONV_OPT_GRADW_TENSOR_PIPE = 0 selects the fp32 kernel instead.  Below 8 channels
 * grad_w is always summed from fp32 products. */
int invconv_backward(const float* grad_x, const float* x, const float* w,
                     float* grad_y, float* grad_w,
                     int B, int C, int H, int W, int k, void* stream);

/* y = f(x): the masked convolution itself, the sampling direction
 * (Eq. 1; Section 4.3).  x in, w in, y out. */
int masked_conv_forward(const float* x, const float* w, float* y,
                        int B, int C, int H, int W, int k, void* stream);

/* logdet[0] = H*W*sum_c log|w[c][c][k-1][k-1]| = log|det df/dx| (Section 4:
 * triangular Jacobian; a unit diagonal gives 0).  Accumulated in double on the
 * device and rounded once to fp32.  The inverse layer's log-det is its
 * negative.  logdet points to ONE device float. */
int invconv_logdet(const float* w, float* logdet, int C, int H, int W, int k, void* stream);

/* The two calls of a flow layer's training step with the log-det folded in
 * (Section 4: the layer contributes its log-det to the likelihood):
 *
 * invconv_forward_logdet = invconv_forward followed, on the same stream, by
 *   invconv_logdet into logdet[0] (ONE device float; the log-det of f -- the
 *   layer z = f^{-1}(y) contributes its negative).
 *
 * invconv_backward_logdet = invconv_backward followed by
 *   grad_w[c][c][k-1][k-1] += grad_logdet[0] * H*W / w[c][c][k-1][k-1]  for every c,
 *   the derivative of grad_logdet[0] * logdet with respect to w (zero for every
 *   other entry).  grad_logdet points to ONE device float (the upstream
 *   gradient of the loss with respect to the log-det value returned above);
 *   grad_w must be non-NULL here.
 * Argument rules, scratch and errors are those of invconv_forward/backward.
 * No extra launch: the log-det is written by a spare warp of the forward kernels (in the shadow of the image's
 * arrival) and its term is added where the final grad_w is written; only the fallback kernels for shapes no
 * specialised family serves use one single-warp launch more. */
int invconv_forward_logdet(const float* y, const float* w, float* x, float* logdet,
                           int B, int C, int H, int W, int k, void* stream);
int invconv_backward_logdet(const float* grad_x, const float* x, const float* w, const float* grad_logdet,
                            float* grad_y, float* grad_w,
                            int B, int C, int H, int W, int k, void* stream);

/* The layer inside one step of the paper's Inverse-Flow model (Section 4, Fig. 3: Inv-Conv, then Actnorm,
 * then a 1x1 convolution), with the two neighbours folded into the layer's calls.  Both neighbours act on one
 * pixel at a time:
 *     z[n,c,h,w] = s[c] * x[n,c,h,w] + b[c]            Actnorm (per-channel affine map)
 *     u[n,o,h,w] = sum_c V[o][c] * z[n,c,h,w]          1x1 convolution (C x C channel mix)
 *
 * invconv_flow_step_forward:  x = f^{-1}(y) (saved for the backward pass) and u = V (s * x + b).
 *   y in; w [C,C,k,k], s [C], b [C], V [C][C] in; x, u [B,C,H,W] out; logdet: ONE device float or NULL,
 *   the step's log-determinant  H*W * ( -sum_c log|w[c][c][k-1][k-1]| + sum_c log|s[c]| + log|det V| )
 *   (accumulated in double; det V by Gaussian elimination with partial pivoting).
 * invconv_flow_step_backward: given grad_u (gradient of the loss with respect to u) and the saved x,
 *   grad_y = M^{-T} ( s * V^T grad_u ),  grad_w as in invconv_backward,
 *   grad_V[o][c] = sum grad_u[n,o,h,w] * z[n,c,h,w],  grad_s[c] = sum (V^T grad_u)[n,c,h,w] * x[n,c,h,w],
 *   grad_b[c] = sum (V^T grad_u)[n,c,h,w]   (sums over batch and pixels, fixed order).  All outputs non-NULL.
 * For shapes of the warp-shuffle family whose images fit shared memory the neighbours are applied inside the
 * wavefront kernel (u is written while x is stored; the incoming gradient is transformed as it is loaded);
 * other shapes run the layer's kernels and per-pixel kernels one after the other -- same results.  Scratch
 * comes from the library's stream-ordered memory pool.  Argument rules and errors as for invconv_forward. */
int invconv_flow_step_forward(const float* y, const float* w, const float* s, const float* b, const float* V,
                              float* x, float* u, float* logdet, int B, int C, int H, int W, int k, void* stream);
int invconv_flow_step_backward(const float* grad_u, const float* x, const float* w, const float* s, const float* b,
                               const float* V, float* grad_y, float* grad_w, float* grad_s, float* grad_b, float* grad_V,
                               int B, int C, int H, int W, int k, void* stream);

/* Reduced-precision storage variant of invconv_forward / invconv_backward: the activations y, x, grad_x and
 * grad_y are bfloat16 in device memory ([B][C][H][W], contiguous, 2 bytes per value; passed as void*), the
 * weights w and grad_w stay fp32.  Only the number format in memory changes: a bfloat16 value is widened
 * exactly to fp32 when it is read, every sum of the method (the substitution chain of Section 3, Theorem 1's
 * transposed solve, Theorem 2's correlation, which takes the fp32 grad_y before it is narrowed and the stored
 * x) is carried in fp32 as in the fp32 calls, and an output is rounded to the nearest bfloat16 (ties to even)
 * when it is written.  So x_stored = bf16(f^-1(y_stored)) up to the fp32 calls' own error, and the per-value
 * error of an output is half a bfloat16 spacing (2^-9 relative) on top of that.  The paper has no such
 * variant (it stores fp32); it halves the activation bytes per step for the batch-scaling regime of the
 * paper's batch-size ablation.
 *
 * Shapes of the warp-shuffle family whose images fit shared memory read and write bfloat16 inside the
 * wavefront kernel (C*H*W a multiple of 8, buffers 16-byte aligned, and -- backward with grad_w -- grad_w
 * riding along in the wavefront): invconv_bf16_in_kernel says so for a shape.  Every other shape is composed:
 * widen into fp32 scratch, the fp32 path, narrow the result -- same results, no bytes saved.
 * Argument rules, errors and scratch (library-owned stream-ordered pool) as for invconv_forward / _backward. */
int invconv_forward_bf16(const void* y_bf16, const float* w, void* x_bf16,
                         int B, int C, int H, int W, int k, void* stream);
int invconv_backward_bf16(const void* grad_x_bf16, const void* x_bf16, const float* w, void* grad_y_bf16, float* grad_w,
                          int B, int C, int H, int W, int k, void* stream);
/* The same two calls with caller-owned device scratch of at least invconv_bf16_workspace_bytes(...) bytes,
 * 256-byte aligned, under the rules of invconv_forward_ws (control words zeroed once, left zero by every
 * call, one call at a time per workspace); these forms allocate nothing.  For a shape handled inside the
 * wavefront kernel the size covers that route only: with buffers off a 16-byte boundary such a call returns
 * INVCONV_WORKSPACE_TOO_SMALL (use the forms above, or pass need + 3 fp32 copies of the activations). */
size_t invconv_bf16_workspace_bytes(int B, int C, int H, int W, int k);
int invconv_forward_bf16_ws(const void* y_bf16, const float* w, void* x_bf16, int B, int C, int H, int W, int k,
                            void* workspace, size_t workspace_bytes, void* stream);
int invconv_backward_bf16_ws(const void* grad_x_bf16, const void* x_bf16, const float* w, void* grad_y_bf16, float* grad_w,
                             int B, int C, int H, int W, int k, void* workspace, size_t workspace_bytes, void* stream);
/* 1 if the call above (backward != 0: invconv_backward_bf16, with_grad_w != 0: grad_w non-NULL) handles
 * bfloat16 inside the wavefront kernel for this shape (given aligned buffers), 0 if it is composed. */
int invconv_bf16_in_kernel(int B, int C, int H, int W, int k, int backward, int with_grad_w);

/* Scratch bytes a forward or backward call of this shape needs (0 if none).
 * Same value for both directions. */
size_t invconv_workspace_bytes(int B, int C, int H, int W, int k);

/* As invconv_forward / invconv_backward, but with caller-owned device scratch
 * of at least invconv_workspace_bytes(...) bytes, 256-byte aligned.  These
 * forms allocate nothing.  The first INVCONV_WS_CONTROL_BYTES bytes are
 * control words: zero them once after allocating the workspace (cudaMemset);
 * every call leaves them zero again.  Calls sharing a workspace must not
 * overlap on the device. */
#define INVCONV_WS_CONTROL_BYTES 256
int invconv_forward_ws(const float* y, const float* w, float* x,
                       int B, int C, int H, int W, int k,
                       void* workspace, size_t workspace_bytes, void* stream);
int invconv_backward_ws(const float* grad_x, const float* x, const float* w,
                        float* grad_y, float* grad_w,
                        int B, int C, int H, int W, int k,
                        void* workspace, size_t workspace_bytes, void* stream);

/* One whole layer step from HOST buffers: copies y, w, grad_x to the device,
 * runs invconv_forward, invconv_backward and invconv_logdet there, and copies
 * x, grad_y, grad_w and the log-det back -- enqueued on `stream`, no
 * synchronisation (use pinned host memory for truly asynchronous copies and
 * synchronise the stream before reading the outputs).  The copy of grad_x in
 * and of x out run on a library-owned side stream (one per device, created on
 * first use) so that the two copy directions overlap each other and the
 * kernels; the side stream is forked from and joined back into `stream` with
 * events inside the call, so `stream` alone orders the whole step.
 *   *_host: host pointers (y, grad_x, x, grad_y: B*C*H*W floats; w, grad_w:
 *   C*C*k*k floats; logdet: 1 float).
 *   device_scratch: caller-owned device memory of at least
 *   invconv_step_scratch_bytes(...) bytes, 256-byte aligned, zeroed once after
 *   allocation; holds the device copies and the kernels' workspace. */
size_t invconv_step_scratch_bytes(int B, int C, int H, int W, int k);
int invconv_step_host(const float* y_host, const float* w_host, const float* grad_x_host,
                      float* x_host, float* grad_y_host, float* grad_w_host, float* logdet_host,
                      int B, int C, int H, int W, int k,
                      void* device_scratch, size_t device_scratch_bytes, void* stream);

/* invconv_backward for callers that must not allocate.  (The paper has no
 * counterpart; this is a deployment convenience.)
 *
 * Some hosts freeze their device-memory map once start-up is over -- an
 * inference server with a fixed memory plan, a real-time loop, a plug-in that
 * runs inside another framework's callback -- and from then on may call
 * neither cudaMalloc nor a pooled allocator.  The other backward entry points
 * need scratch memory (a completion counter and per-CTA partial sums of
 * grad_w) that either the library takes from its stream-ordered memory pool
 * (invconv_backward) or the caller provides (invconv_backward_ws).  This
 * variant keeps that scratch in a fixed array of INVCONV_NOALLOC_SCRATCH_BYTES
 * that is part of the library image itself: every GPU that loads the library
 * holds those bytes until the process exits, whether or not the call is used.
 *
 *  - Same arguments, outputs and arithmetic as invconv_backward; served by the
 *    warp-shuffle kernel family only.  Shapes that family does not serve return
 *    INVCONV_UNSUPPORTED; shapes whose scratch would exceed the fixed array
 *    return INVCONV_WORKSPACE_TOO_SMALL.  Nothing is launched in either case.
 *  - The library itself calls neither cudaMalloc nor cudaFree nor any other
 *    allocating routine here.  The CUDA runtime, however, loads a kernel's code
 *    the first time that kernel is launched, and that may allocate: call once
 *    per (shape, grad_w NULL or not) on each device during start-up, before
 *    memory is frozen.
 *  - The first call on each device also looks up the array's device address
 *    (with that device current) and caches it; make that first call before any
 *    stream capture begins on the device.
 *  - All calls on a device share the one array.  Each call clears the control
 *    words it relies on, on `stream`, before its kernel runs, so a call may
 *    follow an aborted one; but two calls that overlap on the GPU (different
 *    streams without ordering between them) race on the array and produce
 *    garbage in grad_w.  Order them. */
#define INVCONV_NOALLOC_SCRATCH_BYTES (1u << 20)
int invconv_backward_noalloc(const float* grad_x, const float* x, const float* w,
                             float* grad_y, float* grad_w,
                             int B, int C, int H, int W, int k, void* stream);

/* Force a kernel family for subsequent calls from this process (default AUTO).
 * Returns the previous setting. */
int invconv_set_path(int path);

/* The family AUTO would pick for this shape (an invconv_path value). */
int invconv_path_for(int B, int C, int H, int W, int k);

/* CTAs per thread-block cluster of the wavefront kernel AUTO would launch for this shape (1 = no cluster):
 * more than one means that neighbouring diagonals are exchanged through distributed shared memory, which is
 * what sets the latency of one dependent step (Section 3.3: H+W-1 sequential steps). */
int invconv_cluster_size_for(int B, int C, int H, int W, int k);

/* Synchronises `stream`, then reports and clears the device-side status word
 * of the current device: INVCONV_OK, or INVCONV_TIMEOUT if a bounded wait
 * inside a kernel gave up since the last query (its outputs are then invalid).
 * Returns INVCONV_CUDA_ERROR if the synchronisation itself failed. */
int invconv_get_status(void* stream, int* device_status_out);

/* Measures, on the current device, the latency of one dependent wavefront step
 * for a communication mechanism, with no other work on the chain:
 *   mechanism 0: warp shuffle + one FMA (lane = image row);
 *   mechanism 1: shared-memory store, block barrier, load, one FMA;
 *   mechanism 2: store to a cluster peer's shared memory, cluster barrier, load, one FMA.
 * Runs a chain of `steps` dependent steps in one CTA (cluster of 2 for 2) and
 * writes the elapsed SM clock cycles to cycles_out[0] and the chain's final
 * value to cycles_out[1] (device pointer to two 64-bit words).  Used for the
 * critical-path bound of 2*(H+W-1) dependent steps (Section 3.3, complexity). */
int invconv_probe_step_latency(int mechanism, int steps, unsigned long long* cycles_out, void* stream);

/* Self-test of the bounded device-side waits: launches one small kernel that waits, with a limit of
 * `limit_cycles` SM clock cycles (1 <= limit_cycles <= 2^24), on a barrier that nothing completes.  The wait
 * runs out, the kernel raises the device status word to INVCONV_TIMEOUT and returns normally; the context
 * stays usable.  invconv_get_status then reports INVCONV_TIMEOUT once. */
int invconv_selftest_wait_timeout(unsigned limit_cycles, void* stream);

/* Debug-bounds build (the tensor-core and flow-step kernels compiled with -DINVCONV_DEBUG_BOUNDS,
 * libinvconv_b200_debug.so): every index those kernels compute for shared or global memory goes through a
 * checked accessor; an index outside its array is recorded instead of used, and invconv_get_status reports
 * INVCONV_BOUNDS.  invconv_debug_bounds_info fills info[0..3] = {site number, index, limit, number of
 * violations} of the current device and clears the record; it returns INVCONV_UNSUPPORTED in the normal build.
 * invconv_selftest_bounds hands the accessor an index outside its limit on purpose (no memory is touched), to
 * show that the record and the status work; INVCONV_UNSUPPORTED in the normal build. */
int invconv_debug_bounds_info(int* info /* host, 4 ints */);
int invconv_selftest_bounds(void* stream);

/* Development and test controls -- not needed in normal use.  They force one of two equivalent kernels or
 * launch modes so that tests and measurements can compare them; results are the same within rounding.
 * invconv_set_option returns the previous value, or -1 for an unknown option.  Process-wide. */
enum invconv_option {
    INVCONV_OPT_WARP_RING = 0,       /* 1 (default): images larger than shared memory stream through a ring; 0: global-memory mode */
    INVCONV_OPT_WARP_CHANNEL_SPLIT,  /* 1 (default): lane = (row, channel) walk for C >= 3, k = 5; 0: one lane per row */
    INVCONV_OPT_GRADW_SEPARATE,      /* -1 (default): by shape; 0: grad_w inside the warp wavefront; 1: separate pixel-parallel kernel */
    INVCONV_OPT_GRADW_TENSOR_PIPE,   /* 1 (default): many-channel grad_w on the tensor pipe (tf32 operands); 0: fp32 FMA kernel */
    INVCONV_OPT_TEAM_VARIANT,        /* 0 (default): by shape; 1: channel-slice kernel; 2: pixel-team kernel */
    INVCONV_OPT_TEAM_CLUSTER,        /* 0 (default): by shape; 1..8: force the cluster size of the channel-slice kernel */
    INVCONV_OPT_DEPENDENT_LAUNCH,    /* 1 (default): programmatic dependent launch between the library's kernels; 0: off */
    INVCONV_OPT_COUNT
};
int invconv_set_option(int option, int value);

/* Number of kernels this library has launched (or captured into a CUDA graph)
 * from this process since it was loaded. */
unsigned long long invconv_kernel_launch_count(void);

const char* invconv_status_string(int status);
int invconv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* INVCONV_H_ */

/*
 * Float64 CPU oracle for the inverse of a masked, top-left-padded k x k
 * multi-channel convolution and its backpropagation.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It exists so that the CUDA
 * library can be compared element by element with a slow, plain, obviously
 * correct restatement of the paper's definitions.  It shares no code with the
 * CUDA path, is never tuned, and must only be called from the tests, from the
 * smoke check and from the benchmark's CPU-baseline leg.
 *
 * Conventions (0-indexed, fixed once):
 *   activations  x, y, grad_x, grad_y : [B][C][H][W]   contiguous doubles
 *   kernel       w, grad_w            : [C_out][C_in][k][k]
 *   The tap that multiplies pixel (h-dh, w-dw) in the output at (h, w) is
 *   w[co][ci][k-1-dh][k-1-dw], 0 <= dh, dw < k  (Eq. 1: the kernel index is
 *   (k,k) - p + q; Algorithm 1 pairs K[c, k_c, k_H-k_h-1, k_W-k_w-1] with
 *   pixel (h-k_h, w-k_w)).  Pixels with a negative coordinate are the k-1
 *   rows / columns of zero padding on the top and left (Section 3).
 *   The tap aligned with the output pixel itself, w[:, :, k-1, k-1] -- the
 *   paper's "bottom right entry" -- is masked to ci <= co (lower triangular
 *   over channels); its channel diagonal is free and non-zero.  The paper's
 *   own case is that diagonal equal to 1.  Whatever is stored at the masked-
 *   out positions (ci > co) is never read.
 *
 * Every function below is the definition written out with naive loops; the
 * only ordering that matters is that substitution visits pixels in an order
 * compatible with the partial order p <= q (Section 3, Notation), for which
 * plain row-major order is used -- deliberately NOT the anti-diagonal order
 * of the GPU kernels.
 *
 * Pins (tests/test_oracle_pins.py): dense (HWC)x(HWC) Gaussian elimination,
 * a hand-worked 2x2 example, identity / diagonal kernels, a geometric-series
 * closed form, round trips, causality of the support, finite differences,
 * the adjoint identity, the literal recursions of Theorems 1 and 2, a library
 * convolution, and log|det| of the dense matrix.  No function here is
 * "parity unpinned".
 */
#include <math.h>
#include <stddef.h>

#define IDX4(n, c, h, w, C, H, W) ((((size_t)(n) * (C) + (c)) * (H) + (h)) * (W) + (w))
#define WIDX(co, ci, a, b, C, k) ((((size_t)(co) * (C) + (ci)) * (k) + (a)) * (k) + (b))

/* Is kernel entry (co, ci, dh, dw) inside the mask?  Only the tap with
 * dh = dw = 0 is restricted (to ci <= co).  (Section 3; Supplementary
 * "Input Padding and Kernel Masking".) */
static int tap_in_mask(int co, int ci, int dh, int dw)
{
    if (dh == 0 && dw == 0) return ci <= co;
    return 1;
}

/* y = f(x): the masked convolution of Eq. 1, extended over channels as in
 * Algorithm 1's index set (k_h, k_w, k_c).  This is the sampling direction
 * (Section 4.3). */
void oracle_masked_conv(const double *x, const double *w, double *y,
                        int B, int C, int H, int W, int k)
{
    for (int n = 0; n < B; ++n)
        for (int co = 0; co < C; ++co)
            for (int h = 0; h < H; ++h)
                for (int ww = 0; ww < W; ++ww) {
                    double acc = 0.0;
                    for (int ci = 0; ci < C; ++ci)
                        for (int dh = 0; dh < k; ++dh)
                            for (int dw = 0; dw < k; ++dw) {
                                int hh = h - dh, wq = ww - dw;
                                if (hh < 0 || wq < 0) continue;          /* zero padding */
                                if (!tap_in_mask(co, ci, dh, dw)) continue;
                                acc += w[WIDX(co, ci, k - 1 - dh, k - 1 - dw, C, k)] *
                                       x[IDX4(n, ci, hh, wq, C, H, W)];
                            }
                    y[IDX4(n, co, h, ww, C, H, W)] = acc;
                }
}

/* x = f^{-1}(y): forward substitution.  Eq. 1 rearranged for x_q
 * (Supplementary, proof of Theorem 1, the line "x_q = y_q - sum ..."),
 * with the free channel diagonal divided out.  Pixels are visited row-major,
 * channels ascending, so that every x on the right-hand side is already
 * known. */
void oracle_invconv_forward(const double *y, const double *w, double *x,
                            int B, int C, int H, int W, int k)
{
    for (int n = 0; n < B; ++n)
        for (int h = 0; h < H; ++h)
            for (int ww = 0; ww < W; ++ww)
                for (int co = 0; co < C; ++co) {
                    double r = y[IDX4(n, co, h, ww, C, H, W)];
                    for (int ci = 0; ci < C; ++ci)
                        for (int dh = 0; dh < k; ++dh)
                            for (int dw = 0; dw < k; ++dw) {
                                int hh = h - dh, wq = ww - dw;
                                if (hh < 0 || wq < 0) continue;
                                if (dh == 0 && dw == 0 && ci >= co) continue; /* own pixel: only ci < co is known / in mask */
                                r -= w[WIDX(co, ci, k - 1 - dh, k - 1 - dw, C, k)] *
                                     x[IDX4(n, ci, hh, wq, C, H, W)];
                            }
                    x[IDX4(n, co, h, ww, C, H, W)] = r / w[WIDX(co, co, k - 1, k - 1, C, k)];
                }
}

/* grad_y = M^{-T} grad_x, where M is the matrix of f.  Eq. 2 sums
 * dL/dx_q * dx_q/dy_p over q; with Theorem 1's recursion for dx_q/dy_p this
 * is the back substitution of the transposed triangular system: row p of M^T
 * holds the taps through which x_p feeds later pixels q >= p.  Pixels are
 * visited in reverse row-major order, channels descending. */
void oracle_invconv_grad_y(const double *grad_x, const double *w, double *grad_y,
                           int B, int C, int H, int W, int k)
{
    for (int n = 0; n < B; ++n)
        for (int h = H - 1; h >= 0; --h)
            for (int ww = W - 1; ww >= 0; --ww)
                for (int ci = C - 1; ci >= 0; --ci) {
                    double r = grad_x[IDX4(n, ci, h, ww, C, H, W)];
                    for (int co = 0; co < C; ++co)
                        for (int dh = 0; dh < k; ++dh)
                            for (int dw = 0; dw < k; ++dw) {
                                int hh = h + dh, wq = ww + dw;
                                if (hh >= H || wq >= W) continue;
                                if (dh == 0 && dw == 0 && co <= ci) continue; /* own pixel: only co > ci is in mask and known */
                                r -= w[WIDX(co, ci, k - 1 - dh, k - 1 - dw, C, k)] *
                                     grad_y[IDX4(n, co, hh, wq, C, H, W)];
                            }
                    grad_y[IDX4(n, ci, h, ww, C, H, W)] = r / w[WIDX(ci, ci, k - 1, k - 1, C, k)];
                }
}

/* grad_w: Theorem 2 in closed form.  Its recursion (last equation of the
 * proof) reads  d x / d W_a = -M^{-1} shift_a(x); contracting with grad_x
 * (the equation "dL/dW_a = sum_q dL/dx_q * dx_q/dW_a") gives
 *     grad_w[co][ci][k-1-dh][k-1-dw] = - sum_{n,h,w} grad_y[n,co,h,w] * x[n,ci,h-dh,w-dw]
 * over in-bounds pixels; entries outside the mask are 0.  grad_w is
 * overwritten (Algorithm 1 initialises it to zero), summed over the batch. */
void oracle_invconv_grad_w(const double *grad_y, const double *x, double *grad_w,
                           int B, int C, int H, int W, int k)
{
    for (int co = 0; co < C; ++co)
        for (int ci = 0; ci < C; ++ci)
            for (int dh = 0; dh < k; ++dh)
                for (int dw = 0; dw < k; ++dw) {
                    double acc = 0.0;
                    if (tap_in_mask(co, ci, dh, dw)) {
                        for (int n = 0; n < B; ++n)
                            for (int h = dh; h < H; ++h)
                                for (int ww = dw; ww < W; ++ww)
                                    acc += grad_y[IDX4(n, co, h, ww, C, H, W)] *
                                           x[IDX4(n, ci, h - dh, ww - dw, C, H, W)];
                        acc = -acc;
                    }
                    grad_w[WIDX(co, ci, k - 1 - dh, k - 1 - dw, C, k)] = acc;
                }
}

/* log|det df/dx| = H*W*sum_c log|w[c][c][k-1][k-1]|: M is triangular in
 * row-major pixel order with that tap on its diagonal (Section 3; Section 4:
 * a unit diagonal gives determinant 1).  The inverse layer's log-det is the
 * negative of this value. */
double oracle_logdet(const double *w, int C, int H, int W, int k)
{
    double s = 0.0;
    for (int c = 0; c < C; ++c)
        s += log(fabs(w[WIDX(c, c, k - 1, k - 1, C, k)]));
    return (double)H * (double)W * s;
}

/* d logdet / d w, same shape as w: H*W / w[c][c][k-1][k-1] on the channel
 * diagonal of the bottom-right tap, 0 everywhere else (derivative of
 * H*W*sum_c log|w_cc|; the flow's loss adds a multiple of the log-det to the
 * likelihood, Section 4). */
void oracle_logdet_grad_w(const double *w, double *gw, int C, int H, int W, int k)
{
    for (int i = 0; i < C * C * k * k; ++i) gw[i] = 0.0;
    for (int c = 0; c < C; ++c)
        gw[WIDX(c, c, k - 1, k - 1, C, k)] = (double)H * (double)W / w[WIDX(c, c, k - 1, k - 1, C, k)];
}

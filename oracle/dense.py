"""The plainest layer of the oracle, for tiny inputs only (test infrastructure).

* `dense_matrix`   -- the (HWC)x(HWC) matrix M of the masked convolution f,
                      row-major pixel order with channels innermost
                      (Section 3: "multiplication by a m^2 x m^2 matrix";
                      Supplementary Fig. 4: lower triangular, the bottom-right
                      tap on the diagonal).
* `gauss_solve`    -- Gaussian elimination with partial pivoting, written out
                      (the paper's "naive" O(n^3) algorithm, Table 1).
* `theorem1_dx_dy` -- the recursion of Theorem 1 evaluated entry by entry
                      (proof, inductive step: d x_q/d y_p = [q = p] - sum over
                      Delta(q) of W * d x_r/d y_p).
* `theorem2_dx_dw` -- the recursion that closes the proof of Theorem 2
                      (d x_q/d W_a = -x_{q-a} - sum over Delta(q) of W * d x_r/d W_a).

The two recursions are written for any channel count and a free channel
diagonal d_c = w[c,c,k-1,k-1]: dividing the defining equation by d_c is the
only change from the paper's unit-diagonal, one-channel statement.
"""
from __future__ import annotations

import numpy as np


def unknown_index(h: int, w: int, c: int, W: int, C: int) -> int:
    return (h * W + w) * C + c


def tap(wt: np.ndarray, co: int, ci: int, dh: int, dw: int) -> float:
    """Masked kernel entry that multiplies x[ci, h-dh, w-dw] in y[co, h, w] (Eq. 1)."""
    k = wt.shape[2]
    if dh == 0 and dw == 0 and ci > co:
        return 0.0
    return float(wt[co, ci, k - 1 - dh, k - 1 - dw])


def dense_matrix(wt, H: int, W: int) -> np.ndarray:
    wt = np.asarray(wt, dtype=np.float64)
    C, k = wt.shape[0], wt.shape[2]
    n = H * W * C
    M = np.zeros((n, n), dtype=np.float64)
    for h in range(H):
        for w in range(W):
            for co in range(C):
                row = unknown_index(h, w, co, W, C)
                for dh in range(k):
                    for dw in range(k):
                        if h - dh < 0 or w - dw < 0:
                            continue
                        for ci in range(C):
                            M[row, unknown_index(h - dh, w - dw, ci, W, C)] = tap(wt, co, ci, dh, dw)
    return M


def to_vec(a) -> np.ndarray:
    """[C,H,W] image -> vector in the (h, w, c) order of `dense_matrix`."""
    return np.ascontiguousarray(np.transpose(np.asarray(a, dtype=np.float64), (1, 2, 0))).reshape(-1)


def from_vec(v, C: int, H: int, W: int) -> np.ndarray:
    return np.ascontiguousarray(np.transpose(np.asarray(v).reshape(H, W, C), (2, 0, 1)))


def gauss_solve(A, b) -> np.ndarray:
    """Solve A z = b by Gaussian elimination with partial pivoting, then back substitution."""
    A = np.array(A, dtype=np.float64, copy=True)
    b = np.array(b, dtype=np.float64, copy=True)
    n = A.shape[0]
    for col in range(n):
        piv = col + int(np.argmax(np.abs(A[col:, col])))
        if A[piv, col] == 0.0:
            raise ZeroDivisionError("singular matrix")
        if piv != col:
            A[[col, piv]] = A[[piv, col]]
            b[[col, piv]] = b[[piv, col]]
        below = np.nonzero(A[col + 1:, col])[0] + col + 1
        for r in below:
            f = A[r, col] / A[col, col]
            A[r, col:] -= f * A[col, col:]
            b[r] -= f * b[col]
    z = np.zeros(n, dtype=np.float64)
    for r in range(n - 1, -1, -1):
        z[r] = (b[r] - A[r, r + 1:] @ z[r + 1:]) / A[r, r]
    return z


def _delta(h: int, w: int, c: int, k: int, C: int):
    """The unknowns x_r that appear beside x_(h,w,c) in its own equation:
    Delta(p) of the paper (pixels in the k x k window up and to the left,
    p itself excluded) for every channel, plus the lower channels of p."""
    for dh in range(k):
        for dw in range(k):
            if h - dh < 0 or w - dw < 0:
                continue
            for ci in range(C):
                if dh == 0 and dw == 0 and ci >= c:
                    continue
                yield dh, dw, ci


def theorem1_dx_dy(wt, H: int, W: int) -> np.ndarray:
    """J[q, p] = d x_q / d y_p, entry by entry from Theorem 1's recursion.

    For each p the unknowns q are visited in row-major order; the derivative
    is zero unless p precedes q in that order (a superset of the partial
    order's support, so the zeros of the theorem's second case come out of
    the recursion itself).
    """
    wt = np.asarray(wt, dtype=np.float64)
    C, k = wt.shape[0], wt.shape[2]
    n = H * W * C
    J = np.zeros((n, n), dtype=np.float64)
    for p in range(n):
        for h in range(H):
            for w in range(W):
                for c in range(C):
                    q = unknown_index(h, w, c, W, C)
                    if q < p:
                        continue
                    acc = 1.0 if q == p else 0.0
                    for dh, dw, ci in _delta(h, w, c, k, C):
                        acc -= tap(wt, c, ci, dh, dw) * J[unknown_index(h - dh, w - dw, ci, W, C), p]
                    J[q, p] = acc / wt[c, c, k - 1, k - 1]
    return J


def theorem2_dx_dw(wt, x_img, co_a: int, ci_a: int, dh_a: int, dw_a: int) -> np.ndarray:
    """d x_q / d W_a for the kernel entry a = (co_a, ci_a, offset (dh_a, dw_a)),
    entry by entry: the direct term -x_{q-a} (only in output channel co_a, only
    where the shifted pixel exists) plus the recursive term through Delta(q).
    Returns a [C,H,W] image."""
    wt = np.asarray(wt, dtype=np.float64)
    x_img = np.asarray(x_img, dtype=np.float64)
    C, H, W = x_img.shape
    k = wt.shape[2]
    D = np.zeros((C, H, W), dtype=np.float64)
    for h in range(H):
        for w in range(W):
            for c in range(C):
                acc = 0.0
                if c == co_a and h - dh_a >= 0 and w - dw_a >= 0:
                    acc -= x_img[ci_a, h - dh_a, w - dw_a]
                for dh, dw, ci in _delta(h, w, c, k, C):
                    acc -= tap(wt, c, ci, dh, dw) * D[ci, h - dh, w - dw]
                D[c, h, w] = acc / wt[c, c, k - 1, k - 1]
    return D

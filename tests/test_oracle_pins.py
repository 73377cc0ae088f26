"""Pins of the float64 oracle against things other than itself.

Each test ties one oracle function to a fact the paper or the mathematics
fixes: a hand-worked example, the dense matrix of the operator solved by
Gaussian elimination, closed forms, invariants, a library convolution,
finite differences, and the literal recursions of Theorems 1 and 2.
A dropped term, a wrong sign, a transposed channel index or a flipped kernel
fails at least one of them.
"""
import os

import numpy as np
import pytest

from oracle import api, dense
from paper_2410_14634_b200 import workloads
from conftest import nmax_err

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

TINY = [  # (B, C, H, W, k)
    (2, 1, 4, 4, 2),
    (2, 3, 5, 4, 3),
    (1, 2, 3, 6, 3),
    (2, 2, 4, 3, 1),
    (1, 3, 2, 2, 4),   # kernel larger than the image
    (1, 1, 1, 7, 3),   # single row
    (1, 2, 6, 1, 2),   # single column
]


def tiny_inputs(seed, B, C, H, W, k, **kw):
    w, y, gx = workloads.make_custom(seed, B, C, H, W, k, sigma=0.3, **kw)
    return w.astype(np.float64), y.astype(np.float64), gx.astype(np.float64)


# ---------------------------------------------------------------- hand-worked example

def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


def test_hand_worked_2x2():
    g = read_golden("hand_2x2.txt")
    w = g["w"].reshape(1, 1, 2, 2)
    x = g["x"].reshape(1, 1, 2, 2)
    y = g["y"].reshape(1, 1, 2, 2)
    gx = g["grad_x"].reshape(1, 1, 2, 2)
    assert np.allclose(api.masked_conv(x, w), y, atol=1e-15)
    assert np.allclose(api.invconv_forward(y, w), x, atol=1e-15)
    gy, gw = api.invconv_backward(gx, x, w)
    assert np.allclose(gy.reshape(-1), g["grad_y"], atol=1e-15)
    assert np.allclose(gw.reshape(-1), g["grad_w"], atol=1e-15)
    assert api.logdet(w, 2, 2) == g["logdet"][0]


# ---------------------------------------------------------------- structure of M

@pytest.mark.parametrize("B,C,H,W,k", TINY)
def test_dense_matrix_is_lower_triangular_with_centre_tap_on_diagonal(B, C, H, W, k):
    w, _, _ = tiny_inputs(1, B, C, H, W, k, masked_fill=123.0)
    M = dense.dense_matrix(w, H, W)
    assert np.all(np.triu(M, 1) == 0.0)
    d = np.tile(np.array([w[c, c, k - 1, k - 1] for c in range(C)]), H * W)
    assert np.array_equal(np.diag(M), d)


# ---------------------------------------------------------------- f

@pytest.mark.parametrize("B,C,H,W,k", TINY)
def test_masked_conv_equals_dense_matvec(B, C, H, W, k):
    w, x, _ = tiny_inputs(2, B, C, H, W, k, masked_fill=55.0)
    M = dense.dense_matrix(w, H, W)
    y = api.masked_conv(x, w)
    for n in range(B):
        ref = dense.from_vec(M @ dense.to_vec(x[n]), C, H, W)
        assert nmax_err(y[n], ref) < 1e-14


@pytest.mark.parametrize("B,C,H,W,k", [(2, 3, 7, 6, 3), (1, 4, 5, 9, 5), (3, 1, 8, 8, 2)])
def test_masked_conv_equals_library_cross_correlation(B, C, H, W, k):
    torch = pytest.importorskip("torch")
    w, x, _ = tiny_inputs(3, B, C, H, W, k)
    wm = w.copy()
    wm[:, :, k - 1, k - 1] = np.tril(wm[:, :, k - 1, k - 1])
    xp = torch.nn.functional.pad(torch.from_numpy(x), (k - 1, 0, k - 1, 0))
    ref = torch.nn.functional.conv2d(xp, torch.from_numpy(wm)).numpy()
    assert nmax_err(api.masked_conv(x, w), ref) < 1e-13


def identity_kernel(C, k):
    w = np.zeros((C, C, k, k))
    w[np.arange(C), np.arange(C), k - 1, k - 1] = 1.0
    return w


@pytest.mark.parametrize("C,k", [(1, 3), (3, 3), (2, 5)])
def test_identity_kernel_is_the_identity_both_ways(C, k):
    rng = np.random.default_rng(4)
    a = rng.normal(size=(2, C, 6, 5))
    w = identity_kernel(C, k)
    assert np.array_equal(api.masked_conv(a, w), a)
    assert np.array_equal(api.invconv_forward(a, w), a)
    assert np.array_equal(api.invconv_grad_y(a, w), a)
    assert api.logdet(w, 6, 5) == 0.0          # unit diagonal: determinant one (Section 4)


def test_diagonal_only_centre_tap_divides_each_channel():
    rng = np.random.default_rng(5)
    C, k = 3, 3
    d = np.array([0.5, -2.0, 1.25])
    w = np.zeros((C, C, k, k))
    w[np.arange(C), np.arange(C), k - 1, k - 1] = d
    y = rng.normal(size=(2, C, 4, 5))
    assert np.allclose(api.invconv_forward(y, w), y / d[None, :, None, None], rtol=1e-15)
    assert np.allclose(api.invconv_grad_y(y, w), y / d[None, :, None, None], rtol=1e-15)


@pytest.mark.parametrize("offset", [(0, 1), (1, 0), (1, 1), (0, 2)])
def test_single_off_centre_tap_gives_a_geometric_series(offset):
    """C = 1, unit diagonal, one tap a at offset (dh, dw):
    x[h, w] = sum_j (-a)^j y[h - j*dh, w - j*dw]."""
    dh, dw = offset
    k, a = 3, 0.7
    rng = np.random.default_rng(6)
    H, W = 7, 9
    y = rng.normal(size=(1, 1, H, W))
    w = identity_kernel(1, k)
    w[0, 0, k - 1 - dh, k - 1 - dw] = a
    ref = np.zeros_like(y)
    for h in range(H):
        for ww in range(W):
            j = 0
            while h - j * dh >= 0 and ww - j * dw >= 0:
                ref[0, 0, h, ww] += (-a) ** j * y[0, 0, h - j * dh, ww - j * dw]
                j += 1
    assert nmax_err(api.invconv_forward(y, w), ref) < 1e-14


# ---------------------------------------------------------------- f^{-1} against Gaussian elimination

@pytest.mark.parametrize("B,C,H,W,k", TINY)
def test_inverse_equals_gaussian_elimination_on_dense_matrix(B, C, H, W, k):
    w, y, _ = tiny_inputs(7, B, C, H, W, k, masked_fill=9.0)
    M = dense.dense_matrix(w, H, W)
    x = api.invconv_forward(y, w)
    for n in range(B):
        ref = dense.from_vec(dense.gauss_solve(M, dense.to_vec(y[n])), C, H, W)
        assert nmax_err(x[n], ref) < 1e-12
        lap = dense.from_vec(np.linalg.solve(M, dense.to_vec(y[n])), C, H, W)
        assert nmax_err(x[n], lap) < 1e-12


def test_pr1_config_as_a_dense_768_system():
    """Benchmark config 1 (batch 4, C=3, 16x16, k=3, seed 0): every image is a
    768-unknown system; x, grad_y and log-det against the dense matrix."""
    s, w, y, gx = workloads.make("pr1")
    M = dense.dense_matrix(w, s.H, s.W)
    assert M.shape == (768, 768)
    x = api.invconv_forward(y, w)
    gy = api.invconv_grad_y(gx, w)
    for n in range(s.B):
        ref = dense.from_vec(dense.gauss_solve(M, dense.to_vec(y[n])), s.C, s.H, s.W)
        assert nmax_err(x[n], ref) < 1e-12
        refg = dense.from_vec(dense.gauss_solve(M.T, dense.to_vec(gx[n])), s.C, s.H, s.W)
        assert nmax_err(gy[n], refg) < 1e-12
    sign, lad = np.linalg.slogdet(M)
    assert abs(api.logdet(w, s.H, s.W) - lad) < 1e-10 * max(1.0, abs(lad))


# ---------------------------------------------------------------- round trips and causality

@pytest.mark.parametrize("B,C,H,W,k", [(2, 3, 16, 16, 3), (1, 1, 28, 28, 3), (1, 12, 8, 8, 3), (1, 3, 20, 13, 5), (1, 2, 9, 9, 2)])
def test_round_trips(B, C, H, W, k):
    w, y, _ = workloads.make_custom(8, B, C, H, W, k, masked_fill=float("nan"))
    x = api.invconv_forward(y, w)
    assert np.all(np.isfinite(x))                 # masked-out entries were never read
    assert nmax_err(api.masked_conv(x, w), y) < 1e-12
    assert nmax_err(api.invconv_forward(api.masked_conv(y, w), w), y) < 1e-12


def test_output_pixel_depends_only_on_inputs_above_and_left():
    """x_q depends on y_p exactly when p <= q in the partial order (the usable
    direction of Theorem 1's zero case): perturbing one y_p changes x only at
    pixels with both coordinates >= p's, and does change x_p itself."""
    C, H, W, k = 2, 6, 7, 3
    w, y, _ = tiny_inputs(9, 1, C, H, W, k)
    x0 = api.invconv_forward(y, w)
    for (ph, pw, pc) in [(0, 0, 0), (2, 3, 1), (5, 6, 0), (3, 0, 1)]:
        y1 = y.copy()
        y1[0, pc, ph, pw] += 1.0
        dx = api.invconv_forward(y1, w) - x0
        mask = np.zeros((H, W), dtype=bool)
        mask[ph:, pw:] = True
        assert np.all(dx[0][:, ~mask] == 0.0)
        assert abs(dx[0, pc, ph, pw] - 1.0 / w[pc, pc, k - 1, k - 1]) < 1e-12
        if ph + 1 < H and pw + 1 < W:
            assert np.any(dx[0][:, ph + 1:, pw + 1:] != 0.0)


# ---------------------------------------------------------------- grad_y

@pytest.mark.parametrize("B,C,H,W,k", TINY)
def test_grad_y_equals_transposed_dense_solve(B, C, H, W, k):
    w, _, gx = tiny_inputs(10, B, C, H, W, k, masked_fill=-4.0)
    M = dense.dense_matrix(w, H, W)
    gy = api.invconv_grad_y(gx, w)
    for n in range(B):
        ref = dense.from_vec(dense.gauss_solve(M.T, dense.to_vec(gx[n])), C, H, W)
        assert nmax_err(gy[n], ref) < 1e-12


def test_grad_y_by_central_finite_differences():
    B, C, H, W, k = 1, 2, 4, 5, 3
    w, y, gx = tiny_inputs(11, B, C, H, W, k)
    gy = api.invconv_grad_y(gx, w)
    eps = 1e-6
    fd = np.zeros_like(y)
    for idx in np.ndindex(*y.shape):
        yp, ym = y.copy(), y.copy()
        yp[idx] += eps
        ym[idx] -= eps
        fd[idx] = (np.sum(gx * api.invconv_forward(yp, w)) - np.sum(gx * api.invconv_forward(ym, w))) / (2 * eps)
    assert nmax_err(gy, fd) < 1e-8


@pytest.mark.parametrize("name,batch", [("pr1", None), ("mnist", 8), ("cifar", 4), ("cifar_sq", 4),
                                        ("wide48_k3", 2), ("wide48_k5", 1), ("wide96_k3", 2), ("wide96_k5", 1),
                                        ("large64", 2), ("large256", 1)])
def test_adjoint_identity_at_benchmark_shapes(name, batch):
    """<grad_x, M^{-1} y> = <M^{-T} grad_x, y> needs no dense matrix, so it
    runs at every benchmark shape (on a few images of the batch)."""
    s, w, y, gx = workloads.make(name, batch=batch)
    x = api.invconv_forward(y, w)
    gy = api.invconv_grad_y(gx, w)
    lhs = float(np.sum(gx.astype(np.float64) * x))
    rhs = float(np.sum(gy * y.astype(np.float64)))
    scale = float(np.sqrt(np.sum(gx.astype(np.float64) ** 2) * np.sum(x ** 2)))
    assert abs(lhs - rhs) < 1e-12 * scale
    assert nmax_err(api.masked_conv(x, w), y) < 1e-11     # and the round trip at full image size


@pytest.mark.parametrize("C,H,W,k,unit", [(1, 4, 4, 3, True), (1, 3, 5, 2, True), (2, 3, 3, 2, False), (3, 2, 3, 3, False)])
def test_theorem1_recursion_gives_the_inverse_matrix_and_grad_y(C, H, W, k, unit):
    w, _, gx = tiny_inputs(12, 1, C, H, W, k)
    if unit:                                   # the paper's own setting: bottom-right entry 1
        w[np.arange(C), np.arange(C), k - 1, k - 1] = 1.0
    J = dense.theorem1_dx_dy(w, H, W)          # J[q, p] = dx_q/dy_p, entry by entry
    M = dense.dense_matrix(w, H, W)
    assert np.allclose(J @ M, np.eye(H * W * C), atol=1e-12)
    # Eq. 2: dL/dy_p = sum_q dL/dx_q * dx_q/dy_p
    ref = dense.from_vec(J.T @ dense.to_vec(gx[0]), C, H, W)
    assert nmax_err(api.invconv_grad_y(gx, w)[0], ref) < 1e-12
    # zero case: derivative vanishes unless p <= q in the partial order
    for q in range(H * W * C):
        for p in range(H * W * C):
            qh, qw = divmod(q // C, W)
            ph, pw = divmod(p // C, W)
            if not (ph <= qh and pw <= qw):
                assert J[q, p] == 0.0


# ---------------------------------------------------------------- grad_w

def loss(w, y, gx):
    return float(np.sum(gx * api.invconv_forward(y, w)))


@pytest.mark.parametrize("B,C,H,W,k", [(2, 2, 4, 3, 3), (1, 3, 3, 4, 2), (2, 1, 5, 5, 3)])
def test_grad_w_by_central_finite_differences_on_every_tap(B, C, H, W, k):
    w, y, gx = tiny_inputs(13, B, C, H, W, k)
    x = api.invconv_forward(y, w)
    _, gw = api.invconv_backward(gx, x, w)
    eps = 1e-6
    for co in range(C):
        for ci in range(C):
            for a in range(k):
                for b in range(k):
                    if a == k - 1 and b == k - 1 and ci > co:
                        assert gw[co, ci, a, b] == 0.0          # outside the mask: exactly zero
                        continue
                    wp, wm = w.copy(), w.copy()
                    wp[co, ci, a, b] += eps
                    wm[co, ci, a, b] -= eps
                    fd = (loss(wp, y, gx) - loss(wm, y, gx)) / (2 * eps)
                    assert abs(gw[co, ci, a, b] - fd) < 1e-7 * max(1.0, abs(fd)), (co, ci, a, b)


@pytest.mark.parametrize("C,H,W,k,unit", [(1, 4, 4, 3, True), (1, 5, 3, 2, True), (2, 3, 4, 3, False)])
def test_theorem2_recursion_matches_closed_form(C, H, W, k, unit):
    w, y, gx = tiny_inputs(14, 1, C, H, W, k)
    if unit:
        w[np.arange(C), np.arange(C), k - 1, k - 1] = 1.0
    x = api.invconv_forward(y, w)
    _, gw = api.invconv_backward(gx, x, w)
    for co in range(C):
        for ci in range(C):
            for dh in range(k):
                for dw in range(k):
                    if dh == 0 and dw == 0 and ci > co:
                        continue
                    D = dense.theorem2_dx_dw(w, x[0], co, ci, dh, dw)     # dx_q/dW_a for all q
                    ref = float(np.sum(gx[0] * D))                        # sum_q dL/dx_q * dx_q/dW_a
                    got = gw[co, ci, k - 1 - dh, k - 1 - dw]
                    assert abs(got - ref) < 1e-12 * max(1.0, abs(ref))


@pytest.mark.parametrize("name,batch", [("pr1", None), ("mnist", 4), ("cifar_sq", 2), ("wide96_k3", 1), ("large64", 1)])
def test_grad_w_directional_derivative_at_benchmark_shapes(name, batch):
    s, w, y, gx = workloads.make(name, batch=batch)
    w = w.astype(np.float64); y = y.astype(np.float64); gx = gx.astype(np.float64)
    x = api.invconv_forward(y, w)
    _, gw = api.invconv_backward(gx, x, w)
    rng = np.random.default_rng(15)
    for _ in range(2):
        v = rng.normal(size=w.shape)
        v[:, :, s.k - 1, s.k - 1] = np.tril(v[:, :, s.k - 1, s.k - 1])      # stay inside the mask
        eps = 1e-6
        fd = (loss(w + eps * v, y, gx) - loss(w - eps * v, y, gx)) / (2 * eps)
        assert abs(float(np.sum(gw * v)) - fd) < 2e-6 * max(1.0, abs(fd))


# ---------------------------------------------------------------- log-det

@pytest.mark.parametrize("B,C,H,W,k", TINY)
def test_logdet_equals_slogdet_of_dense_matrix(B, C, H, W, k):
    w, _, _ = tiny_inputs(16, B, C, H, W, k)
    w[0, 0, k - 1, k - 1] *= -1.0                 # a negative diagonal entry: log|.|
    sign, lad = np.linalg.slogdet(dense.dense_matrix(w, H, W))
    assert sign != 0
    assert abs(api.logdet(w, H, W) - lad) < 1e-12 * max(1.0, abs(lad))


def test_logdet_scaling_law():
    C, H, W, k = 3, 5, 7, 3
    w, _, _ = tiny_inputs(17, 1, C, H, W, k)
    s = 1.7
    w2 = w.copy()
    w2[np.arange(C), np.arange(C), k - 1, k - 1] *= s
    assert abs(api.logdet(w2, H, W) - api.logdet(w, H, W) - H * W * C * np.log(s)) < 1e-12 * H * W * C


@pytest.mark.parametrize("B,C,H,W,k", TINY)
def test_logdet_gradient_matches_slogdet_differences(B, C, H, W, k):
    """d logdet / d w against central differences of numpy's slogdet of the dense matrix, entry by entry
    (entries outside the mask and off the bottom-right tap's diagonal do not enter M's diagonal: 0)."""
    w, _, _ = tiny_inputs(18, B, C, H, W, k)
    w[C - 1, C - 1, k - 1, k - 1] *= -1.0
    g = api.logdet_grad_w(w, H, W)
    eps = 1e-6
    for idx in np.ndindex(*w.shape):
        co, ci, a, b = idx
        if a == k - 1 and b == k - 1 and ci > co:
            assert g[idx] == 0.0                   # masked out: not part of M
            continue
        wp, wm = w.copy(), w.copy()
        wp[idx] += eps
        wm[idx] -= eps
        fd = (np.linalg.slogdet(dense.dense_matrix(wp, H, W))[1] - np.linalg.slogdet(dense.dense_matrix(wm, H, W))[1]) / (2 * eps)
        assert abs(g[idx] - fd) < 1e-6 * max(1.0, abs(fd)), (idx, g[idx], fd)

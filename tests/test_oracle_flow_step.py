"""Pins of the oracle for the inverse convolution's neighbours in the Inverse-Flow step (Section 4: Inv-Conv,
Actnorm, 1x1 convolution).  CPU only.  Each function is checked against something other than itself: a library
routine for the special case it reduces to, the dense Jacobian of the whole step, central finite differences."""
import numpy as np
import pytest

from oracle import api, dense, flow_step
from paper_2410_14634_b200 import workloads


def draw_neighbours(seed, C):
    rng = np.random.default_rng(seed)
    s = rng.uniform(0.5, 1.5, size=C) * rng.choice([-1.0, 1.0], size=C)
    b = rng.normal(0.0, 0.3, size=C)
    V = np.linalg.qr(rng.normal(size=(C, C)))[0] + 0.1 * rng.normal(size=(C, C))
    return s, b, V


def test_conv1x1_is_the_library_convolution_with_a_one_pixel_kernel():
    import torch
    rng = np.random.default_rng(0)
    z, V = rng.normal(size=(2, 5, 3, 4)), rng.normal(size=(5, 5))
    ref = torch.nn.functional.conv2d(torch.from_numpy(z), torch.from_numpy(V)[:, :, None, None]).numpy()
    assert np.max(np.abs(flow_step.conv1x1(z, V) - ref)) <= 1e-13


def test_actnorm_special_cases():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(2, 3, 4, 4))
    assert np.array_equal(flow_step.actnorm(x, np.ones(3), np.zeros(3)), x)
    z = flow_step.actnorm(x, np.array([2.0, -1.0, 0.5]), np.array([1.0, 0.0, -3.0]))
    assert np.allclose(z[:, 0], 2 * x[:, 0] + 1) and np.allclose(z[:, 1], -x[:, 1]) and np.allclose(z[:, 2], 0.5 * x[:, 2] - 3)


@pytest.mark.parametrize("shape", [(1, 2, 3, 3, 2), (2, 3, 3, 4, 3)], ids=str)
def test_step_forward_and_logdet_match_the_dense_jacobian(shape):
    """u as a function of y is affine; its Jacobian, built from the dense matrix of f and Kronecker-style
    blocks for the neighbours, reproduces u and its log|det| is the step's log-determinant."""
    B, C, H, W, k = shape
    w, y, _ = workloads.make_custom(11, B, C, H, W, k)
    s, b, V = draw_neighbours(5, C)
    x, u, ld = flow_step.step_forward(y, w, s, b, V)
    M = dense.dense_matrix(w, H, W)                       # index (h*W + w)*C + c
    n = H * W * C
    P = np.zeros((n, n))                                  # per-pixel V diag(s)
    off = np.zeros(n)
    for p in range(H * W):
        P[p * C:(p + 1) * C, p * C:(p + 1) * C] = V @ np.diag(s)
        off[p * C:(p + 1) * C] = V @ b
    J = P @ np.linalg.inv(M)
    for i in range(B):
        yv = np.asarray(y[i], dtype=np.float64).transpose(1, 2, 0).reshape(-1)
        uv = J @ yv + off
        assert np.max(np.abs(uv - u[i].transpose(1, 2, 0).reshape(-1))) <= 1e-11
    assert abs(np.linalg.slogdet(J)[1] - ld) <= 1e-9 * max(1.0, abs(ld))


def test_step_backward_matches_central_differences_of_every_parameter():
    B, C, H, W, k = 2, 3, 3, 3, 2
    w, y, gu = workloads.make_custom(21, B, C, H, W, k)
    w, y, gu = (a.astype(np.float64) for a in (w, y, gu))
    s, b, V = draw_neighbours(7, C)
    x, u, _ = flow_step.step_forward(y, w, s, b, V)
    gy, gw, gs, gb, gV = flow_step.step_backward(gu, x, w, s, b, V)

    def loss(y_=y, w_=w, s_=s, b_=b, V_=V):
        return float(np.sum(gu * flow_step.step_forward(y_, w_, s_, b_, V_)[1]))

    eps = 1e-6

    def fd(arr, idx, key):
        hi, lo = arr.copy(), arr.copy()
        hi[idx] += eps
        lo[idx] -= eps
        return (loss(**{key: hi}) - loss(**{key: lo})) / (2 * eps)

    for c in range(C):
        assert abs(fd(s, (c,), "s_") - gs[c]) <= 1e-6 * max(1.0, abs(gs[c]))
        assert abs(fd(b, (c,), "b_") - gb[c]) <= 1e-6 * max(1.0, abs(gb[c]))
        for o in range(C):
            assert abs(fd(V, (o, c), "V_") - gV[o, c]) <= 1e-6 * max(1.0, abs(gV[o, c]))
    rng = np.random.default_rng(3)
    for _ in range(12):
        idx = tuple(rng.integers(0, d) for d in y.shape)
        assert abs(fd(y, idx, "y_") - gy[idx]) <= 1e-6 * max(1.0, abs(gy[idx]))
    for co in range(C):
        for ci in range(C):
            for a in range(k):
                for bb in range(k):
                    if a == k - 1 and bb == k - 1 and ci > co:
                        assert gw[co, ci, a, bb] == 0.0
                        continue
                    assert abs(fd(w, (co, ci, a, bb), "w_") - gw[co, ci, a, bb]) <= 2e-6 * max(1.0, abs(gw[co, ci, a, bb]))


def test_identity_neighbours_reduce_the_step_to_the_inverse_convolution():
    B, C, H, W, k = 2, 2, 4, 5, 3
    w, y, gu = workloads.make_custom(31, B, C, H, W, k)
    s, b, V = np.ones(C), np.zeros(C), np.eye(C)
    x, u, ld = flow_step.step_forward(y, w, s, b, V)
    assert np.array_equal(u, x) and abs(ld + api.logdet(w, H, W)) <= 1e-12
    gy, gw, gs, gb, gV = flow_step.step_backward(gu, x, w, s, b, V)
    gy0, gw0 = api.invconv_backward(gu, x, w)
    assert np.array_equal(gy, gy0) and np.array_equal(gw, gw0)

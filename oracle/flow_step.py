"""Oracle of the layers that follow the inverse convolution inside one step of the paper's Inverse-Flow model
(Section 4, "Inv_Flow" step, Fig. 3: Inv-Conv -> Actnorm -> 1x1 convolution): plain float64 numpy, test
infrastructure only.

    x = f^{-1}(y)                                   the inverse convolution (oracle.api.invconv_forward)
    z[n,c,h,w] = s[c] * x[n,c,h,w] + b[c]           Actnorm: a per-channel affine map
    u[n,o,h,w] = sum_c V[o,c] * z[n,c,h,w]          1x1 convolution: a C x C channel mix at every pixel

Both neighbours act on one pixel at a time, which is what lets a kernel apply them while it stores x
(forward) or loads the incoming gradient (backward).  The step's log-determinant is the sum of the three
layers': -logdet(f) for the inverse convolution, H*W*sum_c log|s_c| for Actnorm, H*W*log|det V| for the 1x1
convolution.  Gradients follow from the chain rule; with grad_z = V^T grad_u (per pixel):

    grad_V[o,c] = sum_{n,h,w} grad_u[n,o,h,w] * z[n,c,h,w]
    grad_s[c]   = sum_{n,h,w} grad_z[n,c,h,w] * x[n,c,h,w]
    grad_b[c]   = sum_{n,h,w} grad_z[n,c,h,w]
    grad_x      = s * grad_z                         then grad_y, grad_w as for the inverse convolution alone.
"""
from __future__ import annotations

import numpy as np

from . import api


def actnorm(x, s, b) -> np.ndarray:
    x, s, b = (np.asarray(a, dtype=np.float64) for a in (x, s, b))
    z = np.empty_like(x)
    for c in range(x.shape[1]):
        z[:, c] = s[c] * x[:, c] + b[c]
    return z


def conv1x1(z, V) -> np.ndarray:
    z, V = np.asarray(z, dtype=np.float64), np.asarray(V, dtype=np.float64)
    C = z.shape[1]
    u = np.zeros_like(z)
    for o in range(C):
        for c in range(C):
            u[:, o] += V[o, c] * z[:, c]
    return u


def step_forward(y, w, s, b, V):
    """(x, u, logdet) of the step y -> u; x is what the backward pass needs saved."""
    x = api.invconv_forward(y, w)
    u = conv1x1(actnorm(x, s, b), V)
    H, W = x.shape[2], x.shape[3]
    s64, V64 = np.asarray(s, dtype=np.float64), np.asarray(V, dtype=np.float64)
    ld = -api.logdet(w, H, W) + H * W * float(np.sum(np.log(np.abs(s64)))) + H * W * float(np.linalg.slogdet(V64)[1])
    return x, u, ld


def step_backward(grad_u, x, w, s, b, V):
    """(grad_y, grad_w, grad_s, grad_b, grad_V) of L through the step, given grad_u and the saved x."""
    grad_u, x, s, b, V = (np.asarray(a, dtype=np.float64) for a in (grad_u, x, s, b, V))
    C = x.shape[1]
    z = actnorm(x, s, b)
    grad_z = np.zeros_like(grad_u)
    for c in range(C):
        for o in range(C):
            grad_z[:, c] += V[o, c] * grad_u[:, o]
    grad_V = np.empty((C, C))
    for o in range(C):
        for c in range(C):
            grad_V[o, c] = np.sum(grad_u[:, o] * z[:, c])
    grad_s = np.array([np.sum(grad_z[:, c] * x[:, c]) for c in range(C)])
    grad_b = np.array([np.sum(grad_z[:, c]) for c in range(C)])
    grad_x = np.empty_like(grad_z)
    for c in range(C):
        grad_x[:, c] = s[c] * grad_z[:, c]
    grad_y, grad_w = api.invconv_backward(grad_x, x, w)
    return grad_y, grad_w, grad_s, grad_b, grad_V

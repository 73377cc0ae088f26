"""ctypes front end of the float64 C oracle (`invconv_oracle.c`).

Test infrastructure only: callers are the tests, the smoke check and the
benchmark's CPU-baseline leg.  Inputs of any float dtype are promoted to
float64 (so fp32 inputs are seen bit-identically by oracle and GPU path);
outputs are float64 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "invconv_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, no fast-math, no threads)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-ffp-contract=off", _SRC, "-o", tmp, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        ci = ctypes.c_int
        for name in ("oracle_masked_conv", "oracle_invconv_forward", "oracle_invconv_grad_y", "oracle_invconv_grad_w"):
            fn = getattr(lib, name)
            fn.argtypes = [dp, dp, dp, ci, ci, ci, ci, ci]
            fn.restype = None
        lib.oracle_logdet.argtypes = [dp, ci, ci, ci, ci]
        lib.oracle_logdet.restype = ctypes.c_double
        lib.oracle_logdet_grad_w.argtypes = [dp, dp, ci, ci, ci, ci]
        lib.oracle_logdet_grad_w.restype = None
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _dims(act: np.ndarray, w: np.ndarray):
    if act.ndim != 4 or w.ndim != 4:
        raise ValueError("activations are [B,C,H,W], kernel is [C,C,k,k]")
    B, C, H, W = act.shape
    if w.shape[0] != C or w.shape[1] != C or w.shape[2] != w.shape[3]:
        raise ValueError(f"kernel shape {w.shape} does not match C={C}")
    return B, C, H, W, w.shape[2]


def masked_conv(x, w) -> np.ndarray:
    """y = f(x), Eq. 1 with the channel mask on the bottom-right tap."""
    x, w = _f64(x), _f64(w)
    B, C, H, W, k = _dims(x, w)
    y = np.empty_like(x)
    _load().oracle_masked_conv(_ptr(x), _ptr(w), _ptr(y), B, C, H, W, k)
    return y


def invconv_forward(y, w) -> np.ndarray:
    """x = f^{-1}(y) by row-major forward substitution."""
    y, w = _f64(y), _f64(w)
    B, C, H, W, k = _dims(y, w)
    x = np.empty_like(y)
    _load().oracle_invconv_forward(_ptr(y), _ptr(w), _ptr(x), B, C, H, W, k)
    return x


def invconv_grad_y(grad_x, w) -> np.ndarray:
    """grad_y = M^{-T} grad_x (Eq. 2 with Theorem 1)."""
    grad_x, w = _f64(grad_x), _f64(w)
    B, C, H, W, k = _dims(grad_x, w)
    gy = np.empty_like(grad_x)
    _load().oracle_invconv_grad_y(_ptr(grad_x), _ptr(w), _ptr(gy), B, C, H, W, k)
    return gy


def invconv_grad_w(grad_y, x, k: int) -> np.ndarray:
    """grad_w = -corr(grad_y, x) on the masked taps (Theorem 2, closed form)."""
    grad_y, x = _f64(grad_y), _f64(x)
    if grad_y.shape != x.shape or x.ndim != 4:
        raise ValueError("grad_y and x must both be [B,C,H,W]")
    B, C, H, W = x.shape
    gw = np.empty((C, C, k, k), dtype=np.float64)
    _load().oracle_invconv_grad_w(_ptr(grad_y), _ptr(x), _ptr(gw), B, C, H, W, k)
    return gw


def invconv_backward(grad_x, x, w):
    """(grad_y, grad_w) of L through x = f^{-1}(y), given grad_x and the saved x."""
    gy = invconv_grad_y(grad_x, w)
    gw = invconv_grad_w(gy, x, np.asarray(w).shape[2])
    return gy, gw


def logdet(w, H: int, W: int) -> float:
    """H*W*sum_c log|w[c,c,k-1,k-1]|  (log|det df/dx|)."""
    w = _f64(w)
    if w.ndim != 4:
        raise ValueError("kernel is [C,C,k,k]")
    return float(_load().oracle_logdet(_ptr(w), w.shape[0], H, W, w.shape[2]))


def logdet_grad_w(w, H: int, W: int) -> np.ndarray:
    """d logdet / d w: H*W / w[c,c,k-1,k-1] on the channel diagonal of the bottom-right tap, 0 elsewhere."""
    w = _f64(w)
    if w.ndim != 4:
        raise ValueError("kernel is [C,C,k,k]")
    gw = np.empty_like(w)
    _load().oracle_logdet_grad_w(_ptr(w), _ptr(gw), w.shape[0], H, W, w.shape[2])
    return gw

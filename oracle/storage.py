"""Oracle of the reduced-precision storage variant: activations (y, x, grad_x, grad_y) live in memory as bfloat16
while every sum of the method (the substitution chain of Section 3, the gradients of Theorems 1 and 2) is
carried in full precision.  Plain float64 numpy, test infrastructure only.

The paper has no such variant; it is a bandwidth option of this library for the batch-scaling regime (the
paper's batch-size ablation in the supplementary material), so what is stated here is only the number format:
bfloat16 = sign, 8 exponent bits (bias 127), 7 stored fraction bits -> 8 significant bits; conversion rounds to
the nearest representable value, ties to the one with an even last bit; magnitudes below 2^-126 lie on the
fixed subnormal grid 2^-133; magnitudes that round beyond the largest finite value become infinite.

    x_stored = round_to_bf16(f^{-1}(y_stored))            (y_stored holds bfloat16 values)
    grad_y_stored = round_to_bf16(M^{-T} grad_x_stored)
    grad_w = -corr(M^{-T} grad_x_stored, x_stored) on the mask   (weights and their gradient stay float32)
"""
from __future__ import annotations

import numpy as np

_SIG_BITS = 8                 # significant bits of bfloat16 (one implicit)
_MIN_NORMAL_EXP = -126        # 2^-126 is the smallest normal magnitude
_MAX_FINITE = (2.0 - 2.0 ** -7) * 2.0 ** 127


def round_to_bf16(a) -> np.ndarray:
    """Nearest bfloat16 value of every element (ties to even), returned as float64."""
    a = np.asarray(a, dtype=np.float64)
    out = np.array(a, copy=True)
    finite = np.isfinite(a) & (a != 0.0)
    v = a[finite]
    # v = m * 2^e with 0.5 <= |m| < 1  ->  the leading bit of v has weight 2^(e-1)
    _, e = np.frexp(v)
    lead = np.maximum(e - 1, _MIN_NORMAL_EXP)
    quantum = np.ldexp(1.0, lead - (_SIG_BITS - 1))          # spacing of bfloat16 values in v's binade
    r = np.rint(v / quantum) * quantum                        # np.rint rounds halves to even
    r = np.where(np.abs(r) > _MAX_FINITE, np.copysign(np.inf, v), r)
    out[finite] = r
    return out


def bf16_spacing(a) -> np.ndarray:
    """Distance between neighbouring bfloat16 values around every element (the quantum of its binade)."""
    a = np.abs(np.asarray(a, dtype=np.float64))
    _, e = np.frexp(np.where(a == 0.0, 2.0 ** _MIN_NORMAL_EXP, a))
    lead = np.maximum(e - 1, _MIN_NORMAL_EXP)
    return np.ldexp(1.0, lead - (_SIG_BITS - 1))

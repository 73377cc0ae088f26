"""Seeded synthetic inputs shaped like the paper's flow workloads.

This module only draws random numbers: it holds none of the method's
arithmetic and imports neither the CUDA binding nor the CPU oracle, so both
sides of a parity test can be fed from it.

The paper trains on MNIST (1x28x28) and CIFAR10 (3x32x32, squeezed to
12x16x16, 48x8x8 ...) (Section 5); the operator's control flow does not depend
on the data, so standard-normal tensors of those shapes stand in for the
datasets.  Recipe, per workload (one `numpy.random.default_rng(seed)` per
config; sub-shapes of one config draw from the same generator in listed order):

    1. every off-centre tap                 ~ N(0, sigma)      (sigma is a std-dev)
    2. the centre tap's strict lower part   ~ N(0, sigma)      (ci < co)
    3. the centre tap's channel diagonal    ~ U(lo, hi)
    4. y                                    ~ N(0, 1)
    5. grad_x                               ~ N(0, 1)

"Centre tap" is the bottom-right kernel entry w[:, :, k-1, k-1], the one that
multiplies the output pixel itself under top-left padding.  Entries outside the
channel mask (ci > co on that tap) are filled with `masked_fill` (default 0);
they are never supposed to be read.  Everything is drawn in float64 and rounded
to float32 once; a float64 consumer promotes those float32 values back, so that
every implementation sees bit-identical inputs.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Shape:
    name: str
    config: int          # 1-based index into the five benchmark configs
    B: int
    C: int
    H: int
    W: int
    k: int
    sigma: float
    diag_lo: float
    diag_hi: float
    seed: int

    @property
    def elements(self) -> int:
        return self.B * self.C * self.H * self.W

    @property
    def n_diagonals(self) -> int:
        return self.H + self.W - 1


SHAPES = (
    Shape("pr1", 1, 4, 3, 16, 16, 3, 0.05, 0.8, 1.2, 0),
    Shape("mnist", 2, 256, 1, 28, 28, 3, 0.05, 0.8, 1.2, 1),
    Shape("cifar", 3, 256, 3, 32, 32, 3, 0.05, 0.8, 1.2, 2),
    Shape("cifar_sq", 3, 256, 12, 16, 16, 3, 0.05, 0.8, 1.2, 2),
    Shape("wide48_k3", 4, 64, 48, 16, 16, 3, 0.05 / math.sqrt(48), 0.8, 1.2, 3),
    Shape("wide48_k5", 4, 64, 48, 16, 16, 5, 0.05 / math.sqrt(48), 0.8, 1.2, 3),
    Shape("wide96_k3", 4, 64, 96, 8, 8, 3, 0.05 / math.sqrt(96), 0.8, 1.2, 3),
    Shape("wide96_k5", 4, 64, 96, 8, 8, 5, 0.05 / math.sqrt(96), 0.8, 1.2, 3),
    Shape("large64", 5, 16, 3, 64, 64, 5, 0.05, 0.9, 1.1, 4),
    Shape("large256", 5, 4, 1, 256, 256, 5, 0.05, 0.9, 1.1, 4),
)
BY_NAME = {s.name: s for s in SHAPES}


def draw(rng: np.random.Generator, B: int, C: int, H: int, W: int, k: int,
         sigma: float, diag_lo: float, diag_hi: float, masked_fill: float = 0.0):
    """One (w, y, grad_x) triple in float32, drawn in the fixed order above."""
    w = np.empty((C, C, k, k), dtype=np.float64)
    off = rng.normal(0.0, sigma, size=(C, C, k, k))
    centre_lower = rng.normal(0.0, sigma, size=(C, C))
    diag = rng.uniform(diag_lo, diag_hi, size=C)
    w[...] = off
    centre = np.full((C, C), masked_fill, dtype=np.float64)
    il = np.tril_indices(C, -1)
    centre[il] = centre_lower[il]
    centre[np.arange(C), np.arange(C)] = diag
    w[:, :, k - 1, k - 1] = centre
    y = rng.normal(0.0, 1.0, size=(B, C, H, W))
    grad_x = rng.normal(0.0, 1.0, size=(B, C, H, W))
    return w.astype(np.float32), y.astype(np.float32), grad_x.astype(np.float32)


def make(name: str, masked_fill: float = 0.0, batch: int | None = None):
    """Inputs of a named benchmark shape.  Sub-shapes of one config share a
    generator, so earlier sub-shapes are drawn (and discarded) first.
    `batch` overrides B *after* the draw position is fixed by the full-size
    earlier sub-shapes (used for bounded CPU samples of a workload)."""
    target = BY_NAME[name]
    rng = np.random.default_rng(target.seed)
    for s in SHAPES:
        if s.config != target.config:
            continue
        B = s.B
        if s.name == name and batch is not None:
            B = batch
        w, y, gx = draw(rng, B, s.C, s.H, s.W, s.k, s.sigma, s.diag_lo, s.diag_hi, masked_fill)
        if s.name == name:
            return s, w, y, gx
    raise KeyError(name)


def make_custom(seed: int, B: int, C: int, H: int, W: int, k: int, sigma: float = 0.05,
                diag_lo: float = 0.8, diag_hi: float = 1.2, masked_fill: float = 0.0):
    """Inputs of an arbitrary shape (edge cases, ragged sizes) from the same recipe."""
    return draw(np.random.default_rng(seed), B, C, H, W, k, sigma, diag_lo, diag_hi, masked_fill)

"""fp64 reference of the decode linear layers, y = x . w^T (the projections whose flops the paper's
T_compute^d counts as BS * (8 h1^2 + 4 h1 h2) per layer, Section IV-C).

TEST INFRASTRUCTURE ONLY.  The definition written out: every output is the plain dot product of a
token row with a weight row, accumulated in fp64 over inputs widened exactly from their 16-bit
values.  ``numpy.matmul`` serves as the contraction step.
"""
from __future__ import annotations

import numpy as np

from .attn import to_f64


def linear(x, w) -> np.ndarray:
    """x [M, K], w [N, K] (fp16 numpy, bf16 torch or float arrays) -> y [M, N] float64."""
    x64 = to_f64(x)
    w64 = to_f64(w)
    assert x64.ndim == 2 and w64.ndim == 2 and x64.shape[1] == w64.shape[1]
    return np.matmul(x64, w64.T)


def linear_flops_per_layer(BS: int, h1: int, h2: int) -> float:
    """Flops of one layer's decode projections: QKV (3 h1^2), output (h1^2) and the two MLP
    matrices (2 h1 h2), two flops per multiply-add: BS * (8 h1^2 + 4 h1 h2)."""
    return 2.0 * BS * (3 * h1 * h1 + h1 * h1 + 2 * h1 * h2)

"""fp64 CPU oracle of the batch-invariant linear layer and of RMS normalisation
(Sec. "Relational Kernel Contracts": matmul of M x K token rows with fixed
weights; Sec. "Relational Structural Analysis": zero fp32 accumulator, products
accumulated over the whole contracted range; the normalisation kernels of the
evaluation table).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline may import this; the product path must not.  It shares nothing with
the CUDA library.  The definitions are the mathematical ones written out in
fp64 on the exactly widened bf16 inputs: y = x W^T, and
y = x / sqrt(mean(x^2) + eps) * w.  bf16 tensors cross as numpy.uint16 bit
patterns.
"""
from __future__ import annotations

import numpy as np


def widen(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64, exactly."""
    b = np.ascontiguousarray(bits)
    assert b.dtype == np.uint16, b.dtype
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def linear(x_bits: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """x [M, K], w [N, K] (one weight row per output feature) -> y [M, N] = x w^T in fp64."""
    x, w = widen(x_bits), widen(w_bits)
    assert x.ndim == 2 and w.ndim == 2 and x.shape[1] == w.shape[1]
    return x @ w.T


def rmsnorm(x_bits: np.ndarray, w_bits: np.ndarray, eps: float) -> np.ndarray:
    """x [M, K], w [K] -> y [M, K] = x * rsqrt(mean_k x^2 + eps) * w in fp64."""
    x, w = widen(x_bits), widen(w_bits)
    assert x.ndim == 2 and w.shape == (x.shape[1],)
    ms = (x * x).sum(axis=1, keepdims=True) / x.shape[1]
    return x / np.sqrt(ms + float(eps)) * w

"""Definitional tier of the oracle in numpy fp64: the paper's formulas taken literally.

TEST INFRASTRUCTURE ONLY.  Used to pin the fp32 oracle (`dhq_oracle.c`): the Hadamard matrix of
Eq. 3, the two-sided orthonormal transform of Eq. 4-5, and the unquantized SIREN forward that a
quantized network must approach as the bit-width grows.
"""
from __future__ import annotations

import numpy as np


def hadamard(n: int) -> np.ndarray:
    """Eq. 3 by block doubling, fp64."""
    assert n >= 1 and n & (n - 1) == 0
    H = np.ones((1, 1))
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


def transform_2d(W: np.ndarray) -> np.ndarray:
    """Eq. 5: W' = H_m W H_n / sqrt(m n)."""
    m, n = W.shape
    return hadamard(m) @ W.astype(np.float64) @ hadamard(n) / np.sqrt(m * n)


def input_side_fold(W: np.ndarray) -> np.ndarray:
    """W H_K / K: the factor of Eq. 4 that acts on the input dimension, scaled so that
    (W H_K / K)(H_K x) = W x."""
    K = W.shape[1]
    return W.astype(np.float64) @ hadamard(K) / K


def siren_forward(weights, biases, omega0: float, coords: np.ndarray) -> np.ndarray:
    """Unquantized fp64 SIREN: sin(omega0 (W x + b)) per hidden layer, affine last layer
    (Section III-C: the output layer has no activation)."""
    x = coords.astype(np.float64)
    L = len(weights)
    for l in range(L):
        z = x @ weights[l].astype(np.float64).T + biases[l].astype(np.float64)
        x = np.sin(omega0 * z) if l < L - 1 else z
    return x

"""Definitional tier of the oracle in numpy fp64: the paper's formulas taken literally.

TEST INFRASTRUCTURE ONLY.  Used to pin the fp32 oracle (`dhq_oracle.c`): the Hadamard matrix of
Eq. 3, the two-sided orthonormal transform of Eq. 4-5, and the unquantized SIREN forward that a
quantized network must approach as the bit-width grows, and one DHQ layer with every step in
fp64 and the orthonormal scaling (the tier the fp32 oracle's codes are compared with: they may
differ only by one code step where the value to be rounded sits next to a half-integer).
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


def gabor(z: np.ndarray, omega0: float, s0: float) -> np.ndarray:
    """Real Gabor wavelet (the reading of the WIRE activation): sin(omega0 z) exp(-(s0 z)^2)."""
    return np.sin(omega0 * z) * np.exp(-(s0 * z) ** 2)


def siren_forward(weights, biases, omega0: float, coords: np.ndarray, gabor_s0: float = 0.0) -> np.ndarray:
    """Unquantized fp64 network: sin(omega0 (W x + b)) per hidden layer (or the Gabor wavelet with
    gabor_s0 > 0), affine last layer (Section III-C: the output layer has no activation)."""
    x = coords.astype(np.float64)
    L = len(weights)
    for l in range(L):
        z = x @ weights[l].astype(np.float64).T + biases[l].astype(np.float64)
        x = (gabor(z, omega0, gabor_s0) if gabor_s0 > 0 else np.sin(omega0 * z)) if l < L - 1 else z
    return x


def quantize_def(v: np.ndarray, a, bits: int):
    """The symmetric absmax quantizer of Section III-B in fp64: t = v * qmax / a, q = round half to
    even of t, clipped to +-qmax; a = 0 gives zeros.  `a` broadcasts against v.  Returns (q, t)."""
    qmax = float(2 ** (bits - 1) - 1)
    a = np.broadcast_to(np.asarray(a, dtype=np.float64), v.shape)
    t = np.divide(v * qmax, a, out=np.zeros_like(v, dtype=np.float64), where=a > 0)
    return np.clip(np.rint(t), -qmax, qmax).astype(np.int64), t


def dhq_layer_def(W, b, X, w_bits: int, a_bits: int, per_channel: bool, per_token: bool, omega0: float,
                  sine: bool, a_frozen=None):
    """One DHQ layer exactly as the formulas read, everything in fp64 with the orthonormal scaling
    of Eq. 5 on the input dimension: W' = W H_K / sqrt(K), x' = H_K x / sqrt(K) (so W' x' = W x),
    both quantized by the same absmax quantizer, integer product, dequantization, bias, sine.
    W is the zero-padded [M][K] matrix, X the [n][K] layer inputs.  a_frozen is the per-tensor
    activation absmax in the orthonormal scaling; None takes the maximum over X.
    Returns a dict: qw, tw (pre-rounding weight values), codes, t (pre-rounding), acc, Y, a_x."""
    W = np.asarray(W, dtype=np.float64)
    X = np.asarray(X, dtype=np.float64)
    M, K = W.shape
    H = hadamard(K)
    Wr = W @ H / np.sqrt(K)
    Xr = X @ H.T / np.sqrt(K)
    a_w = np.abs(Wr).max(axis=1, keepdims=True) if per_channel else np.full((M, 1), np.abs(Wr).max())
    qw, tw = quantize_def(Wr, a_w, w_bits)
    if per_token:
        a_x = np.abs(Xr).max(axis=1, keepdims=True)
    else:
        a_x = np.full((X.shape[0], 1), np.abs(Xr).max() if a_frozen is None else float(a_frozen))
    codes, t = quantize_def(Xr, a_x, a_bits)
    acc = codes @ qw.T
    s_w = a_w[:, 0] / float(2 ** (w_bits - 1) - 1)
    s_x = a_x / float(2 ** (a_bits - 1) - 1)
    z = s_w[None, :] * s_x * acc + np.asarray(b, dtype=np.float64)[None, :]
    return {"qw": qw, "tw": tw, "codes": codes, "t": t, "acc": acc, "Y": np.sin(omega0 * z) if sine else z,
            "a_x": a_x[:, 0]}


def w8a32_layer(qw, s_w, b, X, rotate: bool, omega0: float, sine: bool) -> np.ndarray:
    """One layer of the weight-only quantized network (the W8A32 datapath of Section I / Table 2):
    quantized weights q_w with scales s_w (from the same weight-side fold and quantizer as DHQ),
    activations left in floating point.  x~ = H_K x (or x itself without the rotation), exactly, in
    fp64; z = s_w[m] * sum_k q_w[m][k] x~_k + b[m]; sin(omega0 z) for hidden layers.
    qw [M][K] integers, s_w [M], b [M], X [n][K]."""
    X = np.asarray(X, dtype=np.float64)
    K = X.shape[1]
    Xr = X @ hadamard(K).T if rotate else X
    z = (Xr @ np.asarray(qw, dtype=np.float64).T) * np.asarray(s_w, dtype=np.float64)[None, :] + np.asarray(b, dtype=np.float64)[None, :]
    return np.sin(omega0 * z) if sine else z


def pad_first_input(coords: np.ndarray) -> np.ndarray:
    """[x, y] -> [x, y, 0, 0]: the first layer's input padded to the Hadamard size 4."""
    c = np.asarray(coords, dtype=np.float64)
    X = np.zeros((c.shape[0], 4))
    X[:, : c.shape[1]] = c
    return X

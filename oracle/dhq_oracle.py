"""ctypes binding and network-level driver for the C oracle in `dhq_oracle.c`.

TEST INFRASTRUCTURE ONLY (parity tests, the smoke check and the CPU-baseline timing).  The C
file holds the per-layer arithmetic; this file pads, chains layers and freezes per-tensor
activation scales, following Section III-B/C of the paper with the readings listed in the C
file's header.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dhq_oracle.c")
_LIB = os.path.join(_HERE, "libdhq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction) and return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
               "-fvisibility=hidden", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        c_i, c_i64, c_f, c_d, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_double, ctypes.c_void_p
        L.dhq_orc_threads.restype = c_i
        L.dhq_orc_hadamard.argtypes = [c_i, vp]
        L.dhq_orc_hadamard.restype = c_i
        L.dhq_orc_rotate_rows.argtypes = [vp, c_i, c_i64, vp, vp]
        L.dhq_orc_rotate_rows.restype = None
        L.dhq_orc_rotate_rows_butterfly.argtypes = [c_i, c_i64, vp, vp]
        L.dhq_orc_rotate_rows_butterfly.restype = None
        L.dhq_orc_absmax.argtypes = [vp, c_i64]
        L.dhq_orc_absmax.restype = c_f
        L.dhq_orc_scales.argtypes = [c_f, c_i, vp, vp]
        L.dhq_orc_scales.restype = None
        L.dhq_orc_quantize.argtypes = [vp, c_i64, c_f, c_i, vp]
        L.dhq_orc_quantize.restype = None
        L.dhq_orc_prepare_layer.argtypes = [vp, c_i, c_i, c_i, c_i, c_i, c_i, c_i, vp, vp, vp]
        L.dhq_orc_prepare_layer.restype = c_i
        L.dhq_orc_rotated_absmax.argtypes = [vp, c_i64, c_i, c_i, vp]
        L.dhq_orc_rotated_absmax.restype = None
        L.dhq_orc_layer.argtypes = [vp, c_i64, c_i, c_i, vp, vp, vp, c_i, c_i, c_f, c_i, c_d, c_i,
                                    vp, vp, vp, vp, vp, c_d]
        L.dhq_orc_layer.restype = c_i
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().dhq_orc_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def hadamard(n: int) -> np.ndarray:
    """H_n by the recursion of Eq. 3, int8 [n][n]."""
    H = np.empty((n, n), dtype=np.int8)
    if lib().dhq_orc_hadamard(n, _p(H)) != 0:
        raise ValueError("Hadamard size must be a power of two")
    return H


def rotate(V) -> np.ndarray:
    """Tree(H_n v) for each row of V (fp32, balanced pairwise sum in index order)."""
    V = _f32(np.atleast_2d(V))
    rows, n = V.shape
    out = np.empty_like(V)
    lib().dhq_orc_rotate_rows(_p(hadamard(n)), n, rows, _p(V), _p(out))
    return out


def rotate_butterfly(V) -> np.ndarray:
    V = _f32(np.atleast_2d(V))
    rows, n = V.shape
    out = np.empty_like(V)
    lib().dhq_orc_rotate_rows_butterfly(n, rows, _p(V), _p(out))
    return out


def scales(a: float, bits: int):
    s, inv = ctypes.c_float(), ctypes.c_float()
    lib().dhq_orc_scales(ctypes.c_float(a), bits, ctypes.byref(s), ctypes.byref(inv))
    return np.float32(s.value), np.float32(inv.value)


def absmax(v) -> np.float32:
    v = _f32(v).ravel()
    return np.float32(lib().dhq_orc_absmax(_p(v), v.size))


def quantize(v, inv, bits: int) -> np.ndarray:
    v = _f32(v)
    q = np.empty(v.shape, dtype=np.int32)
    lib().dhq_orc_quantize(_p(v), v.size, ctypes.c_float(float(inv)), bits, _p(q))
    return q


def pad_dims(dims, l: int):
    """(K_pad, M_pad) of linear layer l (1-based): the 2 inputs pad to 4 and the outputs of the
    last layer pad to 4, so that both Hadamard sizes are powers of two."""
    L = len(dims) - 1
    K_pad = 4 if l == 1 else int(dims[l - 1])
    M_pad = 4 if l == L else int(dims[l])
    return K_pad, M_pad


@dataclass
class OracleLayer:
    K_pad: int
    M_pad: int
    Wrot: np.ndarray      # fp32 [M_pad][K_pad], rotated and scaled by 1/K_pad
    qw: np.ndarray        # int32 [M_pad][K_pad]
    s_w: np.ndarray       # fp32 [M_pad]
    b_pad: np.ndarray     # fp32 [M_pad]
    sine: bool
    a_frozen: float = float("nan")   # per-tensor activation absmax once calibrated


@dataclass
class OracleNet:
    dims: tuple
    omega0: float
    w_bits: int
    a_bits: int
    w_gran: int
    a_gran: int
    rotate: int           # 0: none, 1: input side (the hot path), 2: both sides (Eq. 4-5 literally)
    layers: list
    gabor_s0: float = 0.0  # > 0: hidden layers use the real Gabor wavelet sin(omega0 z) exp(-(s0 z)^2) (WIRE reading)


def _rot_mode(rotate) -> int:
    """True / 1: input side; False / 0: none; "both" / 2: both sides."""
    if rotate is True or rotate is False:
        return int(rotate)
    if rotate == "both" or rotate == 2:
        return 2
    return int(bool(rotate))


def prepare(weights, biases, dims, omega0, w_bits=8, a_bits=8, w_gran=0, a_gran=0, rotate=True, gabor_s0=0.0) -> OracleNet:
    """Weight-side fold and quantizer for every layer (Eq. 4-5: rotate=True the input-side factor,
    rotate="both" the two-sided transform, rotate=False none)."""
    mode = _rot_mode(rotate)
    L = len(dims) - 1
    layers = []
    for l in range(1, L + 1):
        K_pad, M_pad = pad_dims(dims, l)
        W = _f32(weights[l - 1])
        d_out, d_in = W.shape
        Wrot = np.empty((M_pad, K_pad), dtype=np.float32)
        qw = np.empty((M_pad, K_pad), dtype=np.int32)
        s_w = np.empty(M_pad, dtype=np.float32)
        rc = lib().dhq_orc_prepare_layer(_p(W), d_out, d_in, M_pad, K_pad, w_bits, int(w_gran),
                                         mode, _p(Wrot), _p(qw), _p(s_w))
        if rc != 0:
            raise RuntimeError(f"oracle prepare failed ({rc})")
        b_pad = np.zeros(M_pad, dtype=np.float32)
        b_pad[:d_out] = _f32(biases[l - 1])
        layers.append(OracleLayer(K_pad, M_pad, Wrot, qw, s_w, b_pad, sine=(l < L)))
    return OracleNet(tuple(dims), float(omega0), w_bits, a_bits, int(w_gran), int(a_gran), mode, layers, float(gabor_s0))


def pad_coords(coords) -> np.ndarray:
    """X_1 = [x, y, 0, 0] for every token."""
    c = _f32(coords)
    X = np.zeros((c.shape[0], 4), dtype=np.float32)
    X[:, : c.shape[1]] = c
    return X


def rotated_absmax(net: OracleNet, l: int, X) -> np.ndarray:
    """Per-token absmax of the rotated input of layer l (1-based)."""
    X = _f32(X)
    lay = net.layers[l - 1]
    amax = np.empty(X.shape[0], dtype=np.float32)
    lib().dhq_orc_rotated_absmax(_p(X), X.shape[0], lay.K_pad, int(net.rotate != 0), _p(amax))
    return amax


def layer(net: OracleNet, l: int, X, want=("Xrot", "codes", "s_x", "acc", "Y"), a_frozen=None):
    """Layer l (1-based) applied to the given fp32 inputs X [n][K_pad] (teacher forcing when X
    comes from elsewhere).  Returns a dict with the requested arrays."""
    X = _f32(X)
    n = X.shape[0]
    lay = net.layers[l - 1]
    assert X.shape[1] == lay.K_pad
    out = {
        "Xrot": np.empty((n, lay.K_pad), np.float32) if "Xrot" in want else None,
        "codes": np.empty((n, lay.K_pad), np.int32) if "codes" in want else None,
        "s_x": np.empty(n, np.float32) if "s_x" in want else None,
        "acc": np.empty((n, lay.M_pad), np.int64) if "acc" in want else None,
        "Y": np.empty((n, lay.M_pad), np.float64) if "Y" in want else None,
    }
    per_token = int(net.a_gran == 1)
    if per_token:
        af = 0.0
    else:
        af = lay.a_frozen if a_frozen is None else a_frozen
        if not np.isfinite(af):
            raise RuntimeError("per-tensor activation scale of this layer is not calibrated")
    rc = lib().dhq_orc_layer(_p(X), n, lay.K_pad, lay.M_pad, _p(lay.qw), _p(lay.s_w), _p(lay.b_pad),
                             net.a_bits, per_token, ctypes.c_float(float(af)), int(lay.sine),
                             ctypes.c_double(net.omega0), int(net.rotate), _p(out["Xrot"]),
                             _p(out["codes"]), _p(out["s_x"]), _p(out["acc"]), _p(out["Y"]), ctypes.c_double(net.gabor_s0))
    if rc == -3 and max(net.a_bits, net.w_bits) <= 8:
        raise OverflowError("accumulator left the int32 range")
    if rc not in (0, -3):
        raise RuntimeError(f"oracle layer failed ({rc})")
    return {k: v for k, v in out.items() if v is not None}


def calibrate(net: OracleNet, coords) -> list:
    """Freeze per-tensor activation scales layer by layer: layer l's absmax is taken over all
    calibration tokens with layers < l already quantized.  Returns the frozen values."""
    X = pad_coords(coords)
    frozen = []
    for l in range(1, len(net.layers) + 1):
        a = float(rotated_absmax(net, l, X).max()) if X.shape[0] else 0.0
        net.layers[l - 1].a_frozen = a
        frozen.append(a)
        if l < len(net.layers):
            X = layer(net, l, X, want=("Y",))["Y"].astype(np.float32)
    return frozen


def forward(net: OracleNet, coords, return_layers=False):
    """Free-running chain: X_{l+1} = fp32(Y_l).  Returns the fp64 output [n][d_L] (and, on
    request, the per-layer dicts)."""
    X = pad_coords(coords)
    per = []
    L = len(net.layers)
    for l in range(1, L + 1):
        want = ("Xrot", "codes", "s_x", "acc", "Y") if return_layers else ("Y",)
        r = layer(net, l, X, want=want)
        if return_layers:
            r["X"] = X
            per.append(r)
        if l < L:
            X = r["Y"].astype(np.float32)
    out = r["Y"][:, : net.dims[-1]]
    return (out, per) if return_layers else out


def forward_w8a32(net: OracleNet, coords, chain_fp32=True, return_layers=False):
    """Weight-only quantized forward (W8A32): the weights of `net` (folded and quantized exactly as
    for DHQ), activations not quantized.  Each layer is odef.w8a32_layer in fp64; between layers
    the activation is rounded to fp32 (chain_fp32), as a datapath with fp32 activations holds it."""
    from . import odef
    X = odef.pad_first_input(coords)
    if chain_fp32:
        X = X.astype(np.float32).astype(np.float64)
    per = []
    L = len(net.layers)
    for l, lay in enumerate(net.layers, start=1):
        Y = odef.w8a32_layer(lay.qw, lay.s_w, lay.b_pad, X, net.rotate == 1, net.omega0, lay.sine)
        per.append({"X": X.astype(np.float32), "Y": Y})
        if l < L:
            X = Y.astype(np.float32).astype(np.float64) if chain_fp32 else Y
    out = Y[:, : net.dims[-1]]
    return (out, per) if return_layers else out


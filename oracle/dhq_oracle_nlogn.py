"""Driver for `dhq_oracle_nlogn.c`: the same layer and the same free-running chain as
`dhq_oracle.py`, with the rotation as an O(n log n) butterfly.

TEST INFRASTRUCTURE ONLY: the second timed CPU baseline.  It reuses the network description
(`OracleNet`: padded, rotated, quantized weights) prepared by `dhq_oracle.prepare`; only the
per-token work differs.  Not the parity reference.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import dhq_oracle as _orc

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dhq_oracle_nlogn.c")
_LIB = os.path.join(_HERE, "libdhq_oracle_nlogn.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
                        "-fvisibility=hidden", "-o", _LIB, _SRC, "-lm"], check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        c_i, c_i64, c_f, c_d, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_double, ctypes.c_void_p
        L.dhq_orcn_layer.argtypes = [vp, c_i64, c_i, c_i, vp, vp, vp, c_i, c_i, c_f, c_i, c_d, c_i, vp, vp, vp, vp, vp]
        L.dhq_orcn_layer.restype = c_i
        _lib = L
    return _lib


def layer(net, l: int, X, want=("Xrot", "codes", "s_x", "acc", "Y"), a_frozen=None):
    """Layer l (1-based) of `net` on the fp32 inputs X [n][K_pad]; same outputs as dhq_oracle.layer."""
    X = np.ascontiguousarray(X, dtype=np.float32)
    n = X.shape[0]
    lay = net.layers[l - 1]
    out = {
        "Xrot": np.empty((n, lay.K_pad), np.float32) if "Xrot" in want else None,
        "codes": np.empty((n, lay.K_pad), np.int32) if "codes" in want else None,
        "s_x": np.empty(n, np.float32) if "s_x" in want else None,
        "acc": np.empty((n, lay.M_pad), np.int64) if "acc" in want else None,
        "Y": np.empty((n, lay.M_pad), np.float64) if "Y" in want else None,
    }
    if net.gabor_s0 > 0:
        raise NotImplementedError("the O(n log n) baseline covers the sine network only")
    per_token = int(net.a_gran == 1)
    af = 0.0 if per_token else (lay.a_frozen if a_frozen is None else a_frozen)
    if not np.isfinite(af):
        raise RuntimeError("per-tensor activation scale of this layer is not calibrated")
    p = _orc._p
    rc = lib().dhq_orcn_layer(p(X), n, lay.K_pad, lay.M_pad, p(lay.qw), p(lay.s_w), p(lay.b_pad), net.a_bits,
                              per_token, ctypes.c_float(float(af)), int(lay.sine), ctypes.c_double(net.omega0),
                              int(net.rotate), p(out["Xrot"]), p(out["codes"]), p(out["s_x"]), p(out["acc"]), p(out["Y"]))
    if rc != 0:
        raise RuntimeError(f"nlogn oracle layer failed ({rc})")
    return {k: v for k, v in out.items() if v is not None}


def forward(net, coords):
    """Free-running chain X_{l+1} = fp32(Y_l); fp64 output [n][d_L]."""
    X = _orc.pad_coords(coords)
    L = len(net.layers)
    for l in range(1, L + 1):
        Y = layer(net, l, X, want=("Y",))["Y"]
        if l < L:
            X = Y.astype(np.float32)
    return Y[:, : net.dims[-1]]

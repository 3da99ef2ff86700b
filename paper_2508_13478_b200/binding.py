"""ctypes binding over libdhq_b200.so: argument marshalling only.

Function names and argument order follow `include/dhq.h`.  Tensors are torch CUDA tensors (used
for device memory and streams only); every step of the forward path runs inside the library's
kernels.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdhq_b200.so")
_lib = None

DHQ_GRAN_TENSOR = 0
DHQ_GRAN_CHANNEL_OR_TOKEN = 1
DHQ_ROT_INPUT = 0
DHQ_ROT_BOTH = 1
DHQ_ROT_NONE = 2
DHQ_STATIC_MAX_TOKENS = 4096
DHQ_BITS_FLOAT = 32
DHQ_ACT_SINE = 0
DHQ_ACT_GABOR = 1

PIPES = {"ffma": 0, "fadd": 1, "mufu_sin": 2, "i2f": 3, "f2i": 4, "prmt": 5, "fmnmx": 6, "tensor_i8": 7, "fadd2": 8, "ffma2": 9,
         "pass1": 10, "pass2": 11, "pass12": 12}


class DhqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        super().__init__(f"{where}: {dhq_status_string(code)} (status {code})")


class _Config(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int), ("dims", ctypes.POINTER(ctypes.c_int)),
                ("w_bits", ctypes.c_int), ("a_bits", ctypes.c_int), ("omega0", ctypes.c_float),
                ("w_gran", ctypes.c_int), ("a_gran", ctypes.c_int), ("rotation", ctypes.c_int),
                ("activation", ctypes.c_int), ("act_s0", ctypes.c_float)]


class _DebugBufs(ctypes.Structure):
    _fields_ = [("X", ctypes.POINTER(ctypes.c_void_p)), ("codes", ctypes.POINTER(ctypes.c_void_p)),
                ("s_x", ctypes.POINTER(ctypes.c_void_p)), ("acc", ctypes.POINTER(ctypes.c_void_p)),
                ("Y", ctypes.POINTER(ctypes.c_void_p))]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libdhq_b200.so; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2508_13478_b200.build` "
                          "(nvcc, sm_100a); this package has no fallback path")
    L = ctypes.CDLL(_LIB_PATH)
    vp, c_i, c_i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    L.dhq_prepare.argtypes = [ctypes.POINTER(_Config), ctypes.POINTER(vp), ctypes.POINTER(vp), vp, ctypes.POINTER(vp)]
    L.dhq_calibrate.argtypes = [vp, vp, c_i64, vp]
    L.dhq_calibrate_layer.argtypes = [vp, c_i, vp, c_i64, vp]
    L.dhq_get_act_absmax.argtypes = [vp, c_i, ctypes.POINTER(ctypes.c_float), vp]
    L.dhq_set_act_absmax.argtypes = [vp, c_i, ctypes.c_float, vp]
    L.dhq_forward.argtypes = [vp, vp, c_i64, vp, vp]
    L.dhq_forward_host.argtypes = [vp, vp, c_i64, vp, vp]
    L.dhq_forward_static_scratch.argtypes = [vp, vp, c_i64, vp, vp]
    L.dhq_forward_static_scratch.restype = c_i
    L.dhq_forward_debug.argtypes = [vp, vp, c_i64, vp, ctypes.POINTER(_DebugBufs), vp]
    L.dhq_forward_fused_debug.argtypes = [vp, vp, c_i64, vp, ctypes.POINTER(_DebugBufs), vp]
    L.dhq_set_wait_limit.argtypes = [vp, c_i64]
    L.dhq_last_launch_clock.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    L.dhq_last_launch_clock.restype = c_i
    L.dhq_export.argtypes = [vp, vp, c_i64, ctypes.POINTER(c_i64)]
    L.dhq_import.argtypes = [ctypes.c_char_p, c_i64, vp, ctypes.POINTER(vp)]
    L.dhq_debug_stall_next_forward.argtypes = [vp]
    L.dhq_measure_sine_error.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_longlong, c_i, vp, ctypes.POINTER(ctypes.c_double)]
    L.dhq_get_layer.argtypes = [vp, c_i, vp, vp, vp]
    L.dhq_layer_dims.argtypes = [vp, c_i, ctypes.POINTER(c_i), ctypes.POINTER(c_i)]
    L.dhq_last_status.argtypes = [vp]
    L.dhq_launch_count.argtypes = [vp]
    L.dhq_launch_count.restype = c_i64
    L.dhq_destroy.argtypes = [vp]
    L.dhq_destroy.restype = None
    L.dhq_status_string.argtypes = [c_i]
    L.dhq_status_string.restype = ctypes.c_char_p
    L.dhq_measure_pipe.argtypes = [c_i, c_i, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    for name in ("dhq_calibrate_layer", "dhq_get_act_absmax", "dhq_set_act_absmax", "dhq_forward_fused_debug",
                 "dhq_set_wait_limit", "dhq_debug_stall_next_forward", "dhq_measure_sine_error", "dhq_export", "dhq_import"):
        getattr(L, name).restype = c_i
    for name in ("dhq_prepare", "dhq_calibrate", "dhq_forward", "dhq_forward_host", "dhq_forward_debug",
                 "dhq_get_layer", "dhq_layer_dims", "dhq_last_status", "dhq_measure_pipe"):
        getattr(L, name).restype = c_i
    _lib = L
    return L


def dhq_status_string(code: int) -> str:
    return load_library().dhq_status_string(int(code)).decode()


def _stream_ptr(stream):
    if stream is None:
        if not torch.cuda.is_available():      # argument checks of the library can still be exercised
            return ctypes.c_void_p(None)
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(code, where):
    if code != 0:
        raise DhqError(code, where)


def _dev_ptr(t, dtype, what):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{what}: expected a contiguous CUDA tensor of dtype {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def dhq_prepare(dims, weights, biases, omega0=30.0, w_bits=8, a_bits=8, w_gran=DHQ_GRAN_TENSOR,
                a_gran=DHQ_GRAN_TENSOR, rotation=DHQ_ROT_INPUT, stream=None, activation=DHQ_ACT_SINE, act_s0=0.0):
    """dims: L+1 ints; weights[l]: CUDA fp32 [dims[l+1]][dims[l]]; biases[l]: CUDA fp32 [dims[l+1]].
    Returns the opaque handle (an integer address)."""
    L = len(dims) - 1
    dims_arr = (ctypes.c_int * (L + 1))(*[int(d) for d in dims])
    cfg = _Config(L, dims_arr, int(w_bits), int(a_bits), float(omega0), int(w_gran), int(a_gran), int(rotation),
                  int(activation), float(act_s0))
    W = (ctypes.c_void_p * L)(*[_dev_ptr(w, torch.float32, "weights") for w in weights])
    B = (ctypes.c_void_p * L)(*[_dev_ptr(b, torch.float32, "biases") for b in biases])
    out = ctypes.c_void_p()
    _check(load_library().dhq_prepare(ctypes.byref(cfg), W, B, _stream_ptr(stream), ctypes.byref(out)), "dhq_prepare")
    return out.value


def dhq_calibrate(handle, coords, stream=None):
    n = coords.shape[0]
    _check(load_library().dhq_calibrate(handle, _dev_ptr(coords, torch.float32, "coords"), n, _stream_ptr(stream)),
           "dhq_calibrate")


def dhq_calibrate_layer(handle, layer, coords, stream=None):
    """Measure layer `layer` (1-based) on this part of the calibration set; coords may be empty."""
    n = 0 if coords is None else coords.shape[0]
    ptr = _dev_ptr(coords, torch.float32, "coords") if n else None
    _check(load_library().dhq_calibrate_layer(handle, int(layer), ptr, n, _stream_ptr(stream)), "dhq_calibrate_layer")


def dhq_get_act_absmax(handle, layer, stream=None) -> float:
    a = ctypes.c_float()
    _check(load_library().dhq_get_act_absmax(handle, int(layer), ctypes.byref(a), _stream_ptr(stream)), "dhq_get_act_absmax")
    return float(a.value)


def dhq_set_act_absmax(handle, layer, absmax, stream=None):
    _check(load_library().dhq_set_act_absmax(handle, int(layer), ctypes.c_float(float(absmax)), _stream_ptr(stream)),
           "dhq_set_act_absmax")


def dhq_forward(handle, coords, out, stream=None):
    """coords: CUDA fp32 [n][2]; out: CUDA fp32 [n][d_L]."""
    n = coords.shape[0]
    _check(load_library().dhq_forward(handle, _dev_ptr(coords, torch.float32, "coords"), n,
                                      _dev_ptr(out, torch.float32, "out"), _stream_ptr(stream)), "dhq_forward")


def dhq_forward_static_scratch(handle, coords, out, stream=None):
    """The forward pass for callers that must not allocate device memory: same arguments as
    dhq_forward, at most DHQ_STATIC_MAX_TOKENS coordinates per call, scratch in a fixed array
    inside the library.  This wrapper allocates nothing either."""
    n = coords.shape[0]
    _check(load_library().dhq_forward_static_scratch(handle, _dev_ptr(coords, torch.float32, "coords"), n,
                                                     _dev_ptr(out, torch.float32, "out"), _stream_ptr(stream)),
           "dhq_forward_static_scratch")


def dhq_forward_host(handle, coords_host, out_host, stream=None):
    """coords_host / out_host: CPU fp32 tensors (pinned for asynchronous copies)."""
    for t in (coords_host, out_host):
        if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous():
            raise TypeError("dhq_forward_host: expected contiguous CPU fp32 tensors")
    n = coords_host.shape[0]
    _check(load_library().dhq_forward_host(handle, ctypes.c_void_p(coords_host.data_ptr()), n,
                                           ctypes.c_void_p(out_host.data_ptr()), _stream_ptr(stream)),
           "dhq_forward_host")


def dhq_layer_dims(handle, layer):
    K, M = ctypes.c_int(), ctypes.c_int()
    _check(load_library().dhq_layer_dims(handle, int(layer), ctypes.byref(K), ctypes.byref(M)), "dhq_layer_dims")
    return K.value, M.value


def dhq_forward_debug(handle, coords, out=None, bufs=None, stream=None, fused=False):
    """bufs: dict with any of 'X', 'codes', 's_x', 'acc', 'Y', each a list of L CUDA tensors or
    None entries (dtypes fp32, int8, fp32, int32, fp32).  fused=True calls dhq_forward_fused_debug:
    the same dumps written from inside the fused kernel."""
    n = coords.shape[0]
    dtypes = {"X": torch.float32, "codes": torch.int8, "s_x": torch.float32, "acc": torch.int32, "Y": torch.float32}
    st = _DebugBufs()
    keep = []
    if bufs:
        n_layers = 0
        while n_layers < 16 and load_library().dhq_layer_dims(handle, n_layers + 1, None, None) == 0:
            n_layers += 1
        for key, dt in dtypes.items():
            lst = bufs.get(key)
            if lst is None:
                continue
            if len(lst) != n_layers:       # the library indexes these arrays by layer: never pass a short one
                raise ValueError(f"dhq_forward_debug: bufs[{key!r}] needs {n_layers} entries (one per layer)")
            arr = (ctypes.c_void_p * len(lst))(*[_dev_ptr(t, dt, key) for t in lst])
            keep.append(arr)
            setattr(st, key, arr)
    fn = load_library().dhq_forward_fused_debug if fused else load_library().dhq_forward_debug
    _check(fn(handle, _dev_ptr(coords, torch.float32, "coords"), n, _dev_ptr(out, torch.float32, "out"),
              ctypes.byref(st) if bufs else None, _stream_ptr(stream)),
           "dhq_forward_fused_debug" if fused else "dhq_forward_debug")


def dhq_forward_fused_debug(handle, coords, out, bufs=None, stream=None):
    dhq_forward_debug(handle, coords, out, bufs, stream, fused=True)


def dhq_set_wait_limit(handle, nanoseconds: int):
    _check(load_library().dhq_set_wait_limit(handle, int(nanoseconds)), "dhq_set_wait_limit")


def dhq_debug_stall_next_forward(handle):
    _check(load_library().dhq_debug_stall_next_forward(handle), "dhq_debug_stall_next_forward")


def dhq_measure_sine_error(lo, hi, count=1 << 22, mode=0, stream=None) -> float:
    """Largest |f(x) - sin(x)| over `count` fp32 arguments in [lo, hi] (see dhq_peaks.h)."""
    err = ctypes.c_double()
    rc = load_library().dhq_measure_sine_error(float(lo), float(hi), int(count), int(mode), _stream_ptr(stream), ctypes.byref(err))
    if rc != 0:
        raise RuntimeError(f"dhq_measure_sine_error failed with {rc}")
    return err.value


def dhq_get_layer(handle, layer):
    """Returns (codes int8 [M][K], w_scales fp32 [M], act_absmax float) as numpy values."""
    K, M = dhq_layer_dims(handle, layer)
    codes = np.empty((M, K), dtype=np.int8)
    scales = np.empty(M, dtype=np.float32)
    a = ctypes.c_float()
    _check(load_library().dhq_get_layer(handle, int(layer), codes.ctypes.data_as(ctypes.c_void_p),
                                        scales.ctypes.data_as(ctypes.c_void_p), ctypes.byref(a)), "dhq_get_layer")
    return codes, scales, float(a.value)


def dhq_export(handle) -> bytes:
    """The prepared handle as a block of bytes (see dhq.h)."""
    L = load_library()
    need = ctypes.c_int64()
    _check(L.dhq_export(handle, None, 0, ctypes.byref(need)), "dhq_export")
    buf = ctypes.create_string_buffer(need.value)
    _check(L.dhq_export(handle, buf, need.value, ctypes.byref(need)), "dhq_export")
    return buf.raw


def dhq_import(blob: bytes, stream=None):
    """A new handle on the current device from an exported block."""
    out = ctypes.c_void_p()
    _check(load_library().dhq_import(blob, len(blob), _stream_ptr(stream), ctypes.byref(out)), "dhq_import")
    return out.value


def dhq_last_status(handle) -> int:
    return int(load_library().dhq_last_status(handle))


def dhq_last_launch_clock(handle):
    """(SM MHz, milliseconds) of the handle's last fused-kernel launch, measured inside the kernel."""
    mhz, ms = ctypes.c_double(), ctypes.c_double()
    _check(load_library().dhq_last_launch_clock(handle, ctypes.byref(mhz), ctypes.byref(ms)), "dhq_last_launch_clock")
    return mhz.value, ms.value


def dhq_launch_count(handle) -> int:
    return int(load_library().dhq_launch_count(handle))


def dhq_destroy(handle):
    load_library().dhq_destroy(handle)


def dhq_measure_pipe(pipe, iters=2000, stream=None):
    """Returns (ops_per_second, milliseconds) of one pipe micro-benchmark (see dhq_peaks.h)."""
    code = PIPES[pipe] if isinstance(pipe, str) else int(pipe)
    ops, ms = ctypes.c_double(), ctypes.c_double()
    rc = load_library().dhq_measure_pipe(code, int(iters), _stream_ptr(stream), ctypes.byref(ops), ctypes.byref(ms))
    if rc != 0:
        raise RuntimeError(f"dhq_measure_pipe({pipe}) failed with {rc}")
    return ops.value, ms.value

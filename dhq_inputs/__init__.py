"""Seeded synthetic inputs for the DHQ forward path: SIREN-initialised layers and pixel grids.

This module only produces data (weights, biases, coordinate grids, the list of named
workloads).  It holds none of the method's arithmetic: no Hadamard transform, no quantizer, no
matmul.  Both the CPU oracle's tests and the CUDA library's tests/bench draw their inputs here,
so that the two implementations see bit-identical fp32 arrays.

Random numbers come from a counter-based splitmix64 stream written out below, so the arrays do
not depend on the numpy or torch version.  The networks stand in for the trained SIREN models of
the paper's experiments (Section IV), which need image datasets that are not available; the
shapes follow that workload: a 2-D pixel grid in, grey or RGB out.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def splitmix64(seed: int, start: int, count: int) -> np.ndarray:
    """Outputs `start .. start+count-1` of the splitmix64 stream with the given seed (uint64)."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


class Stream:
    """Sequential reader over one splitmix64 stream; `uniform` gives doubles in [0, 1)."""

    def __init__(self, seed: int):
        self.seed = int(seed)
        self.pos = 0

    def uniform(self, count: int) -> np.ndarray:
        r = splitmix64(self.seed, self.pos, count)
        self.pos += count
        return (r >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)

    def uniform_sym(self, count: int, bound: float) -> np.ndarray:
        """Doubles uniform in [-bound, bound)."""
        return (2.0 * self.uniform(count) - 1.0) * bound


def siren_init(dims, omega0: float, seed: int):
    """SIREN initialisation (Sitzmann et al. 2020) for an MLP with layer sizes `dims`.

    Layer 1 weights are U(-1/d_in, 1/d_in) (for d_in = 2 this is the +-0.5 range the paper
    reports for its first layer, Section III-A); later layers U(+-sqrt(6/d_in)/omega0); biases
    U(+-1/sqrt(d_in)).  Values are drawn layer by layer, weights (row-major [d_out][d_in]) then
    bias, in fp64 and rounded to fp32.  Returns (weights, biases) as lists of fp32 arrays.
    """
    st = Stream(seed)
    weights, biases = [], []
    for l in range(len(dims) - 1):
        d_in, d_out = int(dims[l]), int(dims[l + 1])
        wb = 1.0 / d_in if l == 0 else math.sqrt(6.0 / d_in) / omega0
        w = st.uniform_sym(d_out * d_in, wb).reshape(d_out, d_in)
        b = st.uniform_sym(d_out, 1.0 / math.sqrt(d_in))
        weights.append(np.ascontiguousarray(w.astype(np.float32)))
        biases.append(np.ascontiguousarray(b.astype(np.float32)))
    return weights, biases


def trained_like_init(dims, omega0: float, seed: int):
    """Stress set: hidden weights bell-shaped in about +-0.04 and a two-peaked last layer,

    mimicking the distributions the paper describes for a trained SIREN (Section III-A).  The
    first layer and the biases stay as in `siren_init`.
    """
    weights, biases = siren_init(dims, omega0, seed)
    st = Stream(seed + 0x5151)
    nl = len(dims) - 1
    for l in range(1, nl):
        d_in, d_out = int(dims[l]), int(dims[l + 1])
        cnt = d_out * d_in
        # sum of 12 uniforms - 6: a bell curve without calling any library sampler
        g = st.uniform(12 * cnt).reshape(cnt, 12).sum(axis=1) - 6.0
        if l < nl - 1:
            w = np.clip(0.013 * g, -0.04, 0.04)
        else:
            side = np.where(st.uniform(cnt) < 0.5, -1.0, 1.0)
            w = side * 0.03 + 0.008 * g
        weights[l] = np.ascontiguousarray(w.reshape(d_out, d_in).astype(np.float32))
    return weights, biases


def grid_coords(height: int, width: int) -> np.ndarray:
    """Endpoint-inclusive pixel grid on [-1, 1]^2, fp32 array [height*width][2].

    g_i = -1 + 2 i / (N - 1) computed in fp64 and rounded; token t = i*width + j holds
    (g_i over the height axis, g_j over the width axis).
    """
    def axis(n):
        if n == 1:
            return np.zeros(1, dtype=np.float64)
        return -1.0 + 2.0 * np.arange(n, dtype=np.float64) / (n - 1)

    gy, gx = axis(height), axis(width)
    out = np.empty((height, width, 2), dtype=np.float32)
    out[:, :, 0] = gy[:, None].astype(np.float32)
    out[:, :, 1] = gx[None, :].astype(np.float32)
    return np.ascontiguousarray(out.reshape(height * width, 2))


def procedural_image(height: int, width: int, channels: int, seed: int) -> np.ndarray:
    """Seeded synthetic target image, fp32 [height][width][channels] in [0, 1], standing in for the
    photographs of the paper's quality experiments (Section IV: cameraman, Kodak, CT), which are not
    available: a smooth background gradient, soft blobs, a few hard-edged discs and boxes (object
    outlines), and a patch of fine oriented texture whose frequency sweeps (detail that a
    sinusoidal network has to work for)."""
    st = Stream(seed + 0x1A6E)
    yy, xx = np.meshgrid(np.linspace(-1, 1, height), np.linspace(-1, 1, width), indexing="ij")
    img = np.zeros((height, width, channels), dtype=np.float64)
    for c in range(channels):
        g = st.uniform_sym(2, 0.15)
        plane = 0.45 + g[0] * yy + g[1] * xx
        for _ in range(6):                                   # soft blobs
            cy, cx, r, a = st.uniform_sym(1, 0.8)[0], st.uniform_sym(1, 0.8)[0], 0.1 + 0.3 * st.uniform(1)[0], st.uniform_sym(1, 0.25)[0]
            plane += a * np.exp(-((yy - cy) ** 2 + (xx - cx) ** 2) / (2 * r * r))
        for _ in range(4):                                   # hard-edged discs
            cy, cx, r, a = st.uniform_sym(1, 0.7)[0], st.uniform_sym(1, 0.7)[0], 0.05 + 0.2 * st.uniform(1)[0], st.uniform_sym(1, 0.3)[0]
            plane += a * (((yy - cy) ** 2 + (xx - cx) ** 2) < r * r)
        for _ in range(3):                                   # boxes
            cy, cx, hh, ww, a = (st.uniform_sym(1, 0.7)[0], st.uniform_sym(1, 0.7)[0], 0.05 + 0.25 * st.uniform(1)[0],
                                 0.05 + 0.25 * st.uniform(1)[0], st.uniform_sym(1, 0.25)[0])
            plane += a * ((np.abs(yy - cy) < hh) & (np.abs(xx - cx) < ww))
        ang, f0, f1, amp = st.uniform(1)[0] * np.pi, 6 + 10 * st.uniform(1)[0], 10 + 20 * st.uniform(1)[0], 0.08 + 0.08 * st.uniform(1)[0]
        u = np.cos(ang) * xx + np.sin(ang) * yy
        window = np.exp(-((yy - 0.35) ** 2 + (xx + 0.3) ** 2) / (2 * 0.35 ** 2))
        plane += amp * window * np.sin(np.pi * (f0 * u + 0.5 * (f1 - f0) * u * u))
        img[:, :, c] = plane
    return np.clip(img, 0.0, 1.0).astype(np.float32)


def sweep_grid(k: int) -> np.ndarray:
    """Grid with 2**k points, 2**ceil(k/2) rows by 2**floor(k/2) columns (batch-size sweep)."""
    return grid_coords(1 << ((k + 1) // 2), 1 << (k // 2))


@dataclass(frozen=True)
class Workload:
    """One named network + grid.  `w_gran` / `a_gran`: 0 = per tensor, 1 = per output channel
    (weights) / per token (activations)."""
    name: str
    dims: tuple
    omega0: float
    seed: int
    w_bits: int
    a_bits: int
    w_gran: int
    a_gran: int
    grid: tuple
    note: str = ""

    @property
    def n(self) -> int:
        return self.grid[0] * self.grid[1]

    def network(self):
        return siren_init(self.dims, self.omega0, self.seed)

    def coords(self) -> np.ndarray:
        return grid_coords(*self.grid)


def _mlp(width, hidden, d_out):
    return tuple([2] + [width] * hidden + [d_out])


WORKLOADS = {
    "C1": Workload("C1", _mlp(64, 3, 1), 30.0, 0, 8, 8, 0, 0, (64, 64), "grey, 4,096 points"),
    "C2": Workload("C2", _mlp(256, 3, 3), 30.0, 1, 8, 8, 0, 0, (256, 256), "RGB, 65,536 points"),
    "C3": Workload("C3", _mlp(256, 5, 3), 30.0, 2, 8, 8, 1, 1, (512, 512),
                   "per-channel W, per-token A"),
    "C4-W4A4": Workload("C4-W4A4", _mlp(256, 5, 3), 30.0, 3, 4, 4, 1, 1, (1024, 1024), "4-bit codes"),
    "C4-W6A6": Workload("C4-W6A6", _mlp(256, 5, 3), 30.0, 3, 6, 6, 1, 1, (1024, 1024), "6-bit codes"),
    "C5": Workload("C5", _mlp(512, 4, 3), 30.0, 4, 8, 8, 0, 0, (2048, 2048), "4,194,304 points"),
}

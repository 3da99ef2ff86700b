"""Reconstruction quality of the quantized forward pass: a harness around the library.

The paper's claim (Section IV, Table 1) is about image quality: at 8/8 bits the Hadamard
quantizer loses less PSNR/SSIM against the full-precision network than a plain uniform quantizer.
Its images (cameraman, Kodak, CT) and trained networks are not available, so this harness
 (1) draws a seeded procedural target image (dhq_inputs.procedural_image),
 (2) fits a small fp32 sinusoidal network to it with a short Adam run (PyTorch autograd; this is
     harness code: the library itself only does inference), and
 (3) evaluates the fitted weights through the library's C ABI in every datapath: W32A32, W8A32,
     DHQ (input-side rotation), the two-sided transform, and the same quantizer without rotation
     ("Uniform"), at 8/8, 6/6 and 4/4 bits, per-tensor and per-channel/per-token scales,
and prints one JSON record with PSNR (dB) and SSIM of each against the target and against the
fp32 network's own output.

    python -m paper_2508_13478_b200.quality --size 256 --width 256 --hidden 3 --steps 3000
"""
from __future__ import annotations

import argparse
import json
import math
import sys

import numpy as np


def psnr(a: np.ndarray, b: np.ndarray, peak: float = 1.0) -> float:
    """10 log10(peak^2 / MSE) over all pixels and channels."""
    mse = float(np.mean((a.astype(np.float64) - b.astype(np.float64)) ** 2))
    return float("inf") if mse == 0 else 10.0 * math.log10(peak * peak / mse)


def _gauss_filter(img: np.ndarray, sigma: float = 1.5, radius: int = 5) -> np.ndarray:
    """Separable Gaussian window (11 taps), 'valid' region only, applied to [H][W]."""
    k = np.exp(-0.5 * (np.arange(-radius, radius + 1) / sigma) ** 2)
    k /= k.sum()
    tmp = np.apply_along_axis(lambda v: np.convolve(v, k, mode="valid"), 0, img)
    return np.apply_along_axis(lambda v: np.convolve(v, k, mode="valid"), 1, tmp)


def ssim(a: np.ndarray, b: np.ndarray, peak: float = 1.0) -> float:
    """Structural similarity index (Wang et al. 2004): 11x11 Gaussian window, sigma 1.5,
    K1 = 0.01, K2 = 0.03, mean over the valid region and the channels."""
    a = a.astype(np.float64).reshape(a.shape[0], a.shape[1], -1)
    b = b.astype(np.float64).reshape(b.shape[0], b.shape[1], -1)
    c1, c2 = (0.01 * peak) ** 2, (0.03 * peak) ** 2
    vals = []
    for ch in range(a.shape[2]):
        x, y = a[:, :, ch], b[:, :, ch]
        mx, my = _gauss_filter(x), _gauss_filter(y)
        sxx = _gauss_filter(x * x) - mx * mx
        syy = _gauss_filter(y * y) - my * my
        sxy = _gauss_filter(x * y) - mx * my
        vals.append(np.mean(((2 * mx * my + c1) * (2 * sxy + c2)) / ((mx * mx + my * my + c1) * (sxx + syy + c2))))
    return float(np.mean(vals))


def fit_network(dims, omega0, target, coords, steps, lr, seed, gabor_s0=0.0, log=None):
    """Short fp32 fit of sin(omega0 (W x + b)) layers (or the Gabor wavelet) to `target` [n][d_L] in
    [-1, 1] by Adam on the mean squared error, from the seeded SIREN initialisation.  Returns the
    fitted (weights, biases) as fp32 numpy arrays and the network's own fp32 output."""
    import torch
    import dhq_inputs
    w0, b0 = dhq_inputs.siren_init(dims, omega0, seed)
    W = [torch.tensor(w, device="cuda", requires_grad=True) for w in w0]
    B = [torch.tensor(b, device="cuda", requires_grad=True) for b in b0]
    x0 = torch.from_numpy(coords).cuda()
    t = torch.from_numpy(target).cuda()
    opt = torch.optim.Adam(W + B, lr=lr)
    torch.backends.cuda.matmul.allow_tf32 = False

    def forward():
        x = x0
        for l in range(len(W)):
            z = x @ W[l].T + B[l]
            if l < len(W) - 1:
                x = torch.sin(omega0 * z)
                if gabor_s0 > 0:
                    x = x * torch.exp(-(gabor_s0 * z) ** 2)
            else:
                x = z
        return x

    for step in range(steps):
        opt.zero_grad(set_to_none=True)
        loss = torch.mean((forward() - t) ** 2)
        loss.backward()
        opt.step()
        if log and (step % max(1, steps // 10) == 0 or step == steps - 1):
            log(f"step {step}: mse {loss.item():.3e}")
    with torch.no_grad():
        out = forward().cpu().numpy()
    return [w.detach().cpu().numpy() for w in W], [b.detach().cpu().numpy() for b in B], out


def to_image(out, shape):
    """Network output in [-1, 1] -> image in [0, 1]."""
    return np.clip(out.reshape(shape).astype(np.float64) * 0.5 + 0.5, 0.0, 1.0)


def evaluate(dims, omega0, weights, biases, coords, variants, gabor_s0=0.0):
    """Runs every variant through the library.  variants: list of dicts with keys name, w_bits,
    a_bits, gran (0 per tensor / 1 per channel and token), rotation.  Returns {name: output}."""
    import torch
    from . import binding as dhq
    cd = torch.from_numpy(coords).cuda()
    W = [torch.from_numpy(np.ascontiguousarray(w)).cuda() for w in weights]
    B = [torch.from_numpy(np.ascontiguousarray(b)).cuda() for b in biases]
    outs = {}
    for v in variants:
        if gabor_s0 > 0 and v["a_bits"] == dhq.DHQ_BITS_FLOAT:
            continue                                    # the floating-point datapaths are sine-only
        h = dhq.dhq_prepare(dims, W, B, omega0, v["w_bits"], v["a_bits"], v["gran"], v["gran"], rotation=v["rotation"],
                            activation=dhq.DHQ_ACT_GABOR if gabor_s0 > 0 else dhq.DHQ_ACT_SINE, act_s0=gabor_s0)
        try:
            out = torch.empty((coords.shape[0], dims[-1]), device="cuda")
            dhq.dhq_forward(h, cd, out)                 # per-tensor scales calibrate on this grid
            torch.cuda.synchronize()
            if dhq.dhq_last_status(h) != 0:
                raise RuntimeError("device-side wait timed out")
            outs[v["name"]] = out.cpu().numpy()
        finally:
            dhq.dhq_destroy(h)
    return outs


def default_variants():
    from . import binding as dhq
    F = dhq.DHQ_BITS_FLOAT
    v = [{"name": "W32A32", "w_bits": F, "a_bits": F, "gran": 0, "rotation": dhq.DHQ_ROT_NONE},
         {"name": "W8A32 DHQ weights", "w_bits": 8, "a_bits": F, "gran": 0, "rotation": dhq.DHQ_ROT_INPUT},
         {"name": "W8A32 uniform weights", "w_bits": 8, "a_bits": F, "gran": 0, "rotation": dhq.DHQ_ROT_NONE}]
    for bits in (8, 6, 4):
        for gran, gname in ((0, "per tensor"), (1, "per channel/token")):
            v.append({"name": f"DHQ {bits}/{bits} {gname}", "w_bits": bits, "a_bits": bits, "gran": gran, "rotation": dhq.DHQ_ROT_INPUT})
            v.append({"name": f"DHQ two-sided {bits}/{bits} {gname}", "w_bits": bits, "a_bits": bits, "gran": gran, "rotation": dhq.DHQ_ROT_BOTH})
            v.append({"name": f"Uniform {bits}/{bits} {gname}", "w_bits": bits, "a_bits": bits, "gran": gran, "rotation": dhq.DHQ_ROT_NONE})
    return v


def run(size=256, width=256, hidden=3, channels=1, steps=3000, lr=1e-4, omega0=30.0, seed=7, gabor_s0=0.0, log=None):
    import dhq_inputs
    dims = (2,) + (width,) * hidden + (channels,)
    image = dhq_inputs.procedural_image(size, size, channels, seed)
    coords = dhq_inputs.grid_coords(size, size)
    target = (image.reshape(-1, channels) * 2.0 - 1.0).astype(np.float32)
    weights, biases, fp32_out = fit_network(dims, omega0, target, coords, steps, lr, seed, gabor_s0, log)
    shape = (size, size, channels)
    ref = to_image(fp32_out, shape)
    record = {"target": f"procedural image {size}x{size}x{channels}, seed {seed}", "dims": list(dims), "omega0": omega0,
              "activation": "gabor" if gabor_s0 > 0 else "sine", "gabor_s0": gabor_s0, "fit": {"steps": steps, "lr": lr},
              "fp32_torch": {"psnr": psnr(ref, image), "ssim": ssim(ref, image)}, "variants": {}}
    for name, out in evaluate(dims, omega0, weights, biases, coords, default_variants(), gabor_s0).items():
        img = to_image(out, shape)
        record["variants"][name] = {"psnr": psnr(img, image), "ssim": ssim(img, image),
                                    "psnr_vs_fp32": psnr(img, ref), "max_abs_vs_fp32": float(np.abs(out - fp32_out).max())}
    return record


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--size", type=int, default=256)
    ap.add_argument("--width", type=int, default=256)
    ap.add_argument("--hidden", type=int, default=3)
    ap.add_argument("--channels", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--lr", type=float, default=1e-4)
    ap.add_argument("--omega0", type=float, default=30.0)
    ap.add_argument("--seed", type=int, default=7)
    ap.add_argument("--gabor-s0", type=float, default=0.0, help="> 0: the wavelet activation (WIRE reading) instead of the sine")
    args = ap.parse_args()
    rec = run(args.size, args.width, args.hidden, args.channels, args.steps, args.lr, args.omega0, args.seed, args.gabor_s0,
              log=lambda m: print(m, file=sys.stderr))
    print(json.dumps(rec))


if __name__ == "__main__":
    main()

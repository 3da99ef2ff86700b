"""Helpers for the GPU parity tests: run the library, feed its per-layer inputs to the oracle
(layer-local teacher forcing) and compare stage by stage."""
import numpy as np
import torch

import paper_2508_13478_b200 as dhq
from oracle import dhq_oracle as orc

TOL_Y = 1e-5   # absolute tolerance on fp32 layer outputs against the fp64 epilogue


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def prepare_pair(dims, weights, biases, omega0, w_bits, a_bits, w_gran, a_gran, rotate=True, gabor_s0=0.0):
    h = dhq.dhq_prepare(dims, [to_dev(w) for w in weights], [to_dev(b) for b in biases], omega0,
                        w_bits, a_bits, w_gran, a_gran, rotation=1 if rotate == "both" else 0 if rotate else 2,
                        activation=dhq.DHQ_ACT_GABOR if gabor_s0 > 0 else dhq.DHQ_ACT_SINE, act_s0=gabor_s0)
    net = orc.prepare(weights, biases, dims, omega0, w_bits, a_bits, w_gran, a_gran, rotate=rotate, gabor_s0=gabor_s0)
    return h, net


def check_weights(h, net):
    for l, lay in enumerate(net.layers, start=1):
        codes, scales, _ = dhq.dhq_get_layer(h, l)
        assert codes.shape == lay.qw.shape
        assert np.array_equal(codes.astype(np.int32), lay.qw), f"weight codes of layer {l}"
        assert np.array_equal(scales.view(np.uint32), lay.s_w.view(np.uint32)), f"weight scales of layer {l}"


def run_debug(h, net, coords_dev, fused=False):
    """Per-layer dumps of the layer-by-layer path, or (fused=True) written by the fused tensor-core
    kernel itself from where each value is produced."""
    n = coords_dev.shape[0]
    L = len(net.layers)
    bufs = {"X": [], "codes": [], "s_x": [], "acc": [], "Y": []}
    for lay in net.layers:
        bufs["X"].append(torch.empty((n, lay.K_pad), dtype=torch.float32, device="cuda"))
        bufs["codes"].append(torch.empty((n, lay.K_pad), dtype=torch.int8, device="cuda"))
        bufs["s_x"].append(torch.empty((n,), dtype=torch.float32, device="cuda"))
        bufs["acc"].append(torch.empty((n, lay.M_pad), dtype=torch.int32, device="cuda"))
        bufs["Y"].append(torch.empty((n, lay.M_pad), dtype=torch.float32, device="cuda"))
    out = torch.empty((n, net.dims[-1]), dtype=torch.float32, device="cuda")
    dhq.dhq_forward_debug(h, coords_dev, out, bufs, fused=fused)
    torch.cuda.synchronize()
    assert dhq.dhq_last_status(h) == 0
    return out, bufs


def check_layers_against_oracle(h, net, coords_np, out_dev, bufs, calib_is_this_set=True):
    """Layer-local teacher forcing: the oracle gets the library's fp32 input of each layer and
    must reproduce codes, scales and accumulators exactly and the fp32 output within TOL_Y."""
    L = len(net.layers)
    n = coords_np.shape[0]
    X1 = bufs["X"][0].cpu().numpy()
    assert np.array_equal(X1.view(np.uint32), orc.pad_coords(coords_np).view(np.uint32))
    worst = 0.0
    for l in range(1, L + 1):
        X = bufs["X"][l - 1].cpu().numpy()
        if net.a_gran == 0:
            _, _, a_gpu = dhq.dhq_get_layer(h, l)
            if calib_is_this_set:
                a_orc = float(orc.rotated_absmax(net, l, X).max())
                assert np.float32(a_gpu) == np.float32(a_orc), f"frozen absmax of layer {l}"
            net.layers[l - 1].a_frozen = a_gpu
        r = orc.layer(net, l, X, want=("codes", "s_x", "acc", "Y"))
        codes = bufs["codes"][l - 1].cpu().numpy().astype(np.int32)
        assert np.array_equal(codes, r["codes"]), f"activation codes of layer {l}"
        s_x = bufs["s_x"][l - 1].cpu().numpy()
        assert np.array_equal(s_x.view(np.uint32), r["s_x"].view(np.uint32)), f"activation scales of layer {l}"
        acc = bufs["acc"][l - 1].cpu().numpy().astype(np.int64)
        assert np.array_equal(acc, r["acc"]), f"accumulators of layer {l}"
        Y = bufs["Y"][l - 1].cpu().numpy()
        err = np.abs(Y.astype(np.float64) - r["Y"]).max() if n else 0.0
        worst = max(worst, float(err))
        assert err <= TOL_Y, f"layer {l} output off by {err}"
        if l < L:
            Xn = bufs["X"][l].cpu().numpy()
            assert np.array_equal(Xn.view(np.uint32), Y.view(np.uint32)), "dump chain does not close"
    out = out_dev.cpu().numpy()
    assert np.array_equal(out.view(np.uint32), Y[:, : net.dims[-1]].view(np.uint32))
    return worst

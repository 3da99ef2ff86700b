"""The comparison datapaths W8A32 (weights quantized as for DHQ, activations fp32) and W32A32
(plain fp32 network) through the C ABI against their fp64 definitions.

Layer-local: the definition is fed the library's own fp32 input of each layer, so the difference
is one layer's fp32 arithmetic: K products summed in fp32 (error about sqrt(K) 2^-24 sum|w x|,
i.e. about 1e-6 at K = 512), the fp32 rotation (W8A32), and the fp32 phase omega0 z (30 rad x 2^-23
= 3.6e-6).  Gate 2e-5 per layer (measured worst case 5.6e-6, printed by the tests).
"""
import numpy as np
import pytest
import torch

import dhq_inputs
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu

dhq = pytest.importorskip("paper_2508_13478_b200")
from oracle import dhq_oracle as orc  # noqa: E402
from oracle import odef  # noqa: E402

TOL_FLOAT = 2e-5


def _run(w, coords, w_bits, rotation):
    weights, biases = w.network()
    L = len(w.dims) - 1
    h = dhq.dhq_prepare(w.dims, [to_dev(x) for x in weights], [to_dev(x) for x in biases], w.omega0,
                        w_bits, dhq.DHQ_BITS_FLOAT, w.w_gran, w.a_gran, rotation=rotation)
    try:
        cd = to_dev(coords)
        n = coords.shape[0]
        X = [torch.empty((n, dhq.dhq_layer_dims(h, l)[0]), device="cuda") for l in range(1, L + 1)]
        Y = [torch.empty((n, dhq.dhq_layer_dims(h, l)[1]), device="cuda") for l in range(1, L + 1)]
        out_dbg = torch.empty((n, w.dims[-1]), device="cuda")
        dhq.dhq_forward_debug(h, cd, out_dbg, {"X": X, "Y": Y})
        out = torch.full_like(out_dbg, float("nan"))
        dhq.dhq_forward(h, cd, out)
        oh = torch.zeros((n, w.dims[-1])).pin_memory()
        dhq.dhq_forward_host(h, torch.from_numpy(coords).pin_memory(), oh)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int32), out_dbg.view(torch.int32))
        assert torch.equal(oh.view(torch.int32), out.cpu().view(torch.int32))
        codes = [dhq.dhq_get_layer(h, l) for l in range(1, L + 1)]
        return [x.cpu().numpy() for x in X], [y.cpu().numpy() for y in Y], out.cpu().numpy(), codes
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("name,count,rotate", [("C1", 4096, True), ("C2", 6000, True), ("C3", 5000, True), ("C2", 4000, False),
                                               ("C5", 3000, True), ("C4-W4A4", 3000, True)])
def test_w8a32_matches_its_definition_layer_by_layer(name, count, rotate):
    w = dhq_inputs.WORKLOADS[name]
    coords = w.coords()
    coords = np.ascontiguousarray(coords[np.linspace(0, coords.shape[0] - 1, count).astype(np.int64)])
    X, Y, out, codes = _run(w, coords, w.w_bits, 0 if rotate else 2)
    weights, biases = w.network()
    net = orc.prepare(weights, biases, w.dims, w.omega0, w.w_bits, 8, w.w_gran, 1, rotate=rotate)
    worst = 0.0
    for l, lay in enumerate(net.layers, start=1):
        assert np.array_equal(codes[l - 1][0].astype(np.int32), lay.qw)               # the same weight codes as DHQ
        assert np.array_equal(codes[l - 1][1].view(np.uint32), lay.s_w.view(np.uint32))
        want = odef.w8a32_layer(lay.qw, lay.s_w, lay.b_pad, X[l - 1], rotate, w.omega0, lay.sine)
        worst = max(worst, float(np.abs(Y[l - 1] - want).max()))
        if l < len(net.layers):
            assert np.array_equal(X[l].view(np.uint32), Y[l - 1].view(np.uint32))     # the chain closes
    assert np.array_equal(X[0].view(np.uint32), orc.pad_coords(coords).view(np.uint32))
    free = np.abs(out - orc.forward_w8a32(net, coords)).max()
    print(f"W{w.w_bits}A32 {name} rotate={rotate}: layer-local max |d| = {worst:.2e}, free-running = {free:.2e}")
    assert worst <= TOL_FLOAT and free <= 10 * TOL_FLOAT


@pytest.mark.parametrize("name,count", [("C1", 4096), ("C2", 6000), ("C5", 3000)])
def test_w32a32_matches_the_fp64_network_layer_by_layer(name, count):
    w = dhq_inputs.WORKLOADS[name]
    coords = w.coords()
    coords = np.ascontiguousarray(coords[np.linspace(0, coords.shape[0] - 1, count).astype(np.int64)])
    X, Y, out, _ = _run(w, coords, dhq.DHQ_BITS_FLOAT, 0)
    weights, biases = w.network()
    L = len(weights)
    worst = 0.0
    for l in range(1, L + 1):
        x = X[l - 1].astype(np.float64)[:, : weights[l - 1].shape[1]]
        z = x @ weights[l - 1].astype(np.float64).T + biases[l - 1].astype(np.float64)
        want = np.sin(w.omega0 * z) if l < L else z
        worst = max(worst, float(np.abs(Y[l - 1][:, : want.shape[1]] - want).max()))
        assert not Y[l - 1][:, want.shape[1]:].any()                                   # padded outputs stay zero
    free = np.abs(out - odef.siren_forward(weights, biases, w.omega0, coords)).max()
    print(f"W32A32 {name}: layer-local max |d| = {worst:.2e}, free-running = {free:.2e}")
    assert worst <= TOL_FLOAT and free <= 10 * TOL_FLOAT


def test_float_datapaths_reject_what_they_do_not_offer():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    W, B = [to_dev(x) for x in weights], [to_dev(x) for x in biases]
    with pytest.raises(dhq.DhqError) as e:
        dhq.dhq_prepare(w.dims, W, B, w_bits=dhq.DHQ_BITS_FLOAT, a_bits=8)            # A8 with fp32 weights: no such datapath
    assert e.value.code == 2
    with pytest.raises(dhq.DhqError) as e:
        dhq.dhq_prepare(w.dims, W, B, w_bits=8, a_bits=dhq.DHQ_BITS_FLOAT, rotation=1)
    assert e.value.code == 2
    h = dhq.dhq_prepare(w.dims, W, B, w_bits=8, a_bits=dhq.DHQ_BITS_FLOAT)
    try:
        cd = to_dev(w.coords()[:64])
        out = torch.empty((64, 1), device="cuda")
        dhq.dhq_calibrate(h, cd)                                                       # no-op
        for fn in (dhq.dhq_forward_fused_debug, dhq.dhq_forward_static_scratch):
            with pytest.raises(dhq.DhqError) as e:
                fn(h, cd, out)
            assert e.value.code == 2
        blob = dhq.dhq_export(h)
        h2 = dhq.dhq_import(blob)
        out2 = torch.empty_like(out)
        dhq.dhq_forward(h, cd, out)
        dhq.dhq_forward(h2, cd, out2)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int32), out2.view(torch.int32))
        dhq.dhq_destroy(h2)
    finally:
        dhq.dhq_destroy(h)

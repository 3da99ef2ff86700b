"""Pins for the parts of the oracle that decide integers in fp32.

(1) The per-output-channel weight quantizer: a hand-derived fixture and properties that fail if a
row were quantized with the tensor's absmax.  (2) The fp32 oracle against the fp64, orthonormally
scaled statement of the same layer (Eq. 3-5, Section III-B): the codes may differ only by one step
and only where the value to be rounded lies within 1e-4 of a half-integer; the rate is reported.
(3) The O(n log n) variant of the oracle used for the second CPU baseline is bit-identical to the
definition.  No GPU.
"""
import numpy as np
import pytest

import dhq_inputs
from oracle import dhq_oracle as orc
from oracle import dhq_oracle_nlogn as orcn
from oracle import odef


# ---------------------------------------------------------------- per-output-channel weight scales

def _f5_net(golden, w_gran):
    g = golden("f5_per_channel_weights.txt")
    W1 = np.array([g[f"w{m}"] for m in range(4)], dtype=np.float32)
    weights = [W1, np.zeros((4, 4), np.float32)]
    biases = [np.zeros(4, np.float32), np.zeros(4, np.float32)]
    return g, orc.prepare(weights, biases, (2, 4, 4), 30.0, w_bits=int(g["bits"][0]), a_bits=4, w_gran=w_gran, a_gran=1)


def test_per_channel_weight_quantizer_fixture_f5(golden):
    g, net = _f5_net(golden, w_gran=1)
    lay = net.layers[0]
    for m in range(4):
        assert lay.Wrot[m].tolist() == g[f"folded{m}"]
        assert lay.qw[m].tolist() == g[f"channel_codes{m}"]
        want_s = np.float32(g["row_absmax"][m]) / np.float32(7) if g["row_absmax"][m] else np.float32(0)
        assert lay.s_w[m].view(np.uint32) == np.float32(want_s).view(np.uint32)
    g, net = _f5_net(golden, w_gran=0)
    lay = net.layers[0]
    for m in range(4):
        assert lay.qw[m].tolist() == g[f"tensor_codes{m}"]
        assert lay.s_w[m].view(np.uint32) == (np.float32(g["tensor_absmax"][0]) / np.float32(7)).view(np.uint32)


@pytest.mark.parametrize("name", ["C3", "C4-W4A4", "C4-W6A6"])
def test_per_channel_rows_use_their_own_absmax(name):
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    net = orc.prepare(weights, biases, w.dims, w.omega0, w.w_bits, w.a_bits, w_gran=1, a_gran=1)
    qmax = 2 ** (w.w_bits - 1) - 1
    for lay in net.layers:
        rowmax = np.abs(lay.Wrot).max(axis=1)
        live = rowmax > 0
        assert np.array_equal(np.abs(lay.qw).max(axis=1)[live], np.full(int(live.sum()), qmax))   # every live row reaches qmax
        assert not lay.qw[~live].any() and not lay.s_w[~live].any()
        want = (rowmax / np.float32(qmax)).astype(np.float32)
        assert np.array_equal(lay.s_w.view(np.uint32), want.view(np.uint32))
        # the rows' ranges really differ, so one tensor-wide scale would not pass the lines above
        if live.sum() > 4:
            assert rowmax[live].max() > 1.05 * rowmax[live].min()
        # dequantized rows stay within half a step of the rotated weights, row by row
        err = np.abs(lay.Wrot.astype(np.float64) - lay.s_w.astype(np.float64)[:, None] * lay.qw)
        assert np.all(err <= lay.s_w.astype(np.float64)[:, None] / 2 * (1 + 2.0 ** -20))


# ---------------------------------------------------------------- fp32 oracle vs the fp64 statement

def _compare_tiers(name, count, w_gran, a_gran):
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    coords = w.coords()
    idx = np.linspace(0, coords.shape[0] - 1, count).astype(np.int64)
    coords = np.ascontiguousarray(coords[idx])
    net = orc.prepare(weights, biases, w.dims, w.omega0, w.w_bits, w.a_bits, w_gran, a_gran)
    if a_gran == 0:
        orc.calibrate(net, coords)
    _, per = orc.forward(net, coords, return_layers=True)
    L = len(net.layers)
    flips_w = flips_x = total_w = total_x = 0
    worst_y = 0.0
    for l in range(1, L + 1):
        lay, r = net.layers[l - 1], per[l - 1]
        K, M = lay.K_pad, lay.M_pad
        Wp = np.zeros((M, K))
        Wp[: weights[l - 1].shape[0], : weights[l - 1].shape[1]] = weights[l - 1]
        d = odef.dhq_layer_def(Wp, lay.b_pad, r["X"], w.w_bits, w.a_bits, bool(w_gran), bool(a_gran), w.omega0, lay.sine)
        for mine, theirs, t in ((lay.qw, d["qw"], d["tw"]), (r["codes"], d["codes"], d["t"])):
            diff = mine.astype(np.int64) - theirs
            bad = diff != 0
            assert np.all(np.abs(diff[bad]) == 1), f"layer {l}: a code differs by more than one step"
            frac = np.abs(t[bad] - np.floor(t[bad]) - 0.5)
            assert np.all(frac < 1e-4), f"layer {l}: codes differ away from a rounding tie ({frac.max() if frac.size else 0})"
        flips_w += int((lay.qw != d["qw"]).sum()); total_w += lay.qw.size
        flips_x += int((r["codes"] != d["codes"]).sum()); total_x += r["codes"].size
        # where the whole token and all weights agree, the accumulators are equal and the outputs differ
        # only by the fp32 rounding of the scales (1.2e-7 of a phase of tens of radians)
        if not (lay.qw != d["qw"]).any():
            same = ~(r["codes"] != d["codes"]).any(axis=1)
            assert np.array_equal(r["acc"][same], d["acc"][same])
            if same.any():
                worst_y = max(worst_y, float(np.abs(r["Y"][same] - d["Y"][same]).max()))
        # orthonormal absmax = un-normalised absmax / sqrt(K)
        if a_gran == 1:
            assert np.allclose(d["a_x"] * np.sqrt(K), np.abs(r["Xrot"]).max(axis=1), rtol=1e-6, atol=1e-30)
    assert worst_y < 3e-5
    return flips_w / total_w, flips_x / total_x, worst_y


@pytest.mark.parametrize("name,count,w_gran,a_gran", [("C1", 4096, 0, 0), ("C2", 1500, 0, 0), ("C2", 1500, 1, 1),
                                                      ("C4-W4A4", 600, 1, 1)])
def test_fp32_oracle_codes_agree_with_the_fp64_orthonormal_statement(name, count, w_gran, a_gran):
    rate_w, rate_x, worst_y = _compare_tiers(name, count, w_gran, a_gran)
    print(f"{name} gran=({w_gran},{a_gran}): weight codes differing {rate_w:.2e}, activation codes differing "
          f"{rate_x:.2e} (all by one step at a rounding tie), outputs within {worst_y:.1e} where codes agree")
    assert rate_w < 1e-3 and rate_x < 1e-3


def test_a_planted_scale_mistake_is_caught_by_the_tier_comparison():
    # the comparison has teeth: an oracle whose per-token absmax skipped the last feature would
    # disagree far from any tie
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    net = orc.prepare(weights, biases, w.dims, w.omega0, a_gran=1)
    X = np.random.default_rng(0).uniform(-1, 1, (200, 64)).astype(np.float32)
    r = orc.layer(net, 2, X)
    Wp = weights[1].astype(np.float64)
    d = odef.dhq_layer_def(Wp, biases[1], X, 8, 8, False, True, w.omega0, True)
    assert (np.abs(r["codes"] - d["codes"]) <= 1).all()
    Xbad = orc.rotate(X)
    a_bad = np.abs(Xbad[:, :-1]).max(axis=1)                      # planted: one feature left out
    s_bad = [orc.scales(float(a), 8)[1] for a in a_bad]
    planted = np.stack([orc.quantize(Xbad[i], s_bad[i], 8) for i in range(X.shape[0])])
    assert (np.abs(planted - d["codes"]) > 1).any() or (planted != d["codes"]).mean() > 1e-2


# ---------------------------------------------------------------- O(n log n) variant

@pytest.mark.parametrize("name,l,n", [("C1", 2, 300), ("C2", 3, 200), ("C3", 4, 150), ("C5", 2, 60), ("C5", 5, 60), ("C2", 1, 500)])
def test_nlogn_variant_is_bit_identical_to_the_definition(name, l, n):
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    net = orc.prepare(weights, biases, w.dims, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    lay = net.layers[l - 1]
    rng = np.random.default_rng(l * 100 + n)
    X = orc.pad_coords(w.coords()[:n]) if l == 1 else rng.uniform(-1, 1, (n, lay.K_pad)).astype(np.float32)
    a = float(orc.rotated_absmax(net, l, X).max()) * 0.9          # frozen scale that some tokens exceed
    ref = orc.layer(net, l, X, a_frozen=a)
    got = orcn.layer(net, l, X, a_frozen=a)
    for key in ("Xrot", "s_x"):
        assert np.array_equal(ref[key].view(np.uint32), got[key].view(np.uint32)), key
    assert np.array_equal(ref["codes"], got["codes"]) and np.array_equal(ref["acc"], got["acc"])
    assert np.array_equal(ref["Y"].view(np.uint64), got["Y"].view(np.uint64))
    for rot in (False,):
        plain = orc.prepare(weights, biases, w.dims, w.omega0, w.w_bits, w.a_bits, w.w_gran, 1, rotate=rot)
        assert np.array_equal(orc.layer(plain, l, X)["Y"].view(np.uint64), orcn.layer(plain, l, X)["Y"].view(np.uint64))


def test_nlogn_forward_equals_definition_forward():
    w = dhq_inputs.WORKLOADS["C3"]
    weights, biases = w.network()
    net = orc.prepare(weights, biases, w.dims, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    coords = w.coords()[1000:1200]
    assert np.array_equal(orc.forward(net, coords).view(np.uint64), orcn.forward(net, coords).view(np.uint64))


# ---------------------------------------------------------------- absmax without a finite scale

def test_absmax_whose_reciprocal_scale_overflows_counts_as_zero():
    # Reading of the quantizer's degenerate end: qmax / a must be a finite fp32 number.  4-wide brute
    # force: below the threshold every code is zero and the layer returns its bias term; above it
    # the absmax element maps to +-qmax as usual.
    for bits in (4, 8):
        qmax = 2 ** (bits - 1) - 1
        fmax = float(np.finfo(np.float32).max)
        below = np.float32(qmax / fmax * 0.9)
        above = np.float32(qmax / fmax * 1.2)
        assert orc.scales(float(below), bits) == (0.0, 0.0)
        s, inv = orc.scales(float(above), bits)
        assert s > 0 and np.isfinite(inv) and inv == np.float32(qmax) / above
        v = np.array([above, -above / 2, 0.0, above / 4], np.float32)
        assert orc.quantize(v, inv, bits)[0] == qmax
    W2 = np.eye(4, dtype=np.float32)
    b2 = np.array([0.5, -0.25, 0.0, 1.0], np.float32)
    net = orc.prepare([np.zeros((4, 2), np.float32), W2], [np.zeros(4, np.float32), b2], (2, 4, 4), 30.0, a_gran=1, rotate=False)
    X = np.array([[1e-39, -1e-39, 0, 5e-40], [2e-38, 0, 0, 0], [1e-36, -5e-37, 0, 0]], np.float32)
    r = orc.layer(net, 2, X)
    assert not r["codes"][:2].any() and not r["s_x"][:2].any() and not r["acc"][:2].any()
    assert np.array_equal(r["Y"][:2], np.tile(b2.astype(np.float64), (2, 1)))
    assert r["codes"][2].tolist() == [127, -64, 0, 0] or r["codes"][2].tolist() == [127, -63, 0, 0]
    assert np.array_equal(orcn.layer(net, 2, X)["codes"], r["codes"])


# ---------------------------------------------------------------- comparison datapaths: W8A32, W32A32

def _w8a32_error(w_bits, rotate=True):
    dims = (2, 64, 64, 3)
    weights, biases = dhq_inputs.siren_init(dims, 30.0, 21)
    coords = dhq_inputs.grid_coords(12, 12)
    net = orc.prepare(weights, biases, dims, 30.0, w_bits=w_bits, a_bits=8, w_gran=1, a_gran=1, rotate=rotate)
    got = orc.forward_w8a32(net, coords)
    return np.abs(got - odef.siren_forward(weights, biases, 30.0, coords)).max(), got, net, coords


def test_weight_only_quantized_network_converges_to_the_unquantized_siren():
    # W8A32 (Section I, Fig. 1; Table 2's middle column): only the weights carry quantization error,
    # so the distance to the fp64 SIREN shrinks with the weight bit-width alone
    e8, g8, net8, coords = _w8a32_error(8)
    e12, _, _, _ = _w8a32_error(12)
    e16, g16, _, _ = _w8a32_error(16)
    assert e12 < e8 / 4 and e16 < e12 / 4 and e16 < 1e-4
    _, g16_plain, _, _ = _w8a32_error(16, rotate=False)
    assert np.abs(g16 - g16_plain).max() < 1e-3                 # the rotation changes nothing in the limit
    # and it is the a_bits -> infinity limit of the fully quantized network with the same weights
    net_a16 = orc.prepare(*dhq_inputs.siren_init((2, 64, 64, 3), 30.0, 21), (2, 64, 64, 3), 30.0, w_bits=8, a_bits=16, w_gran=1, a_gran=1)
    assert np.abs(orc.forward(net_a16, coords) - g8).max() < 2e-3
    net_a8 = orc.prepare(*dhq_inputs.siren_init((2, 64, 64, 3), 30.0, 21), (2, 64, 64, 3), 30.0, w_bits=8, a_bits=8, w_gran=1, a_gran=1)
    assert np.abs(orc.forward(net_a16, coords) - g8).max() < np.abs(orc.forward(net_a8, coords) - g8).max()


def test_w8a32_layer_by_hand():
    # 4-wide layer, rotation on: x = [1, 2, 3, 4] -> H_4 x = [10, -2, -4, 0]; q_w rows [1, 0, -1, 2] and
    # [3, 3, 3, 3] with scales 0.5 and 0.25, biases 0.125 and -1:
    #   z0 = 0.5 * (10 + 4 + 0) + 0.125 = 7.125 ;  z1 = 0.25 * 3 * (10 - 2 - 4 + 0) - 1 = 2.0
    qw = np.array([[1, 0, -1, 2], [3, 3, 3, 3]])
    z = odef.w8a32_layer(qw, [0.5, 0.25], [0.125, -1.0], np.array([[1.0, 2.0, 3.0, 4.0]]), True, 30.0, False)
    assert z.tolist() == [[7.125, 2.0]]
    y = odef.w8a32_layer(qw, [0.5, 0.25], [0.125, -1.0], np.array([[1.0, 2.0, 3.0, 4.0]]), False, 2.0, True)
    # without the rotation: z0 = 0.5 * (1 - 3 + 8) + 0.125 = 3.125, z1 = 0.25 * 30 - 1 = 6.5
    assert np.allclose(y, np.sin(2.0 * np.array([[3.125, 6.5]])), atol=1e-15)


# ---------------------------------------------------------------- wavelet activation (WIRE reading)

def test_gabor_activation_by_hand_and_its_limits():
    # psi(z) = sin(omega0 z) exp(-(s0 z)^2): z = 0.1, omega0 = 10, s0 = 5 -> sin(1) exp(-0.25)
    import math
    assert abs(float(odef.gabor(np.array([0.1]), 10.0, 5.0)[0]) - math.sin(1.0) * math.exp(-0.25)) < 1e-16
    z = np.linspace(-2, 2, 1001)
    assert np.abs(odef.gabor(z, 30.0, 10.0)).max() <= 1.0                       # bounded like the sine
    assert np.array_equal(odef.gabor(z, 30.0, 0.0), np.sin(30.0 * z))           # s0 = 0 is the sine
    # the layer routine applies it to z = s_w s_x acc + b of hidden layers only
    W2 = np.eye(4, dtype=np.float32) * 0.5
    b2 = np.array([0.05, -0.02, 0.0, 0.1], np.float32)
    for sine_layer in (True, False):
        dims = (2, 4, 4, 4) if sine_layer else (2, 4, 4)
        weights = [np.zeros((4, 2), np.float32), W2] + ([np.zeros((4, 4), np.float32)] if sine_layer else [])
        biases = [np.zeros(4, np.float32), b2] + ([np.zeros(4, np.float32)] if sine_layer else [])
        net = orc.prepare(weights, biases, dims, 30.0, a_gran=1, rotate=False, gabor_s0=7.0)
        X = np.array([[0.25, -0.5, 1.0, 0.125]], np.float32)
        r = orc.layer(net, 2, X)
        z = net.layers[1].s_w.astype(np.float64) * float(r["s_x"][0]) * r["acc"][0] + b2.astype(np.float64)
        want = odef.gabor(z, 30.0, 7.0) if sine_layer else z
        assert np.allclose(r["Y"][0], want, rtol=0, atol=1e-15)


def test_quantized_gabor_network_converges_to_the_unquantized_one():
    dims = (2, 64, 64, 3)
    weights, biases = dhq_inputs.siren_init(dims, 30.0, 33)
    coords = dhq_inputs.grid_coords(12, 12)
    want = odef.siren_forward(weights, biases, 30.0, coords, gabor_s0=6.0)
    errs = []
    for bits in (8, 12, 16):
        net = orc.prepare(weights, biases, dims, 30.0, w_bits=bits, a_bits=bits, w_gran=1, a_gran=1, gabor_s0=6.0)
        errs.append(np.abs(orc.forward(net, coords) - want).max())
    assert errs[1] < errs[0] / 4 and errs[2] < errs[1] / 4 and errs[2] < 2e-4
    assert np.abs(want - odef.siren_forward(weights, biases, 30.0, coords)).max() > 1e-2   # and it is not the sine network

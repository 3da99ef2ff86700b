"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the passage it pins.  None of these tests needs a GPU.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import dhq_inputs
from oracle import dhq_oracle as orc
from oracle import odef


SIZES = [1, 2, 4, 8, 16, 32, 64, 128, 256, 512]


# ---------------------------------------------------------------- Hadamard matrix (Eq. 3)

def closed_form(n):
    i = np.arange(n)
    pc = np.vectorize(lambda v: bin(v).count("1"))(i[:, None] & i[None, :])
    return np.where(pc % 2 == 0, 1, -1).astype(np.int64)


@pytest.mark.parametrize("n", SIZES)
def test_hadamard_recursion_equals_closed_form_and_is_orthogonal(n):
    H = orc.hadamard(n).astype(np.int64)
    assert np.array_equal(H, closed_form(n))            # Sylvester recursion <=> (-1)^popcount(i&j)
    assert np.array_equal(H @ H.T, n * np.eye(n, dtype=np.int64))   # H^T H = n I
    assert np.array_equal(H, H.T)
    assert np.array_equal(H, odef.hadamard(n).astype(np.int64))


def test_hadamard_h4_rows_as_printed_by_the_recursion():
    assert orc.hadamard(4).tolist() == [[1, 1, 1, 1], [1, -1, 1, -1], [1, 1, -1, -1], [1, -1, -1, 1]]


def test_hadamard_rejects_non_power_of_two():
    with pytest.raises(ValueError):
        orc.hadamard(12)


# ---------------------------------------------------------------- rotation (vector form below Eq. 3)

@pytest.mark.parametrize("n", SIZES[1:])
def test_rotation_exact_on_small_integers(n):
    # every partial sum is an integer below 2^24, so fp32 is exact whatever the rounding:
    # this pins indexing, signs and the natural (Sylvester) output order.
    rng = np.random.default_rng(n)
    V = rng.integers(-1000, 1001, size=(7, n))
    want = V @ closed_form(n).T
    got = orc.rotate(V.astype(np.float32))
    assert np.array_equal(got.astype(np.int64), want)
    # involution: H (H v) = n v
    again = orc.rotate(got)
    assert np.array_equal(again.astype(np.int64), n * V)


@pytest.mark.parametrize("n", [4, 64, 256, 512])
def test_rotation_close_to_fp64_product(n):
    rng = np.random.default_rng(100 + n)
    V = rng.uniform(-1, 1, size=(16, n)).astype(np.float32)
    want = V.astype(np.float64) @ odef.hadamard(n).T
    got = orc.rotate(V).astype(np.float64)
    bound = math.log2(n) * 2.0 ** -24 * np.abs(V).astype(np.float64).sum(axis=1, keepdims=True)
    assert np.all(np.abs(got - want) <= bound)


def test_rotation_fixture_f1(golden):
    g = golden("f1_rotation_quantizer.txt")
    assert orc.rotate(g["x"])[0].tolist() == g["rotated"]


def test_rotation_summation_order_fixture_f4(golden):
    g = golden("f4_pairwise_order.txt")
    assert orc.rotate(np.array(g["v"], dtype=np.float32))[0].tolist() == g["rotated"]


@pytest.mark.parametrize("n", [2, 4, 32, 64, 256, 512])
def test_butterfly_form_is_bit_identical_to_the_tree_definition(n):
    rng = np.random.default_rng(7 * n)
    V = (rng.standard_normal((9, n)) * np.exp(rng.uniform(-8, 8, size=(9, n)))).astype(np.float32)
    a, b = orc.rotate(V), orc.rotate_butterfly(V)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_rotation_preserves_energy():
    # "redistributes its values while preserving its total energy": |Hx|^2 = n |x|^2
    rng = np.random.default_rng(3)
    V = rng.uniform(-1, 1, size=(4, 256)).astype(np.float32)
    r = orc.rotate(V).astype(np.float64)
    assert np.allclose((r ** 2).sum(1), 256 * (V.astype(np.float64) ** 2).sum(1), rtol=1e-6)


# ---------------------------------------------------------------- weight fold (Eq. 4-5)

def test_two_sided_transform_preserves_frobenius_norm():
    rng = np.random.default_rng(5)
    W = rng.uniform(-0.5, 0.5, size=(64, 4))
    assert math.isclose(np.linalg.norm(odef.transform_2d(W)), np.linalg.norm(W), rel_tol=1e-12)


@pytest.mark.parametrize("shape", [(64, 2), (64, 64), (3, 256), (512, 512)])
def test_weight_fold_norm_and_compute_invariance(shape):
    d_out, d_in = shape
    rng = np.random.default_rng(d_out * 1000 + d_in)
    W = rng.uniform(-0.1, 0.1, size=shape).astype(np.float32)
    dims = (2, d_out, 1) if d_in == 2 else (2, d_in, d_out if d_out > 4 else d_out)
    l = 1 if d_in == 2 else 2
    # build a 2-layer net description whose layer l has this shape
    if d_in == 2:
        weights = [W, np.zeros((1, d_out), np.float32)]
        biases = [np.zeros(d_out, np.float32), np.zeros(1, np.float32)]
        dims = (2, d_out, 1)
    else:
        weights = [np.zeros((d_in, 2), np.float32), W]
        biases = [np.zeros(d_in, np.float32), np.zeros(d_out, np.float32)]
        dims = (2, d_in, d_out)
    if d_out > 4 and d_in != 2:
        # make it a hidden layer so that M is not padded to 4
        weights.append(np.zeros((1, d_out), np.float32))
        biases.append(np.zeros(1, np.float32))
        dims = (2, d_in, d_out, 1)
    net = orc.prepare(weights, biases, dims, 30.0)
    lay = net.layers[l - 1]
    K = lay.K_pad
    Wp = np.zeros((lay.M_pad, K))
    Wp[:d_out, :d_in] = W
    Wrot = lay.Wrot.astype(np.float64)
    # ||W H / sqrt(K)||_F = ||W||_F  (Wrot = W H / K, so multiply by sqrt(K))
    assert math.isclose(np.linalg.norm(Wrot) * math.sqrt(K), np.linalg.norm(Wp), rel_tol=1e-5)
    assert np.allclose(Wrot, odef.input_side_fold(Wp), atol=1e-7)
    # W x = (W H / K)(H x)
    x = rng.uniform(-1, 1, size=K)
    x[d_in:] = 0
    lhs = Wp @ x
    rhs = odef.input_side_fold(Wp) @ (odef.hadamard(K) @ x)
    assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-13)
    # zero padding adds nothing: padded rows stay zero
    assert not Wrot[d_out:].any()


def test_weight_fold_fixture_f3(golden):
    g = golden("f3_weight_fold.txt")
    folded = orc.rotate(g["row"])[0] * np.float32(0.25)
    assert folded.tolist() == g["folded"]
    xr = orc.rotate(g["x"])[0]
    assert float(np.dot(folded.astype(np.float64), xr.astype(np.float64))) == g["dot"][0]
    assert float(np.dot(g["row"], g["x"])) == g["dot"][0]


# ---------------------------------------------------------------- quantizer

@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
def test_quantizer_properties(bits):
    rng = np.random.default_rng(bits)
    v = (rng.standard_normal(4096) * 3).astype(np.float32)
    a = orc.absmax(v)
    assert a == np.abs(v).max()
    s, inv = orc.scales(a, bits)
    qmax = 2 ** (bits - 1) - 1
    assert s == np.float32(a) / np.float32(qmax) and inv == np.float32(qmax) / np.float32(a)
    q = orc.quantize(v, inv, bits)
    assert np.abs(q).max() == qmax and q[np.abs(v).argmax()] == int(np.sign(v[np.abs(v).argmax()])) * qmax
    err = np.abs(v.astype(np.float64) - float(s) * q)
    assert np.all(err <= float(s) / 2 * (1 + 2.0 ** -20))
    # re-quantizing the dequantized values gives the same codes; Q(-v) = -Q(v)
    deq = (q.astype(np.float32) * s).astype(np.float32)
    assert np.array_equal(orc.quantize(deq, inv, bits), q)
    assert np.array_equal(orc.quantize(-v, inv, bits), -q)


def test_quantizer_fixtures_f1_f2(golden):
    g = golden("f1_rotation_quantizer.txt")
    a = orc.absmax(g["rotated"])
    assert a == g["absmax"][0]
    s, inv = orc.scales(a, int(g["bits"][0]))
    assert orc.quantize(g["rotated"], inv, 8).tolist() == g["codes"]
    g = golden("f2_round_half_even.txt")
    s, inv = orc.scales(orc.absmax(g["values"]), int(g["bits"][0]))
    assert inv == 1.0 and s == 1.0
    assert orc.quantize(g["values"], inv, 4).tolist() == g["codes"]


def test_quantizer_zero_input_and_saturation():
    s, inv = orc.scales(0.0, 8)
    assert s == 0 and inv == 0
    assert not orc.quantize(np.zeros(8, np.float32), inv, 8).any()
    # a frozen scale that is exceeded saturates at +-qmax (never -128)
    s, inv = orc.scales(1.0, 8)
    assert orc.quantize([5.0, -5.0, 1.0, -1.0, 0.999], inv, 8).tolist() == [127, -127, 127, -127, 127]


# ---------------------------------------------------------------- integer matmul, epilogue

def _toy_net(bits, W2, b2, sine_last=False):
    """2 -> 4 -> 4 network whose second layer is the 4-wide toy layer under test."""
    weights = [np.zeros((4, 2), np.float32), W2.astype(np.float32)]
    biases = [np.zeros(4, np.float32), b2.astype(np.float32)]
    return orc.prepare(weights, biases, (2, 4, 4), 30.0, w_bits=bits, a_bits=bits, a_gran=1, rotate=False)


@pytest.mark.parametrize("bits", [2, 3])
def test_brute_force_all_code_vectors_on_a_4_wide_layer(bits):
    qmax = 2 ** (bits - 1) - 1
    rng = np.random.default_rng(bits)
    qw = rng.integers(-qmax, qmax + 1, size=(4, 4))
    qw[0, 0] = qmax                                    # the absmax weight maps to qmax
    W2 = qw * 0.125                                    # s_w = 0.125 * qmax / qmax exactly
    b2 = np.array([0.5, -0.25, 0.0, 1.0])
    net = _toy_net(bits, W2, b2)
    assert np.array_equal(net.layers[1].qw, qw)
    levels = range(-qmax, qmax + 1)
    vecs = np.array([v for v in itertools.product(levels, repeat=4) if max(map(abs, v)) == qmax])
    X = (vecs * 0.5).astype(np.float32)                # absmax = qmax/2 -> s_x = 0.5, codes = vecs
    r = orc.layer(net, 2, X)
    assert np.array_equal(r["codes"], vecs)
    s_w = float(net.layers[1].s_w[0])
    for t, v in enumerate(vecs):
        for m in range(4):
            acc = sum(int(v[k]) * int(qw[m, k]) for k in range(4))     # Python big integers
            assert r["acc"][t, m] == acc
            z = Fraction(s_w) * Fraction(float(r["s_x"][t])) * acc + Fraction(float(b2[m]))
            assert abs(r["Y"][t, m] - float(z)) <= 1e-15       # last layer: affine, no sine


def test_integer_matmul_matches_int64_product_and_hidden_layers_apply_sine():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    net = orc.prepare(weights, biases, w.dims, w.omega0, a_gran=1)
    rng = np.random.default_rng(11)
    X = rng.uniform(-1, 1, size=(33, 64)).astype(np.float32)
    r = orc.layer(net, 2, X)
    lay = net.layers[1]
    assert np.array_equal(r["acc"], r["codes"].astype(np.int64) @ lay.qw.astype(np.int64).T)
    assert np.abs(r["acc"]).max() <= 127 * 127 * 64
    z = lay.s_w.astype(np.float64)[None, :] * r["s_x"].astype(np.float64)[:, None] * r["acc"] + lay.b_pad.astype(np.float64)
    want = np.array([[math.sin(30.0 * v) for v in row] for row in z])
    assert np.allclose(r["Y"], want, rtol=0, atol=1e-15)
    assert np.array_equal(r["Xrot"].view(np.uint32), orc.rotate(X).view(np.uint32))


def test_first_layer_pads_coordinates_and_last_layer_pads_outputs():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    net = orc.prepare(weights, biases, w.dims, w.omega0, a_gran=1)
    assert (net.layers[0].K_pad, net.layers[0].M_pad) == (4, 64)
    assert (net.layers[-1].K_pad, net.layers[-1].M_pad) == (64, 4)
    assert not net.layers[-1].qw[1:].any() and not net.layers[-1].b_pad[1:].any()
    X = orc.pad_coords(w.coords()[:5])
    assert X.shape == (5, 4) and not X[:, 2:].any()
    out, per = orc.forward(net, w.coords()[:5], return_layers=True)
    assert out.shape == (5, 1)
    # the rotated first-layer input has the pattern [x+y, x-y, x+y, x-y]
    xr = per[0]["Xrot"]
    assert np.array_equal(xr[:, 0], xr[:, 2]) and np.array_equal(xr[:, 1], xr[:, 3])


# ---------------------------------------------------------------- whole network

def _net_error(bits, rotate=True):
    dims = (2, 64, 64, 3)
    weights, biases = dhq_inputs.siren_init(dims, 30.0, 21)
    coords = dhq_inputs.grid_coords(12, 12)
    net = orc.prepare(weights, biases, dims, 30.0, w_bits=bits, a_bits=bits, w_gran=1, a_gran=1, rotate=rotate)
    got = orc.forward(net, coords)
    want = odef.siren_forward(weights, biases, 30.0, coords)
    return np.abs(got - want).max(), got


def test_quantized_network_converges_to_the_unquantized_siren():
    # pins layer order, omega0 placement, biases, padding and the linear last layer:
    # any of those wrong leaves an error that does not shrink with the bit-width.
    e8, _ = _net_error(8)
    e12, _ = _net_error(12)
    e16, g16 = _net_error(16)
    assert e16 < 2e-4 and e12 < 4e-3
    assert e12 < e8 / 4 and e16 < e12 / 4
    # the rotation is compute-invariant: with and without it the 16-bit networks agree
    _, g16_plain = _net_error(16, rotate=False)
    assert np.abs(g16 - g16_plain).max() < 1e-3


def test_per_tensor_calibration_is_the_layerwise_maximum_and_freezes():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    coords = w.coords()[::7]
    net = orc.prepare(weights, biases, w.dims, w.omega0)
    with pytest.raises(RuntimeError):
        orc.forward(net, coords)
    frozen = orc.calibrate(net, coords)
    assert len(frozen) == 4 and all(f > 0 for f in frozen)
    out, per = orc.forward(net, coords, return_layers=True)
    for l, r in enumerate(per):
        assert frozen[l] == np.abs(r["Xrot"]).max()
        assert np.abs(r["codes"]).max() == 127
        assert np.all(r["s_x"] == orc.scales(frozen[l], 8)[0])
    # with frozen scales a token's output does not depend on the batch it arrives in
    sub = orc.forward(net, coords[5:9])
    assert np.array_equal(sub, out[5:9])


def test_zero_token_has_zero_codes_per_token():
    dims = (2, 64, 64, 1)
    weights, biases = dhq_inputs.siren_init(dims, 30.0, 0)
    net = orc.prepare(weights, biases, dims, 30.0, a_gran=1)
    out, per = orc.forward(net, np.zeros((1, 2), np.float32), return_layers=True)
    assert not per[0]["codes"].any() and per[0]["s_x"][0] == 0
    # the first layer then outputs sin(omega0 * b)
    assert np.allclose(per[0]["Y"][0], np.sin(30.0 * net.layers[0].b_pad.astype(np.float64)), atol=1e-15)


# ---------------------------------------------------------------- synthetic inputs

def test_synthetic_inputs_have_the_distributions_the_paper_describes():
    # Section III-A: first-layer weights roughly uniform in +-0.5; sine outputs U-shaped in [-1, 1]
    w = dhq_inputs.WORKLOADS["C2"]
    weights, biases = w.network()
    assert 0.45 < np.abs(weights[0]).max() <= 0.5
    assert np.abs(weights[1]).max() <= math.sqrt(6 / 256) / 30
    net = orc.prepare(weights, biases, w.dims, w.omega0, a_gran=1)
    _, per = orc.forward(net, w.coords()[::97], return_layers=True)
    y = per[0]["Y"]
    assert np.abs(y).max() <= 1.0
    assert (np.abs(y) > 0.8).mean() > (np.abs(y) < 0.2).mean()
    # generator self-check against the published first output of splitmix64 with seed 0
    assert int(dhq_inputs.splitmix64(0, 0, 1)[0]) == 0xE220A8397B1DCDAF


# ---------------------------------------------------------------- two-sided transform (Eq. 4-5 literally)

@pytest.mark.parametrize("shape", [(64, 2), (64, 64), (3, 256), (256, 256)])
def test_two_sided_weight_transform_matches_eq5_and_keeps_the_product(shape):
    d_out, d_in = shape
    rng = np.random.default_rng(d_out * 77 + d_in)
    W = rng.uniform(-0.1, 0.1, size=shape).astype(np.float32)
    if d_in == 2:
        weights, biases, dims, l = [W, np.zeros((1, d_out), np.float32)], [np.zeros(d_out, np.float32), np.zeros(1, np.float32)], (2, d_out, 1), 1
    elif d_out <= 4:
        weights, biases, dims, l = [np.zeros((d_in, 2), np.float32), W], [np.zeros(d_in, np.float32), np.zeros(d_out, np.float32)], (2, d_in, d_out), 2
    else:
        weights = [np.zeros((d_in, 2), np.float32), W, np.zeros((1, d_out), np.float32)]
        biases = [np.zeros(d_in, np.float32), np.zeros(d_out, np.float32), np.zeros(1, np.float32)]
        dims, l = (2, d_in, d_out, 1), 2
    lay = orc.prepare(weights, biases, dims, 30.0, rotate="both").layers[l - 1]
    K, M = lay.K_pad, lay.M_pad
    Wp = np.zeros((M, K))
    Wp[:d_out, :d_in] = W
    Wrot = lay.Wrot.astype(np.float64)
    # Eq. 5: W' = H_M W H_K / sqrt(M K); the oracle holds W' / sqrt(M K) (exact powers of two folded in)
    assert np.allclose(Wrot * math.sqrt(M * K), odef.transform_2d(Wp), atol=2e-6)
    # energy preservation (the sentence after Eq. 5)
    assert math.isclose(np.linalg.norm(Wrot) * math.sqrt(M * K), np.linalg.norm(Wp), rel_tol=1e-5)
    # the layer's product survives: H_M (W~ (H_K x)) = W x
    x = rng.uniform(-1, 1, size=K)
    x[d_in:] = 0
    Wt = odef.transform_2d(Wp) / math.sqrt(M * K)
    assert np.allclose(odef.hadamard(M) @ (Wt @ (odef.hadamard(K) @ x)), Wp @ x, rtol=1e-12, atol=1e-13)
    # one-sided and two-sided folds differ exactly by the output-side factor
    one = orc.prepare(weights, biases, dims, 30.0, rotate=True).layers[l - 1].Wrot.astype(np.float64)
    assert np.allclose(Wrot, odef.hadamard(M) @ one / M, atol=1e-7)


def test_two_sided_layer_brute_force_with_exact_rationals():
    # 2 -> 4 -> 4, 3-bit codes, per-token scales: every stage recomputed with Python integers
    # and Fractions from the oracle's own codes and scales; the second rotation must be applied
    # to the dequantized values, before the bias.
    rng = np.random.default_rng(11)
    weights = [rng.uniform(-0.5, 0.5, (4, 2)).astype(np.float32), rng.uniform(-0.3, 0.3, (4, 4)).astype(np.float32)]
    biases = [rng.uniform(-0.2, 0.2, 4).astype(np.float32), rng.uniform(-0.2, 0.2, 4).astype(np.float32)]
    net = orc.prepare(weights, biases, (2, 4, 4), 30.0, w_bits=3, a_bits=3, a_gran=1, rotate="both")
    H = closed_form(4)
    X = rng.uniform(-1, 1, (50, 4)).astype(np.float32)
    r = orc.layer(net, 2, X, want=("codes", "s_x", "acc", "Y"))
    lay = net.layers[1]
    for t in range(X.shape[0]):
        q = [int(v) for v in r["codes"][t]]
        acc = [sum(q[k] * int(lay.qw[m][k]) for k in range(4)) for m in range(4)]
        assert acc == [int(v) for v in r["acc"][t]]
        d = [Fraction(float(lay.s_w[m])) * Fraction(float(r["s_x"][t])) * acc[m] for m in range(4)]
        for j in range(4):
            z = sum(int(H[j][m]) * d[m] for m in range(4)) + Fraction(float(lay.b_pad[j]))
            assert abs(float(z) - r["Y"][t][j]) <= 1e-15 * max(1.0, abs(float(z)))


def test_two_sided_network_converges_to_the_unquantized_siren():
    # the same limit as for the one-sided fold: a misplaced second rotation, a wrong scale (1/M), a
    # bias added before the rotation or a rotated last layer leaves an error that does not shrink.
    e8, _ = _net_error(8, rotate="both")
    e12, _ = _net_error(12, rotate="both")
    e16, g16 = _net_error(16, rotate="both")
    assert e16 < 2e-4 and e12 < 4e-3
    assert e12 < e8 / 4 and e16 < e12 / 4
    _, g16_one = _net_error(16, rotate=True)
    assert np.abs(g16 - g16_one).max() < 1e-3


def test_two_sided_transform_makes_first_and_last_layer_weights_bell_shaped():
    # Section III-B / Fig. 4: after the Hadamard transform the uniform first layer and the two-peaked
    # last layer become bell-shaped.  Sanity statistic, not a parity gate: the excess kurtosis of the
    # entries moves from the flat / two-peaked range (about -1.2 and below -1) to near 0 (Gaussian),
    # while the input-side fold alone leaves a 2-input first layer as flat as it was (K = 4 mixes
    # two values).
    def excess_kurtosis(v):
        v = np.asarray(v, dtype=np.float64).ravel()
        v = v - v.mean()
        return float((v ** 4).mean() / (v ** 2).mean() ** 2 - 3.0)
    dims = (2, 256, 256, 256, 3)
    weights, _ = dhq_inputs.trained_like_init(dims, 30.0, 5)
    first = np.zeros((256, 4)); first[:, :2] = weights[0]
    last = np.zeros((4, 256)); last[:3] = weights[-1]
    assert excess_kurtosis(weights[0]) < -1.0                        # uniform
    assert excess_kurtosis(weights[-1]) < -1.0                       # two peaks
    k_first = excess_kurtosis(odef.transform_2d(first))
    k_last = excess_kurtosis(odef.transform_2d(last))
    assert abs(k_first) < 0.5 and abs(k_last) < 0.6
    assert excess_kurtosis(odef.input_side_fold(first)[:, :2]) < -0.5

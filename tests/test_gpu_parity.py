"""GPU parity: the CUDA library through its C ABI against the CPU oracle.

Integer stages (weight codes, activation codes, int32 accumulators) and scales must match bit
for bit; fp32 layer outputs within 1e-5 absolute of the oracle's fp64 epilogue.  Parity is taken
layer by layer on the library's own layer inputs (teacher forcing), because a sine evaluated in
fp32 cannot be bit-identical to an fp64 one and one flipped code downstream would otherwise
hide everything after it; the dump chain is checked to close, and the fused kernel's output
must equal the layer-by-layer path bit for bit.
"""
import numpy as np
import pytest
import torch

import dhq_inputs
from tests.gpu_util import TOL_Y, check_layers_against_oracle, check_weights, prepare_pair, run_debug, to_dev

pytestmark = pytest.mark.gpu

dhq = pytest.importorskip("paper_2508_13478_b200")
from oracle import dhq_oracle as orc  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2508_13478_b200 import build
    build.build()
    assert torch.cuda.is_available()


def _p1(workload, coords_np, fused=True, rotate=True):
    weights, biases = workload.network()
    h, net = prepare_pair(workload.dims, weights, biases, workload.omega0, workload.w_bits,
                          workload.a_bits, workload.w_gran, workload.a_gran, rotate=rotate)
    try:
        check_weights(h, net)
        cd = to_dev(coords_np)
        if workload.a_gran == 0:
            dhq.dhq_calibrate(h, cd)
        out_dbg, bufs = run_debug(h, net, cd)
        # (two-sided transform with a fused kernel: the scales were frozen by that kernel, on ITS activations,
        # which differ from the layer-by-layer route's in the last bits; the frozen values are compared below)
        both_fused = rotate == "both" and workload.w_gran == 0
        worst = check_layers_against_oracle(h, net, coords_np, out_dbg, bufs, calib_is_this_set=not both_fused)
        if fused:
            out = torch.full((coords_np.shape[0], workload.dims[-1]), float("nan"), device="cuda")
            dhq.dhq_forward(h, cd, out)
            torch.cuda.synchronize()
            assert dhq.dhq_last_status(h) == 0
            if rotate == "both" and workload.w_gran == 0:
                # one weight scale per tensor: dhq_forward runs the two-sided transform inside the fused
                # kernel (output-side rotation on the int32 accumulators, fp32 epilogue), the dumps above
                # come from the layer-by-layer kernel (fp64 rotation): two chains, each checked on its own
                out_obs, obs = run_debug(h, net, cd, fused=True)
                worst = max(worst, check_layers_against_oracle(h, net, coords_np, out_obs, obs))
                assert torch.equal(out.view(torch.int32), out_obs.view(torch.int32)), "dhq_forward != observed fused kernel"
            else:
                assert torch.equal(out.view(torch.int32), out_dbg.view(torch.int32)), "fused != layer-by-layer"
        return worst
    finally:
        dhq.dhq_destroy(h)


def test_layer_by_layer_path_alone_c1_and_per_token():
    w = dhq_inputs.WORKLOADS["C1"]
    _p1(w, w.coords(), fused=False)
    w3 = dhq_inputs.WORKLOADS["C3"]
    _p1(w3, w3.coords()[:3000], fused=False)


def test_c1_full_grid():
    w = dhq_inputs.WORKLOADS["C1"]
    _p1(w, w.coords())


def test_c2_full_grid():
    w = dhq_inputs.WORKLOADS["C2"]
    _p1(w, w.coords())


@pytest.mark.parametrize("name,count", [("C3", 20000 + 77), ("C4-W4A4", 12000 + 1), ("C4-W6A6", 12000 + 1),
                                        ("C5", 6000 + 13)])
def test_c3_c4_c5_sampled_tokens(name, count):
    w = dhq_inputs.WORKLOADS[name]
    coords = w.coords()
    idx = np.linspace(0, coords.shape[0] - 1, count).astype(np.int64)
    _p1(w, np.ascontiguousarray(coords[idx]))


@pytest.mark.parametrize("name", ["C3", "C4-W4A4", "C4-W6A6", "C5"])
def test_full_size_launch_on_sampled_outputs(name):
    # The launch bench.py times: the whole grid of the workload in one dhq_forward call.  The
    # oracle cannot run millions of tokens, so 3,000 tokens sampled over the grid are checked: the
    # full launch's outputs at those tokens must equal, bit for bit, a small launch over only those
    # tokens (same handle, same frozen scales), and that small launch is checked stage by stage
    # against the oracle.
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        check_weights(h, net)
        grid = to_dev(w.coords())
        if w.a_gran == 0:
            dhq.dhq_calibrate(h, grid)                       # scales frozen on the full grid
        full = torch.empty((w.n, w.dims[-1]), device="cuda")
        dhq.dhq_forward(h, grid, full)
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h) == 0
        assert torch.isfinite(full).all()
        idx = np.unique(np.concatenate([np.linspace(0, w.n - 1, 2990).astype(np.int64),
                                        np.arange(w.n - 10, w.n)]))      # includes the last tile
        sample_np = np.ascontiguousarray(w.coords()[idx])
        out_dbg, bufs = run_debug(h, net, to_dev(sample_np))
        check_layers_against_oracle(h, net, sample_np, out_dbg, bufs, calib_is_this_set=False)
        picked = full[torch.from_numpy(idx).cuda()]
        assert torch.equal(picked.view(torch.int32), out_dbg.view(torch.int32))
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("n", [1, 127, 128, 129, 255, 257, 1000])
def test_ragged_tails_small_width(n):
    w = dhq_inputs.WORKLOADS["C1"]
    _p1(w, w.coords()[:n])


@pytest.mark.parametrize("w_gran,a_gran", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("bits", [4, 8])
def test_granularity_and_bit_width_combinations(w_gran, a_gran, bits):
    wl = dhq_inputs.Workload("combo", (2, 128, 128, 128, 3), 30.0, 40 + bits, bits, bits, w_gran, a_gran, (40, 41))
    _p1(wl, wl.coords())


@pytest.mark.parametrize("width,a_gran", [(64, 1), (256, 0), (512, 1), (512, 0)])
def test_every_width_with_ragged_tail_and_several_rounds(width, a_gran):
    # more tiles than one round of the persistent grid holds at width 512, plus a ragged tail
    wl = dhq_inputs.Workload("w", (2, width, width, width, 3), 30.0, width + a_gran, 8, 8, 1 - a_gran, a_gran, (8, 8))
    coords = dhq_inputs.grid_coords(150, 131)[: 148 * 128 + 300 if width == 512 else 3000]
    _p1(wl, coords)


@pytest.mark.parametrize("name,count", [("C1", 4096), ("C2", 9000 + 5), ("C3", 9000 + 5), ("C5", 3000 + 7)])
def test_no_rotation_variant_uniform_quantizer(name, count):
    # DHQ_ROT_NONE: the uniform quantizer of the paper's comparison (Section IV-B), same path
    # without the Hadamard rotation of weights and activations
    w = dhq_inputs.WORKLOADS[name]
    coords = w.coords()
    idx = np.linspace(0, coords.shape[0] - 1, count).astype(np.int64)
    _p1(w, np.ascontiguousarray(coords[idx]), rotate=False)


@pytest.mark.parametrize("name,count", [("C1", 4096), ("C2", 9000 + 5), ("C3", 6000 + 3), ("C4-W4A4", 3000 + 1), ("C5", 2000 + 9)])
def test_two_sided_transform_layer_by_layer(name, count):
    # DHQ_ROT_BOTH: Eq. 4-5 literally.  Weight codes and scales, activation codes, scales and
    # accumulators bit-exact; the outputs (output-side rotation undone in fp64) within 1e-5.
    w = dhq_inputs.WORKLOADS[name]
    coords = w.coords()
    idx = np.linspace(0, coords.shape[0] - 1, count).astype(np.int64)
    _p1(w, np.ascontiguousarray(coords[idx]), rotate="both")


def test_two_sided_transform_wide_phases_host_buffers_and_static_scratch():
    dims = (2, 256, 256, 256, 3)
    weights, biases = dhq_inputs.trained_like_init(dims, 30.0, 12)
    weights[0] = (weights[0] * 4).astype(np.float32)          # phases of hundreds of radians
    weights[1] = (weights[1] * 6).astype(np.float32)
    coords = dhq_inputs.grid_coords(40, 50)
    h, net = prepare_pair(dims, weights, biases, 30.0, 8, 8, 1, 1, rotate="both")
    try:
        check_weights(h, net)
        out_dbg, bufs = run_debug(h, net, to_dev(coords))
        check_layers_against_oracle(h, net, coords, out_dbg, bufs)
        ch = torch.from_numpy(coords).pin_memory()
        oh = torch.zeros((coords.shape[0], 3)).pin_memory()
        dhq.dhq_forward_host(h, ch, oh)
        torch.cuda.synchronize()
        assert torch.equal(oh.view(torch.int32), out_dbg.cpu().view(torch.int32))   # per-channel weight scales: layer by layer
        with pytest.raises(dhq.DhqError) as e:
            dhq.dhq_forward_static_scratch(h, to_dev(coords[:100]), torch.empty((100, 3), device="cuda"))
        assert e.value.code == 2
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("name,count,rotate,s0", [("C1", 4096, True, 8.0), ("C2", 7000 + 3, True, 12.0), ("C3", 5000 + 1, True, 5.0),
                                                  ("C4-W4A4", 3000 + 7, True, 10.0), ("C2", 4000, False, 12.0), ("C2", 4000, "both", 6.0), ("C3", 3000, "both", 6.0),
                                                  ("C5", 2000 + 5, True, 20.0)])
def test_wavelet_activation_layer_by_layer(name, count, rotate, s0):
    # DHQ_ACT_GABOR: sin(omega0 z) exp(-(s0 z)^2) on layers 1..L-1 (the reading of the WIRE experiments'
    # activation); integer stages bit-exact, outputs within 1e-5 of the fp64 definition on the per-layer
    # dumps (layer-by-layer kernel); dhq_forward and the host-buffer route - the fused tensor-core kernel
    # with the wavelet epilogue, except for the two-sided transform with per-channel weight scales - give
    # the same bits (two-sided: within 1e-5 of the definition on each route, fp64 against fp32 epilogue)
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    coords = w.coords()
    coords = np.ascontiguousarray(coords[np.linspace(0, coords.shape[0] - 1, count).astype(np.int64)])
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran, rotate=rotate, gabor_s0=s0)
    try:
        check_weights(h, net)
        cd = to_dev(coords)
        if w.a_gran == 0:
            dhq.dhq_calibrate(h, cd)
        out_dbg, bufs = run_debug(h, net, cd)
        both_fused = rotate == "both" and w.w_gran == 0   # then the scales were frozen on the fused route's activations
        worst = check_layers_against_oracle(h, net, coords, out_dbg, bufs, calib_is_this_set=not both_fused)
        out = torch.full_like(out_dbg, float("nan"))
        dhq.dhq_forward(h, cd, out)
        oh = torch.zeros(out.shape).pin_memory()
        dhq.dhq_forward_host(h, torch.from_numpy(coords).pin_memory(), oh)
        torch.cuda.synchronize()
        if rotate == "both" and w.w_gran == 0:
            # fused two-sided route (integer H_M, fp32 epilogue) against the layer-by-layer one (fp64 H_M):
            # each layer within 1e-5 of the definition on either route, but not the same bits, and the
            # free-running chains then part at rounding ties; the fused route is checked layer by layer below
            assert torch.equal(oh.view(torch.int32), out.cpu().view(torch.int32))
        else:
            assert torch.equal(out.view(torch.int32), out_dbg.view(torch.int32))
            assert torch.equal(oh.view(torch.int32), out_dbg.cpu().view(torch.int32))
        # the envelope is really applied: the hidden activations differ from the plain sine's
        y1 = bufs["Y"][0].cpu().numpy()
        assert np.abs(y1).max() <= 1.0 and np.abs(y1).mean() < 0.6
        print(f"gabor {name} rotate={rotate}: outputs within {worst:.2e}")
        if rotate == "both" and w.w_gran == 1:   # two-sided with per-channel weight scales runs layer by layer: nothing fused to observe
            with pytest.raises(dhq.DhqError) as e:
                dhq.dhq_forward_fused_debug(h, cd, out)
            assert e.value.code == 2
        else:                  # the fused kernel's own per-layer values, same checks
            out_obs, bufs_obs = run_debug(h, net, cd, fused=True)
            check_layers_against_oracle(h, net, coords, out_obs, bufs_obs)
            assert torch.equal(out_obs.view(torch.int32), out.view(torch.int32))
    finally:
        dhq.dhq_destroy(h)


def test_trained_like_weights_and_wide_phases():
    # bell-shaped hidden weights, two-peaked last layer (Section III-A), and a first layer scaled up
    # so that phases reach hundreds of radians
    dims = (2, 256, 256, 256, 3)
    weights, biases = dhq_inputs.trained_like_init(dims, 30.0, 12)
    weights[0] = (weights[0] * 4).astype(np.float32)
    weights[1] = (weights[1] * 6).astype(np.float32)
    coords = dhq_inputs.grid_coords(50, 50)
    h, net = prepare_pair(dims, weights, biases, 30.0, 8, 8, 1, 1)
    try:
        check_weights(h, net)
        out_dbg, bufs = run_debug(h, net, to_dev(coords))
        check_layers_against_oracle(h, net, coords, out_dbg, bufs)
        out = torch.empty_like(out_dbg)
        dhq.dhq_forward(h, to_dev(coords), out)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int32), out_dbg.view(torch.int32))
    finally:
        dhq.dhq_destroy(h)


def test_zero_token_and_empty_batch():
    w = dhq_inputs.WORKLOADS["C3"]
    coords = np.zeros((130, 2), np.float32)
    coords[1:] = w.coords()[:129]
    _p1(w, coords)
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 1, 1)
    try:
        out = torch.zeros((0, 3), device="cuda")
        dhq.dhq_forward(h, torch.zeros((0, 2), device="cuda"), out)   # n = 0: no-op
        assert dhq.dhq_last_status(h) == 0
    finally:
        dhq.dhq_destroy(h)


def test_unsupported_and_invalid_arguments():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    W = [to_dev(x) for x in weights]
    B = [to_dev(x) for x in biases]
    with pytest.raises(dhq.DhqError) as e:
        dhq.dhq_prepare((2, 64, 64, 64, 1), W, B, w_bits=9)
    assert e.value.code == 2
    with pytest.raises(dhq.DhqError) as e:
        dhq.dhq_prepare((3, 64, 64, 64, 1), W, B)
    assert e.value.code == 2
    with pytest.raises(dhq.DhqError) as e:
        dhq.dhq_prepare((2, 64, 64, 64, 1), W, B, rotation=7)      # no such rotation mode
    assert e.value.code == 2
    h = dhq.dhq_prepare(w.dims, W, B)
    try:
        with pytest.raises(dhq.DhqError) as e:     # per-tensor scales not frozen yet
            dhq.dhq_forward_debug(h, to_dev(w.coords()[:8]))
        assert e.value.code == 5
    finally:
        dhq.dhq_destroy(h)


def test_forward_auto_calibrates_and_is_deterministic_and_batch_independent():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 0, 0)
    try:
        cd = to_dev(w.coords())
        out1 = torch.empty((w.n, 1), device="cuda")
        dhq.dhq_forward(h, cd, out1)                      # freezes the scales on this grid
        out2 = torch.empty_like(out1)
        dhq.dhq_forward(h, cd, out2)
        sub = torch.empty((300, 1), device="cuda")
        dhq.dhq_forward(h, cd[1000:1300].contiguous(), sub)
        torch.cuda.synchronize()
        assert torch.equal(out1.view(torch.int32), out2.view(torch.int32))
        assert torch.equal(sub.view(torch.int32), out1[1000:1300].view(torch.int32))
        # the frozen values are the oracle's own calibration on its own free-running chain, up to
        # the fp32-vs-fp64 sine: equal to a few ulps
        frozen = orc.calibrate(net, w.coords())
        for l in range(1, 5):
            a = dhq.dhq_get_layer(h, l)[2]
            assert abs(a - frozen[l - 1]) <= 2e-5 * max(1.0, abs(frozen[l - 1]))
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("a_gran", [0, 1])
def test_non_finite_coordinates_do_not_hang_or_disturb_other_tokens(a_gran):
    w = dhq_inputs.WORKLOADS["C2"]
    weights, biases = w.network()
    h, _ = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 1, a_gran)
    try:
        good = w.coords()[:1000].copy()
        if a_gran == 0:
            dhq.dhq_calibrate(h, to_dev(good))
        ref = torch.empty((1000, 3), device="cuda")
        dhq.dhq_forward(h, to_dev(good), ref)
        bad = good.copy()
        bad[3] = [np.nan, 0.5]
        bad[130] = [np.inf, -np.inf]
        bad[700] = [1e30, -1e30]
        out = torch.empty((1000, 3), device="cuda")
        dhq.dhq_forward(h, to_dev(bad), out)
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h) == 0                     # no wait ran out, the kernel returned
        keep = np.ones(1000, bool)
        keep[[3, 130, 700]] = False                            # every other token is untouched
        k = torch.from_numpy(keep).cuda()
        assert torch.equal(out[k].view(torch.int32), ref[k].view(torch.int32))
    finally:
        dhq.dhq_destroy(h)


def test_forward_on_a_side_stream():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    h, _ = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 0, 1)
    try:
        cd = to_dev(w.coords())
        ref = torch.empty((w.n, 1), device="cuda")
        dhq.dhq_forward(h, cd, ref)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        out = torch.zeros((w.n, 1), device="cuda")
        with torch.cuda.stream(side):
            dhq.dhq_forward(h, cd, out, stream=side)
        side.synchronize()
        assert torch.equal(out.view(torch.int32), ref.view(torch.int32))
    finally:
        dhq.dhq_destroy(h)


def test_forward_host_buffers():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    h, _ = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 0, 1)
    try:
        ch = torch.from_numpy(w.coords()).pin_memory()
        oh = torch.empty((w.n, 1)).pin_memory()
        dhq.dhq_forward_host(h, ch, oh)
        out = torch.empty((w.n, 1), device="cuda")
        dhq.dhq_forward(h, ch.cuda(), out)
        torch.cuda.synchronize()
        assert torch.equal(oh.view(torch.int32), out.cpu().view(torch.int32))
        assert dhq.dhq_launch_count(h) > 0
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("name,n", [("C2", 65536), ("C2", 5 * 37888 + 777), ("C3", 17 * 37888 + 129), ("C5", 3 * 18944 + 1)])
def test_forward_host_pinned_and_pageable(name, n):
    """Host buffers with n spanning several tile rounds.  Pinned buffers are read and written by
    the kernel itself through their device mapping; pageable buffers are staged and the call is
    cut into launches whose copies overlap the kernels.  Either way the result must equal one
    dhq_forward over device buffers: on the first call (which freezes per-tensor scales on all
    coordinates) and on later ones, from the default stream and from a side stream."""
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h, _ = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        coords = w.coords()
        reps = (n + coords.shape[0] - 1) // coords.shape[0]
        coords = np.ascontiguousarray(np.tile(coords, (reps, 1))[:n])
        d_L = w.dims[-1]
        ch = torch.from_numpy(coords).pin_memory()
        oh = torch.zeros((n, d_L)).pin_memory()
        dhq.dhq_forward_host(h, ch, oh)                 # first call: calibrates (per tensor) on all of it
        torch.cuda.synchronize()
        ref = torch.empty((n, d_L), device="cuda")
        dhq.dhq_forward(h, ch.cuda(), ref)
        torch.cuda.synchronize()
        ref_bits = ref.cpu().view(torch.int32)
        assert torch.equal(oh.view(torch.int32), ref_bits)
        oh.zero_()
        before = dhq.dhq_launch_count(h)
        dhq.dhq_forward_host(h, ch, oh)                 # pinned: one launch on the mapped buffers
        torch.cuda.synchronize()
        assert dhq.dhq_launch_count(h) - before == 1
        assert torch.equal(oh.view(torch.int32), ref_bits)
        side = torch.cuda.Stream()
        oh.zero_()
        with torch.cuda.stream(side):
            dhq.dhq_forward_host(h, ch, oh, stream=side)
        side.synchronize()
        assert torch.equal(oh.view(torch.int32), ref_bits)
        pageable = torch.zeros((n, d_L))
        before = dhq.dhq_launch_count(h)
        dhq.dhq_forward_host(h, torch.from_numpy(coords), pageable)     # staged, cut into launches
        torch.cuda.synchronize()
        assert dhq.dhq_launch_count(h) - before >= 2
        assert torch.equal(pageable.view(torch.int32), ref_bits)
        pageable.zero_()
        with torch.cuda.stream(side):
            dhq.dhq_forward_host(h, torch.from_numpy(coords), pageable, stream=side)
        side.synchronize()
        assert torch.equal(pageable.view(torch.int32), ref_bits)
        assert dhq.dhq_last_status(h) == 0
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("name,parts", [("C2", 2), ("C1", 3)])
def test_sharded_calibration_equals_whole_set(name, parts):
    """The coordinate set split into contiguous blocks, one handle per block (as one GPU each would
    hold), layer-by-layer calibration with the maximum exchanged on the host: the frozen values and
    the outputs must equal, bit for bit, those of one handle calibrated on the whole set.  One
    block is left empty on purpose in the three-way split."""
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    coords = w.coords()
    L = len(w.dims) - 1
    whole, _ = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, 0)
    handles = [prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, 0)[0] for _ in range(parts)]
    try:
        cd = to_dev(coords)
        dhq.dhq_calibrate(whole, cd)
        if parts == 3:
            bounds = [(0, 1000), (1000, 1000), (1000, w.n)]
        else:
            bounds = [dhq.shard_range(w.n, r, parts) for r in range(parts)]
        blocks = [cd[lo:hi].contiguous() for lo, hi in bounds]
        with pytest.raises(dhq.DhqError):
            dhq.dhq_calibrate_layer(handles[0], 2, blocks[0])       # layer 1 is not frozen yet
        for l in range(1, L + 1):
            for h, blk in zip(handles, blocks):
                dhq.dhq_calibrate_layer(h, l, blk)
            a = max(dhq.dhq_get_act_absmax(h, l) for h in handles)
            for h in handles:
                dhq.dhq_set_act_absmax(h, l, a)
        ref = torch.empty((w.n, w.dims[-1]), device="cuda")
        dhq.dhq_forward(whole, cd, ref)
        for h in handles:
            for l in range(1, L + 1):
                assert np.float32(dhq.dhq_get_layer(h, l)[2]).view(np.uint32) == np.float32(dhq.dhq_get_layer(whole, l)[2]).view(np.uint32)
            out = torch.empty((w.n, w.dims[-1]), device="cuda")
            dhq.dhq_forward(h, cd, out)
            torch.cuda.synchronize()
            assert torch.equal(out.view(torch.int32), ref.view(torch.int32))
            assert dhq.dhq_last_status(h) == 0
        # the helper with a host-side maximum over the emulated ranks gives the same values
        again = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, 0)[0]
        handles.append(again)
        others = {l: dhq.dhq_get_layer(whole, l)[2] for l in range(1, L + 1)}
        layer_no = iter(range(1, L + 1))
        frozen = dhq.calibrate_sharded(again, blocks[0], L, allreduce_max=lambda v: max(v, others[next(layer_no)]))
        assert [np.float32(v) for v in frozen] == [np.float32(others[l]) for l in range(1, L + 1)]
    finally:
        dhq.dhq_destroy(whole)
        for h in handles:
            dhq.dhq_destroy(h)


@pytest.mark.parametrize("name", ["C2", "C5"])
def test_buffers_that_are_only_8_byte_aligned_take_the_plain_paths(name):
    """Whole tiles travel by bulk copies only when the buffers are 16-byte aligned (coordinates at
    width 512, results of the host-buffer variant at width <= 256).  Buffers offset by one
    coordinate / one float are legal (8- and 4-byte aligned) and must give the same bits."""
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h, _ = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        n, d_L = 3 * 18944 + 77, w.dims[-1]
        coords = np.ascontiguousarray(w.coords()[: n + 1])
        dhq.dhq_calibrate(h, to_dev(w.coords()))
        cd = to_dev(coords)
        ref = torch.empty((n, d_L), device="cuda")
        dhq.dhq_forward(h, cd[1:].contiguous(), ref)                       # aligned copy of the same coordinates
        out = torch.empty((n, d_L), device="cuda")
        shifted = cd[1:]                                                   # a view: starts 8 bytes into the allocation
        assert shifted.data_ptr() % 16 == 8 and shifted.is_contiguous()
        dhq.dhq_forward(h, shifted, out)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int32), ref.view(torch.int32))
        ch = torch.from_numpy(coords).pin_memory()
        flat = torch.zeros(n * d_L + 1).pin_memory()
        oh = flat[1:].view(n, d_L)                                         # starts 4 bytes into the allocation
        assert oh.data_ptr() % 16 == 4
        dhq.dhq_forward_host(h, ch[1:], oh)
        torch.cuda.synchronize()
        assert torch.equal(oh.view(torch.int32), ref.cpu().view(torch.int32))
        assert dhq.dhq_last_status(h) == 0
    finally:
        dhq.dhq_destroy(h)


def test_pipe_micro_benchmarks_run():
    for pipe in ("ffma", "mufu_sin", "tensor_i8", "pass1", "pass2", "pass12"):
        ops, ms = dhq.dhq_measure_pipe(pipe, 200)
        assert ops > 1e11 and ms > 0


def test_two_handles_on_two_streams_at_once():
    # Two networks, each on its own stream, launches interleaved without waiting: every launch wants
    # all SMs and all of an SM's tensor memory, so the kernels queue behind each other on the device;
    # results must equal the serial ones and no bounded wait may run out.
    wa, wb = dhq_inputs.WORKLOADS["C2"], dhq_inputs.WORKLOADS["C3"]
    weights_a, biases_a = wa.network()
    weights_b, biases_b = wb.network()
    ha, _ = prepare_pair(wa.dims, weights_a, biases_a, wa.omega0, 8, 8, 0, 0)
    hb, _ = prepare_pair(wb.dims, weights_b, biases_b, wb.omega0, 8, 8, 1, 1)
    try:
        ca, cb = to_dev(wa.coords()), to_dev(wb.coords()[:100000])
        dhq.dhq_calibrate(ha, ca)
        ref_a = torch.empty((ca.shape[0], 3), device="cuda")
        ref_b = torch.empty((cb.shape[0], 3), device="cuda")
        dhq.dhq_forward(ha, ca, ref_a)
        dhq.dhq_forward(hb, cb, ref_b)
        torch.cuda.synchronize()
        sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
        outs_a = [torch.zeros_like(ref_a) for _ in range(6)]
        outs_b = [torch.zeros_like(ref_b) for _ in range(6)]
        for i in range(6):
            dhq.dhq_forward(ha, ca, outs_a[i], stream=sa)
            dhq.dhq_forward(hb, cb, outs_b[i], stream=sb)
        sa.synchronize()
        sb.synchronize()
        assert dhq.dhq_last_status(ha) == 0 and dhq.dhq_last_status(hb) == 0
        for o in outs_a:
            assert torch.equal(o.view(torch.int32), ref_a.view(torch.int32))
        for o in outs_b:
            assert torch.equal(o.view(torch.int32), ref_b.view(torch.int32))
    finally:
        dhq.dhq_destroy(ha)
        dhq.dhq_destroy(hb)

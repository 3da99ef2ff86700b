"""GPU parity of the fused tensor-core kernel itself, stage by stage.

dhq_forward_fused_debug runs the kernel that dhq_forward runs, compiled with stores at the places
where each per-layer value exists (codes on their way into the operand tile, activation scales,
int32 accumulators as read from tensor memory, layer outputs after the sine).  The oracle, given
the kernel's own input of each layer, must reproduce codes, scale bits and accumulators exactly and
the fp32 outputs within 1e-5; the chain must close and dhq_forward must return the same bits.
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


def _observe(h, net, coords_np, calib_is_this_set=True):
    cd = to_dev(coords_np)
    out_dump, bufs = run_debug(h, net, cd, fused=True)
    worst = check_layers_against_oracle(h, net, coords_np, out_dump, bufs, calib_is_this_set=calib_is_this_set)
    out = torch.full((coords_np.shape[0], net.dims[-1]), float("nan"), device="cuda")
    dhq.dhq_forward(h, cd, out)
    torch.cuda.synchronize()
    assert dhq.dhq_last_status(h) == 0
    assert torch.equal(out.view(torch.int32), out_dump.view(torch.int32)), "dhq_forward != observed fused kernel"
    return worst


@pytest.mark.parametrize("rotate", [True, False])
@pytest.mark.parametrize("width,a_gran", [(64, 0), (64, 1), (128, 0), (128, 1), (256, 0), (256, 1), (512, 0), (512, 1)])
def test_fused_kernel_stages_match_the_oracle(width, a_gran, rotate):
    # more than one round of the persistent grid (148 SMs x slots x 128 tokens) plus a ragged tail
    wl = dhq_inputs.Workload("obs", (2, width, width, width, 3), 30.0, 700 + width + a_gran, 8, 8, a_gran, a_gran, (8, 8))
    n = 148 * (1 if width == 512 else 2) * 128 + 300
    coords = dhq_inputs.grid_coords(251, 157)[:n]
    weights, biases = wl.network()
    h, net = prepare_pair(wl.dims, weights, biases, wl.omega0, 8, 8, a_gran, a_gran, rotate=rotate)
    try:
        check_weights(h, net)
        if a_gran == 0:
            dhq.dhq_calibrate(h, to_dev(coords))
        _observe(h, net, coords)
    finally:
        dhq.dhq_destroy(h)


def test_all_of_c3_through_the_observed_fused_kernel():
    # every coordinate of the 512 x 512 grid, 65,536 at a time
    w = dhq_inputs.WORKLOADS["C3"]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        check_weights(h, net)
        coords = w.coords()
        worst = 0.0
        for t0 in range(0, w.n, 65536):
            worst = max(worst, _observe(h, net, np.ascontiguousarray(coords[t0:t0 + 65536])))
        print(f"C3, all {w.n} coordinates: integer stages exact, outputs within {worst:.2e}")
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("name", ["C4-W4A4", "C4-W6A6", "C5"])
def test_contiguous_chunk_of_the_large_grids(name):
    # 65,536 consecutive coordinates from the middle of the grid: 1.7 rounds of the persistent grid
    # at width 256, 3.5 at width 512; per-tensor scales (C5) are frozen on the whole grid and the
    # first layer's frozen absmax is checked against the oracle on the whole grid
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        check_weights(h, net)
        coords = w.coords()
        if w.a_gran == 0:
            dhq.dhq_calibrate(h, to_dev(coords))
            a1 = float(orc.rotated_absmax(net, 1, orc.pad_coords(coords)).max())
            assert np.float32(dhq.dhq_get_layer(h, 1)[2]) == np.float32(a1)
        t0 = w.n // 2 - 12345
        _observe(h, net, np.ascontiguousarray(coords[t0:t0 + 65536]), calib_is_this_set=False)
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("name", ["C3", "C4-W4A4", "C4-W6A6", "C5"])
def test_full_grid_launch_equals_the_observed_kernel_on_samples(name):
    # The launch bench.py times (whole grid, one dhq_forward call) against the observed kernel on
    # 3,000 tokens sampled over the grid, the last tile included; those go through the oracle.
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        grid = to_dev(w.coords())
        if w.a_gran == 0:
            dhq.dhq_calibrate(h, grid)
            a1 = float(orc.rotated_absmax(net, 1, orc.pad_coords(w.coords())).max())
            assert np.float32(dhq.dhq_get_layer(h, 1)[2]) == np.float32(a1)
        full = torch.empty((w.n, w.dims[-1]), device="cuda")
        dhq.dhq_forward(h, grid, full)
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h) == 0
        idx = np.unique(np.concatenate([np.linspace(0, w.n - 1, 2990).astype(np.int64), np.arange(w.n - 10, w.n)]))
        sample = np.ascontiguousarray(w.coords()[idx])
        out_dump, bufs = run_debug(h, net, to_dev(sample), fused=True)
        check_layers_against_oracle(h, net, sample, out_dump, bufs, calib_is_this_set=False)
        assert torch.equal(full[torch.from_numpy(idx).cuda()].view(torch.int32), out_dump.view(torch.int32))
    finally:
        dhq.dhq_destroy(h)


def test_observed_kernel_equals_the_layer_by_layer_dumps():
    # two independent CUDA routes (tensor-core fused kernel, dp4a layer kernel) give the same dumps
    w = dhq_inputs.WORKLOADS["C3"]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        cd = to_dev(w.coords()[:5000])
        out_a, a = run_debug(h, net, cd, fused=True)
        out_b, b = run_debug(h, net, cd, fused=False)
        assert torch.equal(out_a.view(torch.int32), out_b.view(torch.int32))
        for key in ("X", "codes", "s_x", "acc", "Y"):
            for l in range(len(net.layers)):
                ta, tb = a[key][l], b[key][l]
                same = torch.equal(ta.view(torch.int32), tb.view(torch.int32)) if ta.dtype == torch.float32 else torch.equal(ta, tb)
                assert same, f"{key} of layer {l + 1}"
    finally:
        dhq.dhq_destroy(h)


def test_absmax_without_a_finite_scale_counts_as_zero():
    # coordinates so small that qmax / absmax overflows fp32: all codes zero, scale zero, and the
    # first layer then returns sin(omega0 b); just above the threshold the quantizer works normally
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 0, 1)
    try:
        coords = np.array([[1e-39, 0.0], [1e-38, -1e-38], [1e-37, 0.0], [3e-37, 1e-37], [1e-36, 0.0], [0.25, -0.5]], np.float32)
        cd = to_dev(coords)
        for fused in (False, True):
            out, bufs = run_debug(h, net, cd, fused=fused)
            check_layers_against_oracle(h, net, coords, out, bufs)
            codes = bufs["codes"][0].cpu().numpy()
            s_x = bufs["s_x"][0].cpu().numpy()
            assert not codes[:3].any() and not s_x[:3].any()
            assert np.abs(codes[3:]).max(axis=1).tolist() == [127, 127, 127] and (s_x[3:] > 0).all()
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("name", ["C2", "C3", "C5"])
def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable(name):
    # The copy warp leaves out one piece (the last layer's weights); nothing is in flight for it.
    # The warps that wait for it give up after the handle's wait limit, the kernel frees its tensor
    # memory and returns, the status word says TIMEOUT, and the next launch is bit-correct again.
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        coords = np.ascontiguousarray(w.coords()[:100])            # one tile
        cd = to_dev(coords)
        if w.a_gran == 0:
            dhq.dhq_calibrate(h, cd)
        ref = torch.empty((100, w.dims[-1]), device="cuda")
        dhq.dhq_forward(h, cd, ref)
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h) == 0
        dhq.dhq_set_wait_limit(h, 5_000_000)                       # 5 ms
        dhq.dhq_debug_stall_next_forward(h)
        junk = torch.zeros_like(ref)
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        dhq.dhq_forward(h, cd, junk)
        t1.record()
        torch.cuda.synchronize()
        assert t0.elapsed_time(t1) < 500.0                         # milliseconds: it gave up, it did not sit out 2 s
        assert dhq.dhq_last_status(h) == 6                         # DHQ_ERR_TIMEOUT
        assert dhq.dhq_last_status(h) == 0                         # reading clears it
        out = torch.zeros_like(ref)
        dhq.dhq_forward(h, cd, out)                                # the hook was for one launch only
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h) == 0
        assert torch.equal(out.view(torch.int32), ref.view(torch.int32))
        out_dump, bufs = run_debug(h, net, cd, fused=True)
        check_layers_against_oracle(h, net, coords, out_dump, bufs)
        with pytest.raises(dhq.DhqError):
            dhq.dhq_set_wait_limit(h, 10)                          # below the minimum
    finally:
        dhq.dhq_destroy(h)


def test_free_running_chains_differ_only_through_code_flips_at_rounding_ties():
    # Oracle on its own chain (fp64 sines rounded to fp32) against the kernel on its own chain (fp32
    # sines).  Every coordinate whose outputs differ by more than 1e-5 must trace back to a first
    # layer where an activation code differs, there by one step only, with the value to be rounded
    # next to a half-integer (as close as the two chains' inputs of that layer allow).
    w = dhq_inputs.WORKLOADS["C2"]
    weights, biases = w.network()
    coords = np.ascontiguousarray(w.coords()[::8])
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 0, 1)      # per-token scales: no calibration coupling
    try:
        out_dump, bufs = run_debug(h, net, to_dev(coords), fused=True)
        ref, per = orc.forward(net, coords, return_layers=True)
        got = out_dump.cpu().numpy().astype(np.float64)
        far = np.abs(got - ref).max(axis=1) > TOL_Y
        L = len(net.layers)
        gpu_codes = [bufs["codes"][l].cpu().numpy().astype(np.int32) for l in range(L)]
        gpu_X = [bufs["X"][l].cpu().numpy() for l in range(L)]
        first = np.full(coords.shape[0], -1)
        for l in range(L - 1, -1, -1):
            differs = (gpu_codes[l] != per[l]["codes"]).any(axis=1)
            first[differs] = l
        assert np.all(first[far] >= 0), "outputs differ although every code agrees"
        agree_everywhere = first < 0
        assert np.abs(got - ref)[agree_everywhere].max() <= TOL_Y
        flips = 0
        for t in np.nonzero(first >= 0)[0]:
            l = first[t]
            diff = gpu_codes[l][t] - per[l]["codes"][t]
            assert np.abs(diff).max() == 1
            inv = orc.scales(float(np.abs(per[l]["Xrot"][t]).max()), 8)[1]
            tq = per[l]["Xrot"][t].astype(np.float64) * float(inv)
            room = float(inv) * np.abs(gpu_X[l][t].astype(np.float64) - per[l]["X"][t]).sum() * 1.5 + 127 * 2.0 ** -20
            k = np.nonzero(diff)[0]
            assert np.all(np.abs(np.abs(tq[k] - np.floor(tq[k])) - 0.5) <= room), "a code differs away from a rounding tie"
            flips += 1
        print(f"free-running: {coords.shape[0]} coordinates, {int(far.sum())} beyond 1e-5 ({100 * far.mean():.2f} %), "
              f"{flips} with a first code flip (all by one step at a tie), max |d| = {np.abs(got - ref).max():.2e}")
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("width,scale", [(64, 10.0), (256, 10.0), (512, 10.0), (128, 16.0), (256, 25.0)])
def test_layers_without_a_phase_bound_decide_per_value(width, scale):
    # Per-token scales and a hidden layer whose phase bound is beyond the short sine's limit (32 rad): the
    # rule is per value - below the limit sin.approx of the plain fma phase, above it the compensated phase
    # with explicit reduction - and the fused kernel, which takes the short route for a whole chunk and
    # redoes the chunk when a warp met a larger phase, must give the bits of the layer-by-layer kernel,
    # which applies the rule value by value.  The weights are scaled so that both sides of the limit occur
    # (scale 10: a fraction of a percent of the phases, in a third of the tokens; 16: a few percent, in nearly
    # every token; 25: a fifth of them, phases to 130 rad).
    # (Beyond 256 rad the fp32 phase itself carries half an ulp of 1.5e-5 or more: outside the 1e-5 claim.)
    dims = (2, width, width, width, width, 3)
    weights, biases = dhq_inputs.Workload("mixed", dims, 30.0, 2100 + width, 8, 8, 1, 1, (8, 8)).network()
    weights[1] = (weights[1] * scale).astype(np.float32)
    weights[2] = (weights[2] * scale).astype(np.float32)
    n = 148 * (1 if width == 512 else 2) * 128 + 55
    coords = dhq_inputs.grid_coords(241, 163)[:n]
    h, net = prepare_pair(dims, weights, biases, 30.0, 8, 8, 1, 1)
    try:
        check_weights(h, net)
        cd = to_dev(coords)
        out_obs, bufs = run_debug(h, net, cd, fused=True)
        check_layers_against_oracle(h, net, coords, out_obs, bufs)
        for l in (2, 3):     # the phases that these layers really met, from the kernel's own accumulators and scales
            lay = net.layers[l - 1]
            acc = bufs["acc"][l - 1].cpu().numpy().astype(np.float64)
            s_x = bufs["s_x"][l - 1].cpu().numpy().astype(np.float64)
            phase = 30.0 * (acc * lay.s_w.astype(np.float64)[None, :] * s_x[:, None] + lay.b_pad.astype(np.float64)[None, :])
            above = float((np.abs(phase) > 32.0).mean())
            rows_clean = float((np.abs(phase).max(axis=1) <= 32.0).mean())
            print(f"width {width} scale {scale} layer {l}: {above:.2%} of the phases above the limit, {rows_clean:.1%} of the tokens all below")
            assert above > 1e-4
            if scale <= 16:
                assert above < 0.2
        out_lw, bufs_lw = run_debug(h, net, cd)                  # layer by layer: the rule value by value
        assert torch.equal(out_lw.view(torch.int32), out_obs.view(torch.int32))
        for l in range(len(dims) - 1):
            assert torch.equal(bufs_lw["Y"][l].view(torch.int32), bufs["Y"][l].view(torch.int32)), f"layer {l + 1} outputs"
        out = torch.empty_like(out_obs)
        dhq.dhq_forward(h, cd, out)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int32), out_obs.view(torch.int32))
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("w_bits,a_bits,d_out,omega0,width,gran", [
    (2, 2, 3, 30.0, 256, 0), (2, 2, 1, 30.0, 128, 1), (3, 5, 2, 30.0, 64, 1), (4, 8, 4, 30.0, 256, 1), (8, 4, 3, 30.0, 512, 0),
    (7, 7, 4, 30.0, 512, 1), (8, 8, 2, -30.0, 256, 0), (8, 8, 3, 1.0, 128, 0), (8, 8, 1, 75.0, 256, 1), (8, 8, 3, 75.0, 512, 0),
    (6, 8, 3, 0.0, 256, 0), (8, 8, 3, 0.0, 64, 1)])
def test_unequal_bit_widths_output_sizes_and_other_frequencies(w_bits, a_bits, d_out, omega0, width, gran):
    # every supported bit-width pair is a pair of 2..8; d_L is 1..4 (padded to 4); omega0 any finite
    # number: negative, small (phases of a fraction of a radian), large (phases of a hundred radians:
    # the explicit-reduction sine) and zero (every hidden activation is sin(0) = 0, so every later
    # layer sees the degenerate absmax 0 and the output is the last bias)
    dims = (2, width, width, width, d_out)
    wl = dhq_inputs.Workload("mix", dims, 30.0, 1700 + w_bits * 10 + a_bits + d_out, w_bits, a_bits, gran, gran, (8, 8))
    n = 148 * (1 if width == 512 else 2) * 128 + 41
    coords = dhq_inputs.grid_coords(229, 173)[:n]
    weights, biases = wl.network()
    h, net = prepare_pair(dims, weights, biases, omega0, w_bits, a_bits, gran, gran)
    try:
        check_weights(h, net)
        if gran == 0:
            dhq.dhq_calibrate(h, to_dev(coords))
        _observe(h, net, coords)
        if omega0 == 0.0:
            out = torch.empty((n, d_out), device="cuda")
            dhq.dhq_forward(h, to_dev(coords), out)
            assert torch.equal(out, torch.from_numpy(biases[-1]).cuda().expand(n, d_out))
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("width,a_gran", [(64, 0), (128, 1), (256, 0), (256, 1), (512, 0), (512, 1)])
@pytest.mark.parametrize("n_linear", [2, 3, 16])
def test_depths_from_one_hidden_layer_to_the_maximum(n_linear, width, a_gran):
    # L = 2 has no hidden layer on the tensor core (layer 1 on the CUDA cores, then the N = 16 last
    # layer), L = 3 one; 16 (the library's maximum) no longer keeps its weights resident in shared
    # memory at width 256 and leaves the width-512 ring few stages beside the per-layer constants
    dims = (2,) + (width,) * (n_linear - 1) + (3,)
    wl = dhq_inputs.Workload("depth", dims, 30.0, 1300 + width + n_linear, 8, 8, a_gran, a_gran, (8, 8))
    n = 148 * (1 if width == 512 else 2) * 128 + 77
    coords = dhq_inputs.grid_coords(233, 171)[:n]
    weights, biases = wl.network()
    h, net = prepare_pair(wl.dims, weights, biases, wl.omega0, 8, 8, a_gran, a_gran)
    try:
        check_weights(h, net)
        if a_gran == 0:
            dhq.dhq_calibrate(h, to_dev(coords))
        _observe(h, net, coords)
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("rotate", [True, False, "both"])
@pytest.mark.parametrize("width,a_gran,s0", [(64, 0, 6.0), (64, 1, 6.0), (128, 0, 9.0), (256, 0, 12.0), (256, 1, 12.0), (512, 0, 20.0), (512, 1, 20.0)])
def test_wavelet_activation_inside_the_fused_kernel(width, a_gran, s0, rotate):
    # DHQ_ACT_GABOR: the instantiation whose epilogue multiplies the sine by exp(-(s0 z)^2), observed
    # like the sine network's: codes, scales and accumulators exact, outputs within 1e-5 of the fp64
    # wavelet, over more than one round of the persistent grid plus a ragged tail
    # (the two-sided transform runs fused with one weight scale per tensor)
    w_gran = 0 if rotate == "both" else a_gran
    wl = dhq_inputs.Workload("obs", (2, width, width, width, 3), 30.0, 900 + width + a_gran, 8, 8, w_gran, a_gran, (8, 8))
    n = 148 * (1 if width == 512 else 2) * 128 + 300
    coords = dhq_inputs.grid_coords(251, 157)[:n]
    weights, biases = wl.network()
    h, net = prepare_pair(wl.dims, weights, biases, wl.omega0, 8, 8, w_gran, a_gran, rotate=rotate, gabor_s0=s0)
    try:
        check_weights(h, net)
        if a_gran == 0:
            dhq.dhq_calibrate(h, to_dev(coords))
        worst = _observe(h, net, coords)
        print(f"wavelet, width {width}, a_gran {a_gran}, rotate {rotate}: outputs within {worst:.2e}")
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.parametrize("width,a_gran", [(64, 0), (64, 1), (128, 1), (256, 0), (256, 1), (512, 0), (512, 1)])
def test_two_sided_transform_inside_the_fused_kernel(width, a_gran):
    # DHQ_ROT_BOTH with one weight scale per tensor: z = H_M (s_w s_x acc) + b with the rotation taken
    # on the int32 accumulators (exact), then the fp32 epilogue.  Accumulators are dumped before that
    # rotation (they are the definition's q_x q_W^T); the outputs must be within 1e-5 of the fp64 H_M product.
    wl = dhq_inputs.Workload("both", (2, width, width, width, 3), 30.0, 900 + width + a_gran, 8, 8, 0, a_gran, (8, 8))
    n = 148 * (1 if width == 512 else 2) * 128 + 300
    coords = dhq_inputs.grid_coords(251, 157)[:n]
    weights, biases = wl.network()
    h, net = prepare_pair(wl.dims, weights, biases, wl.omega0, 8, 8, 0, a_gran, rotate="both")
    try:
        check_weights(h, net)
        if a_gran == 0:
            dhq.dhq_calibrate(h, to_dev(coords))
        worst = _observe(h, net, coords)   # the frozen maxima too: the calibration runs the same kernel
        # the host-buffer route runs the same kernel
        oh = torch.zeros((n, 3)).pin_memory()
        dhq.dhq_forward_host(h, torch.from_numpy(coords).pin_memory(), oh)
        out = torch.empty((n, 3), device="cuda")
        dhq.dhq_forward(h, to_dev(coords), out)
        torch.cuda.synchronize()
        assert torch.equal(oh.view(torch.int32), out.cpu().view(torch.int32))
        print(f"two-sided, fused, width {width}, a_gran {a_gran}: outputs within {worst:.2e}")
    finally:
        dhq.dhq_destroy(h)


def test_two_sided_transform_with_per_channel_weight_scales_stays_layer_by_layer():
    w = dhq_inputs.WORKLOADS["C3"]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, 8, 8, 1, 1, rotate="both")
    try:
        cd = to_dev(w.coords()[:300])
        out = torch.empty((300, 3), device="cuda")
        with pytest.raises(dhq.DhqError) as e:
            dhq.dhq_forward_fused_debug(h, cd, out)
        assert e.value.code == 2
        dhq.dhq_forward(h, cd, out)                      # runs, layer by layer
        torch.cuda.synchronize()
        assert torch.isfinite(out).all() and dhq.dhq_last_status(h) == 0
    finally:
        dhq.dhq_destroy(h)


@pytest.mark.skipif(not __import__("os").environ.get("DHQ_FULL_PARITY"), reason="every coordinate of the large grids through the oracle: "
                    "minutes of CPU time per configuration; set DHQ_FULL_PARITY=1")
@pytest.mark.parametrize("name", ["C4-W4A4", "C4-W6A6", "C5"])
def test_every_coordinate_of_the_large_grids(name):
    # All 1,048,576 (C4) / 4,194,304 (C5) coordinates through the observed fused kernel and the oracle,
    # 65,536 at a time.  With per-tensor scales (C5) the frozen absmax of EVERY layer must equal the
    # maximum of the oracle's rotated absmax over the whole grid (the kernel's own layer inputs).
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h, net = prepare_pair(w.dims, weights, biases, w.omega0, w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        check_weights(h, net)
        coords = w.coords()
        L = len(net.layers)
        if w.a_gran == 0:
            dhq.dhq_calibrate(h, to_dev(coords))
        seen = np.zeros(L, np.float32)
        worst = 0.0
        for t0 in range(0, w.n, 65536):
            chunk = np.ascontiguousarray(coords[t0:t0 + 65536])
            cd = to_dev(chunk)
            out_dump, bufs = run_debug(h, net, cd, fused=True)
            worst = max(worst, check_layers_against_oracle(h, net, chunk, out_dump, bufs, calib_is_this_set=False))
            if w.a_gran == 0:
                for l in range(1, L + 1):
                    seen[l - 1] = max(seen[l - 1], orc.rotated_absmax(net, l, bufs["X"][l - 1].cpu().numpy()).max())
        if w.a_gran == 0:
            frozen = np.array([dhq.dhq_get_layer(h, l)[2] for l in range(1, L + 1)], np.float32)
            assert np.array_equal(frozen.view(np.uint32), seen.view(np.uint32)), (frozen, seen)
        print(f"{name}: all {w.n} coordinates, integer stages exact, outputs within {worst:.2e}")
    finally:
        dhq.dhq_destroy(h)

"""Seeded random configurations through the C ABI against the oracle: width, depth, output size, bit
widths, granularities, rotation mode, activation, omega0, batch size (1, tile edges, ragged, several
grid rounds) and coordinate sets (uniform random, grid, with zero tokens and corners) drawn together.
Each case: weight codes and scales exact; per-layer codes, scales, accumulators exact and outputs within
1e-5 on the kernel that dhq_forward runs (its observing instantiation where the handle has a fused
kernel, else the layer-by-layer dumps); dhq_forward and the host-buffer route return those bits.
"""
import numpy as np
import pytest
import torch

import dhq_inputs
from tests.gpu_util import check_layers_against_oracle, check_weights, prepare_pair, run_debug, to_dev

pytestmark = pytest.mark.gpu

dhq = pytest.importorskip("paper_2508_13478_b200")


def _draw(case):
    rng = np.random.default_rng(77_000 + case)
    width = int(rng.choice([64, 128, 256, 512]))
    n_linear = int(rng.integers(2, 8))
    d_out = int(rng.integers(1, 5))
    w_bits, a_bits = int(rng.integers(2, 9)), int(rng.integers(2, 9))
    w_gran, a_gran = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    rotate = [True, False, "both"][int(rng.integers(0, 3))]
    s0 = float(rng.choice([0.0, 0.0, rng.uniform(2, 25)]))
    omega0 = float(rng.choice([30.0, 30.0, rng.uniform(-60, 60)]))
    slots = 1 if width == 512 else 2
    n = int(rng.choice([1, 2, 127, 128, 129, 255, 1000, int(rng.integers(1, 148 * slots * 128 * 2)),
                        148 * slots * 128 + int(rng.integers(0, 300))]))
    n = min(n, 60000 // max(1, width // 128) if n_linear > 4 else 80000)   # keeps the oracle to seconds
    kind = int(rng.integers(0, 3))
    if kind == 1:
        coords = dhq_inputs.grid_coords(317, 263)[:n]
    else:
        coords = rng.uniform(-1, 1, size=(n, 2)).astype(np.float32)
        if kind == 2:
            coords[rng.integers(0, n, size=max(1, n // 50))] = 0.0           # zero tokens
            coords[rng.integers(0, n, size=max(1, n // 50))] = [1.0, -1.0]    # a corner of the domain
    dims = (2,) + (width,) * (n_linear - 1) + (d_out,)
    return dims, w_bits, a_bits, w_gran, a_gran, rotate, s0, omega0, np.ascontiguousarray(coords)


@pytest.mark.parametrize("case", range(48))
def test_random_configuration(case):
    dims, w_bits, a_bits, w_gran, a_gran, rotate, s0, omega0, coords = _draw(case)
    n = coords.shape[0]
    weights, biases = dhq_inputs.Workload("rnd", dims, 30.0, 9000 + case, w_bits, a_bits, w_gran, a_gran, (8, 8)).network()
    h, net = prepare_pair(dims, weights, biases, omega0, w_bits, a_bits, w_gran, a_gran, rotate=rotate, gabor_s0=s0)
    try:
        check_weights(h, net)
        cd = to_dev(coords)
        if a_gran == 0:
            dhq.dhq_calibrate(h, cd)
        try:
            out_obs, bufs = run_debug(h, net, cd, fused=True)
        except dhq.DhqError as e:       # a handle that runs layer by layer: its own dumps
            assert e.code == 2 and rotate == "both" and w_gran == 1
            out_obs, bufs = run_debug(h, net, cd)
        check_layers_against_oracle(h, net, coords, out_obs, bufs)
        out = torch.full((n, dims[-1]), float("nan"), device="cuda")
        dhq.dhq_forward(h, cd, out)
        oh = torch.zeros((n, dims[-1])).pin_memory()
        dhq.dhq_forward_host(h, torch.from_numpy(coords).pin_memory(), oh)
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h) == 0
        assert torch.equal(out.view(torch.int32), out_obs.view(torch.int32))
        assert torch.equal(oh.view(torch.int32), out.cpu().view(torch.int32))
    finally:
        dhq.dhq_destroy(h)

"""dhq_forward_static_scratch: the forward pass for callers that cannot allocate device memory
(a host framework owns the device heap, the memory budget is fixed at start-up, or an
allocation's implicit synchronisation is unacceptable in the serving loop).  Its scratch is a
fixed 16 MiB array inside the library, shared by every call.

Checked through the C ABI against dhq_forward on two calls in a row: the second call uses other
coordinates, so it also shows that what the first call left in the shared scratch does no harm.
This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import dhq_inputs

pytestmark = pytest.mark.gpu

dhq = pytest.importorskip("paper_2508_13478_b200")

TOL = 1e-5   # the tolerance of the other GPU tests; the two paths are in fact bit-identical


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("name,a_gran", [("C2", 0), ("C3", 1), ("C5", 0)])
def test_static_scratch_forward_matches_forward_twice_in_a_row(name, a_gran):
    from paper_2508_13478_b200 import build
    build.build()
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    grid = w.coords()
    h = dhq.dhq_prepare(w.dims, [_dev(x) for x in weights], [_dev(x) for x in biases], w.omega0,
                        w.w_bits, w.a_bits, w.w_gran, a_gran)
    try:
        if a_gran == 0:
            dhq.dhq_calibrate(h, _dev(grid[::8]))          # the allocating part happens up front
        # the largest batch the scratch holds (at width 512 this fills both halves of the array to
        # their last float), then a ragged one, then a small one
        batches = [grid[: dhq.DHQ_STATIC_MAX_TOKENS], grid[7000:7000 + dhq.DHQ_STATIC_MAX_TOKENS - 1], grid[5000:5000 + 1237]]
        # The documented set-up: the first call on a device looks up the array's address, which is
        # also when the driver brings the library image with its 16 MiB array onto the GPU.
        warm = _dev(grid[:8])
        dhq.dhq_forward_static_scratch(h, warm, torch.empty((8, w.dims[-1]), device="cuda"))
        torch.cuda.synchronize()
        for coords in batches:                              # calls in a row, same scratch
            cd = _dev(coords)
            want = torch.empty((coords.shape[0], w.dims[-1]), device="cuda")
            got = torch.full_like(want, float("nan"))
            dhq.dhq_forward(h, cd, want)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]      # the driver's own count of free device memory
            dhq.dhq_forward_static_scratch(h, cd, got)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
            assert dhq.dhq_last_status(h) == 0
            assert torch.isfinite(got).all()
            assert (got - want).abs().max().item() <= TOL
            assert torch.equal(got.view(torch.int32), want.view(torch.int32))
        # one token more than the fixed scratch holds: refused, nothing enqueued
        too_many = _dev(grid[: dhq.DHQ_STATIC_MAX_TOKENS + 1])
        out = torch.empty((too_many.shape[0], w.dims[-1]), device="cuda")
        with pytest.raises(dhq.DhqError) as e:
            dhq.dhq_forward_static_scratch(h, too_many, out)
        assert e.value.code == 7
    finally:
        dhq.dhq_destroy(h)


def test_static_scratch_forward_needs_frozen_scales():
    w = dhq_inputs.WORKLOADS["C1"]
    weights, biases = w.network()
    h = dhq.dhq_prepare(w.dims, [_dev(x) for x in weights], [_dev(x) for x in biases], w.omega0, 8, 8, 0, 0)
    try:
        cd = _dev(w.coords()[:64])
        out = torch.empty((64, 1), device="cuda")
        with pytest.raises(dhq.DhqError) as e:              # it may not calibrate: that allocates
            dhq.dhq_forward_static_scratch(h, cd, out)
        assert e.value.code == 5
    finally:
        dhq.dhq_destroy(h)

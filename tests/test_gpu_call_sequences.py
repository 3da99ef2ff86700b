"""Seeded random sequences of calls on one handle.  A coordinate's result depends on nothing but the
handle (per-token scales, or per-tensor scales once frozen), so whatever route computes a slice of the
coordinate set - dhq_forward, the pinned and the pageable host routes, the no-allocation entry point,
the observing kernel, the layer-by-layer dumps, an exported and re-imported handle, a side stream, a
forward after calibrating again on the same set - must return the bits of the reference run over the
whole set, whatever ran before it on the same handle.
"""
import numpy as np
import pytest
import torch

import dhq_inputs
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu

dhq = pytest.importorskip("paper_2508_13478_b200")

N = 30000


@pytest.mark.parametrize("case", range(24))
def test_every_route_returns_the_reference_bits(case):
    rng = np.random.default_rng(31_000 + case)
    width = int(rng.choice([64, 128, 256, 512]))
    n_linear, d_out = int(rng.integers(2, 6)), int(rng.integers(1, 5))
    w_bits, a_bits = int(rng.integers(3, 9)), int(rng.integers(3, 9))
    w_gran, a_gran = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    rot = int(rng.integers(0, 3))                                   # DHQ_ROT_INPUT, _BOTH, _NONE
    s0 = float(rng.choice([0.0, 0.0, rng.uniform(2, 20)]))          # > 0: wavelet activation
    dims = (2,) + (width,) * (n_linear - 1) + (d_out,)
    coords = rng.uniform(-1, 1, size=(N, 2)).astype(np.float32)
    weights, biases = dhq_inputs.Workload("seq", dims, 30.0, 6000 + case, w_bits, a_bits, w_gran, a_gran, (8, 8)).network()
    h = dhq.dhq_prepare(dims, [to_dev(w) for w in weights], [to_dev(b) for b in biases], 30.0, w_bits, a_bits, w_gran, a_gran,
                        rotation=rot, activation=dhq.DHQ_ACT_GABOR if s0 > 0 else dhq.DHQ_ACT_SINE, act_s0=s0)
    imported = []
    try:
        cd = to_dev(coords)
        dhq.dhq_calibrate(h, cd)
        ref = torch.empty((N, d_out), device="cuda")
        dhq.dhq_forward(h, cd, ref)
        torch.cuda.synchronize()
        both_fused = rot == dhq.DHQ_ROT_BOTH and w_gran == 0      # then the layer-by-layer route has other bits by design
        static_ok = rot != dhq.DHQ_ROT_BOTH and s0 == 0
        side = torch.cuda.Stream()
        ran = []
        for _ in range(25):
            op = int(rng.integers(0, 9))
            a = int(rng.integers(0, N - 1))
            n = min(int(rng.choice([1, 127, 128, 129, 4096, int(rng.integers(1, N - a + 1))])), N - a)
            want = ref[a:a + n]
            got = torch.full((n, d_out), float("nan"), device="cuda")
            sub = cd[a:a + n].contiguous()
            if op == 0:
                dhq.dhq_forward(h, sub, got)
            elif op in (1, 2):                                      # host buffers: pinned, pageable
                ch, oh = torch.from_numpy(coords[a:a + n].copy()), torch.zeros((n, d_out))
                if op == 1:
                    ch, oh = ch.pin_memory(), oh.pin_memory()
                dhq.dhq_forward_host(h, ch, oh)
                torch.cuda.synchronize()
                got = oh.cuda()
            elif op == 3:
                if not static_ok or n > dhq.DHQ_STATIC_MAX_TOKENS:
                    continue
                dhq.dhq_forward_static_scratch(h, sub, got)
            elif op == 4:
                try:
                    dhq.dhq_forward_fused_debug(h, sub, got)
                except dhq.DhqError as e:                           # a handle that runs layer by layer
                    assert e.code == 2
                    continue
            elif op == 5:
                if both_fused:
                    continue
                dhq.dhq_forward_debug(h, sub, got, None)
            elif op == 6:
                imported.append(dhq.dhq_import(dhq.dhq_export(h)))
                dhq.dhq_forward(imported[-1], sub, got)
            elif op == 7:
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    dhq.dhq_forward(h, sub, got, stream=side)
                side.synchronize()
            else:
                dhq.dhq_calibrate(h, cd)
                dhq.dhq_forward(h, sub, got)
            torch.cuda.synchronize()
            ran.append((op, a, n))
            assert dhq.dhq_last_status(h) == 0
            assert torch.equal(got.view(torch.int32), want.view(torch.int32)), f"route {op} on [{a}, {a + n}) after {ran[-5:-1]}"
        assert len(ran) >= 10
    finally:
        dhq.dhq_destroy(h)
        for x in imported:
            dhq.dhq_destroy(x)


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C5"])
def test_forward_can_be_captured_in_a_cuda_graph_and_replayed(name):
    # A serving loop captures the launch once and replays it on new coordinates in the same buffers.
    # dhq_forward on a calibrated handle enqueues only the fused kernel (no allocation, no synchronisation),
    # so stream capture takes it; the replays must give the bits of plain calls.
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h = dhq.dhq_prepare(w.dims, [to_dev(x) for x in weights], [to_dev(x) for x in biases], w.omega0,
                        w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    try:
        grid = w.coords()
        n = min(20000, grid.shape[0] // 3)
        dhq.dhq_calibrate(h, to_dev(grid[::7]))
        batches = [to_dev(grid[i * n:(i + 1) * n]) for i in range(3)]
        want = []
        for b in batches:
            o = torch.empty((n, w.dims[-1]), device="cuda")
            dhq.dhq_forward(h, b, o)
            want.append(o)
        torch.cuda.synchronize()
        buf_in = batches[0].clone()
        buf_out = torch.full((n, w.dims[-1]), float("nan"), device="cuda")
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            dhq.dhq_forward(h, buf_in, buf_out, stream=side)          # warm-up on the capture stream
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                dhq.dhq_forward(h, buf_in, buf_out, stream=torch.cuda.current_stream())
        launches = dhq.dhq_launch_count(h)
        for b, o in zip(batches, want):
            buf_in.copy_(b)
            buf_out.fill_(float("nan"))
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(buf_out.view(torch.int32), o.view(torch.int32))
        assert dhq.dhq_launch_count(h) == launches                    # replays go through no library call
        assert dhq.dhq_last_status(h) == 0
    finally:
        dhq.dhq_destroy(h)

"""dhq_export / dhq_import: a prepared, calibrated handle as bytes and back, bit-identical."""
import numpy as np
import pytest
import torch

import dhq_inputs
from tests.gpu_util import to_dev

dhq = pytest.importorskip("paper_2508_13478_b200")


def test_import_rejects_blocks_that_are_not_an_export():
    # header checks come before any CUDA call: runs without a GPU
    from paper_2508_13478_b200 import build
    build.build()
    for blob in (b"", b"x" * 64, b"DHQB200\0" + b"\0" * 4000):
        with pytest.raises(dhq.DhqError) as e:
            dhq.dhq_import(blob)
        assert e.value.code == 1


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["C1", "C3", "C5"])
def test_export_import_round_trip_is_bit_identical(name):
    from paper_2508_13478_b200 import build
    build.build()
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h = dhq.dhq_prepare(w.dims, [to_dev(x) for x in weights], [to_dev(x) for x in biases], w.omega0,
                        w.w_bits, w.a_bits, w.w_gran, w.a_gran)
    h2 = None
    try:
        coords = to_dev(w.coords()[: 40000])
        dhq.dhq_calibrate(h, coords)
        blob = dhq.dhq_export(h)
        h2 = dhq.dhq_import(blob)
        for l in range(1, len(w.dims)):
            a, b = dhq.dhq_get_layer(h, l), dhq.dhq_get_layer(h2, l)
            assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
            assert np.float32(a[2]).view(np.uint32) == np.float32(b[2]).view(np.uint32)
        out1 = torch.empty((coords.shape[0], w.dims[-1]), device="cuda")
        out2 = torch.full_like(out1, float("nan"))
        dhq.dhq_forward(h, coords, out1)
        dhq.dhq_forward(h2, coords, out2)        # no calibration happens here: the frozen scales came with the block
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h2) == 0
        assert torch.equal(out1.view(torch.int32), out2.view(torch.int32))
        assert dhq.dhq_export(h2) == blob         # exporting the import gives the same bytes
        bad = bytearray(blob)
        bad[len(bad) // 2] ^= 0x40                # one flipped bit in the arrays: checksum
        with pytest.raises(dhq.DhqError) as e:
            dhq.dhq_import(bytes(bad))
        assert e.value.code == 1
        with pytest.raises(dhq.DhqError):
            dhq.dhq_import(blob[: len(blob) - 100])   # truncated
    finally:
        dhq.dhq_destroy(h)
        if h2:
            dhq.dhq_destroy(h2)


@pytest.mark.gpu
@pytest.mark.parametrize("name,kw", [
    ("C2", dict(rotation=1)),                                   # two-sided transform inside the fused kernel (H_M u, H_M v travel too)
    ("C3", dict(rotation=1)),                                   # two-sided, per-channel scales: layer by layer
    ("C2", dict(rotation=2)),                                   # no rotation
    ("C2", dict(activation=1, act_s0=9.0)),                     # wavelet activation
    ("C5", dict(activation=1, act_s0=20.0, rotation=2)),
    ("C2", dict(a_bits=32)),                                    # W8A32
    ("C2", dict(w_bits=32, a_bits=32)),                         # W32A32 (fp32 weights travel)
    ("C4-W4A4", dict()),
])
def test_export_import_round_trip_of_the_other_datapaths(name, kw):
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    args = dict(w_bits=w.w_bits, a_bits=w.a_bits, w_gran=w.w_gran, a_gran=w.a_gran)
    args.update(kw)
    h = dhq.dhq_prepare(w.dims, [to_dev(x) for x in weights], [to_dev(x) for x in biases], w.omega0, **args)
    h2 = None
    try:
        coords = to_dev(w.coords()[: 20000 + 13])
        dhq.dhq_calibrate(h, coords)
        blob = dhq.dhq_export(h)
        h2 = dhq.dhq_import(blob)
        out1 = torch.empty((coords.shape[0], w.dims[-1]), device="cuda")
        out2 = torch.full_like(out1, float("nan"))
        dhq.dhq_forward(h, coords, out1)
        dhq.dhq_forward(h2, coords, out2)
        torch.cuda.synchronize()
        assert dhq.dhq_last_status(h2) == 0
        assert torch.isfinite(out1).all()
        assert torch.equal(out1.view(torch.int32), out2.view(torch.int32))
        assert dhq.dhq_export(h2) == blob
    finally:
        dhq.dhq_destroy(h)
        if h2:
            dhq.dhq_destroy(h2)


@pytest.mark.gpu
def test_call_log_is_written_when_asked_for():
    # DHQ_LOG is read once per process: run a small forward in a child process
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import torch, dhq_inputs, paper_2508_13478_b200 as d\n"
        "w = dhq_inputs.WORKLOADS['C1']; W, B = w.network()\n"
        "h = d.dhq_prepare(w.dims, [torch.from_numpy(x).cuda() for x in W], [torch.from_numpy(x).cuda() for x in B])\n"
        "c = torch.from_numpy(w.coords()[:300]).cuda(); o = torch.empty((300, 1), device='cuda')\n"
        "d.dhq_forward(h, c, o); torch.cuda.synchronize(); d.dhq_destroy(h)\n")
    for setting, expect in (("1", True), ("0", False)):
        env = dict(os.environ, DHQ_LOG=setting, PYTHONPATH=root)
        r = subprocess.run([sys.executable, "-c", code], env=env, cwd=root, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr
        assert ("[dhq] dhq_forward n=300" in r.stderr) == expect
        assert ("[dhq] dhq_prepare" in r.stderr) == expect
        if expect:
            assert "-> ok" in r.stderr and "fused" in r.stderr

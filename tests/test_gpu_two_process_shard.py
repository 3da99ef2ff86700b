"""One coordinate grid split over two processes (each with its own replica of the handle), as
`bench.py --gpus N --shard` splits it over GPUs: per-tensor scales frozen by the per-layer
all-reduce(max), every process runs only its block, and the blocks put together must equal, bit for
bit, one handle calibrated and run on the whole grid.

Both processes use the one GPU of the test box (their kernels are independent of each other: they
simply take turns on the device); the reduction runs over gloo.  On a multi-GPU node the same code
runs with one GPU per rank and NCCL.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, name, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import dhq_inputs
    import paper_2508_13478_b200 as dhq
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    coords = w.coords()
    lo, hi = dhq.shard_range(coords.shape[0], rank, world)
    h = dhq.dhq_prepare(w.dims, [torch.from_numpy(x).cuda() for x in weights], [torch.from_numpy(x).cuda() for x in biases],
                        w.omega0, w.w_bits, w.a_bits, w.w_gran, 0)
    block = torch.from_numpy(np.ascontiguousarray(coords[lo:hi])).cuda()
    frozen = dhq.calibrate_sharded(h, block, len(w.dims) - 1)          # all-reduce(max) per layer over the group
    res = torch.empty((hi - lo, w.dims[-1]), device="cuda")
    dhq.dhq_forward(h, block, res)
    torch.cuda.synchronize()
    status = dhq.dhq_last_status(h)
    dhq.dhq_destroy(h)
    out.put((rank, lo, hi, [float(f) for f in frozen], res.cpu().numpy(), status))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("name", ["C2", "C1"])
def test_two_processes_each_run_half_of_the_grid(name):
    sys.path.insert(0, ROOT)
    import dhq_inputs
    import paper_2508_13478_b200 as dhq
    from paper_2508_13478_b200 import build
    build.build()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, name, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted((out.get(timeout=300) for _ in procs), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    # the same grid on one handle in this process
    w = dhq_inputs.WORKLOADS[name]
    weights, biases = w.network()
    h = dhq.dhq_prepare(w.dims, [torch.from_numpy(x).cuda() for x in weights], [torch.from_numpy(x).cuda() for x in biases],
                        w.omega0, w.w_bits, w.a_bits, w.w_gran, 0)
    try:
        cd = torch.from_numpy(w.coords()).cuda()
        dhq.dhq_calibrate(h, cd)
        whole = torch.empty((w.n, w.dims[-1]), device="cuda")
        dhq.dhq_forward(h, cd, whole)
        torch.cuda.synchronize()
        want_frozen = [dhq.dhq_get_layer(h, l)[2] for l in range(1, len(w.dims))]
        whole = whole.cpu().numpy()
    finally:
        dhq.dhq_destroy(h)
    assert results[0][1] == 0 and results[0][2] == results[1][1] and results[1][2] == w.n       # disjoint, complete
    for rank, lo, hi, frozen, res, status in results:
        assert status == 0
        assert [np.float32(f) for f in frozen] == [np.float32(f) for f in want_frozen]              # same frozen scales on every rank
        assert np.array_equal(res.view(np.uint32), whole[lo:hi].view(np.uint32))                    # and the same bits

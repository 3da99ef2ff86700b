"""The N > 1 bookkeeping of bench.py on CPU: two gloo ranks, replicas of the same grid, the
slowest rank defines the step time and the aggregate is N times one replica's coordinates."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    import dhq_inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = dhq_inputs.WORKLOADS["C1"]
    coords = w.coords()                                   # every rank builds the same replica
    mine = [10.0 + 5.0 * rank, 20.0 - 3.0 * rank]          # per-rank timings (ms)
    total_ms, e2e_ms = bench.max_over_ranks(mine, world, "cpu")
    value = bench.aggregate_throughput(coords.shape[0], world, total_ms / 4)
    checksum = torch.tensor([float(coords.sum())], dtype=torch.float64)
    both = [torch.zeros_like(checksum) for _ in range(world)]
    dist.all_gather(both, checksum)
    out.put((rank, total_ms, e2e_ms, value, [float(b) for b in both]))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_replicas():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total_ms, e2e_ms, value, sums in results:
        assert total_ms == 15.0 and e2e_ms == 20.0            # max over ranks, element-wise
        assert value == 4096 * 2 / (15.0 / 4 * 1e-3)          # two replicas of 4,096 coordinates
        assert sums[0] == sums[1]                             # identical seeded inputs on both ranks

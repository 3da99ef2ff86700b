"""The N > 1 bookkeeping of bench.py on CPU: two gloo ranks.  Replicas of the same grid: the
slowest rank defines the step time and the aggregate is N times one replica's coordinates.  One
grid split over the ranks (--shard): the blocks are disjoint and complete, the aggregate is the one
grid over the slowest rank's time, and the per-layer maxima are exchanged by all-reduce."""
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
    value = bench.aggregate_throughput(coords.shape[0] * world, total_ms / 4)
    checksum = torch.tensor([float(coords.sum())], dtype=torch.float64)
    both = [torch.zeros_like(checksum) for _ in range(world)]
    dist.all_gather(both, checksum)
    # the sharded mode: this rank's block of the one grid
    from paper_2508_13478_b200.sharded import shard_range
    lo, hi = shard_range(coords.shape[0], rank, world)
    block = torch.tensor([float(hi - lo), float(coords[lo:hi].sum())], dtype=torch.float64)
    dist.all_reduce(block)
    sharded_value = bench.aggregate_throughput(coords.shape[0], total_ms / 4)
    out.put((rank, total_ms, e2e_ms, value, [float(b) for b in both], (lo, hi), [float(v) for v in block], sharded_value,
             float(coords.sum())))
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
    for rank, total_ms, e2e_ms, value, sums, block, reduced, sharded_value, whole_sum in results:
        assert total_ms == 15.0 and e2e_ms == 20.0            # max over ranks, element-wise
        assert value == 4096 * 2 / (15.0 / 4 * 1e-3)          # two replicas of 4,096 coordinates
        assert sums[0] == sums[1]                             # identical seeded inputs on both ranks
        assert block == (rank * 2048, (rank + 1) * 2048)      # --shard: contiguous halves of the one grid
        assert reduced[0] == 4096.0 and abs(reduced[1] - whole_sum) < 1e-6   # together they are the grid, once
        assert sharded_value == 4096 / (15.0 / 4 * 1e-3)      # strong scaling: one grid over the slowest rank's time


class _FakeApi:
    """Stands in for the C-ABI binding on a machine without a GPU: layer l of rank r 'measures'
    the value 1 + ((3 * r + 5 * l) % 7), and a layer may only be measured once the layer before it
    has been set, as the library demands."""

    def __init__(self, rank):
        self.rank, self.done, self.calls, self.set_values = rank, 0, [], []

    def dhq_calibrate_layer(self, handle, layer, coords, stream=None):
        assert layer == self.done + 1, "layers before this one are not frozen"
        self.calls.append(("measure", layer, 0 if coords is None else len(coords)))

    def dhq_get_act_absmax(self, handle, layer, stream=None):
        return float(1 + ((3 * self.rank + 5 * layer) % 7))

    def dhq_set_act_absmax(self, handle, layer, value, stream=None):
        self.done = layer
        self.set_values.append(value)


def _calib_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2508_13478_b200.sharded import calibrate_sharded, shard_range
    lo, hi = shard_range(4097, rank, world)
    api = _FakeApi(rank)
    frozen = calibrate_sharded(object(), list(range(lo, hi)), 4, api=api)     # default reduce: all-reduce(max) over gloo
    out.put((rank, (lo, hi), frozen, api.set_values, api.calls))
    dist.destroy_process_group()


def test_sharded_calibration_exchanges_one_maximum_per_layer_over_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    world = 2
    procs = [ctx.Process(target=_calib_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    expect = [float(max(1 + ((3 * r + 5 * l) % 7) for r in range(world))) for l in range(1, 5)]
    assert results[0][1] == (0, 2049) and results[1][1] == (2049, 4097)        # contiguous, disjoint, complete
    for rank, _, frozen, set_values, calls in results:
        assert frozen == expect and set_values == expect                       # every rank freezes the same maxima
        assert [c[1] for c in calls] == [1, 2, 3, 4]                           # one measurement per layer, in order


def test_shard_range_partitions_any_count():
    sys.path.insert(0, ROOT)
    from paper_2508_13478_b200.sharded import shard_range
    for n in (0, 1, 7, 4096, 65537):
        for world in (1, 2, 3, 8):
            blocks = [shard_range(n, r, world) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == n
            assert all(blocks[i][1] == blocks[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in blocks]
            assert max(sizes) - min(sizes) <= 1

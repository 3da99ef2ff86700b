"""Calibration of per-tensor activation scales when the coordinate set is split over ranks.

Coordinates are independent, so N GPUs each run the forward pass on their own contiguous block
with a replica of the handle and no communication.  The only quantity that couples the blocks
is the frozen per-tensor activation absmax of each layer, which is the maximum over the whole
set: one float per layer, exchanged between the measurement of a layer and its freezing.
"""
from __future__ import annotations

from . import binding


def shard_range(n: int, rank: int, world: int):
    """Contiguous block [lo, hi) of n coordinates for `rank` of `world`: sizes differ by at most one,
    earlier ranks take the larger blocks, every coordinate belongs to exactly one rank."""
    if world < 1 or not 0 <= rank < world or n < 0:
        raise ValueError("shard_range: need 0 <= rank < world and n >= 0")
    base, extra = divmod(n, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def _allreduce_max_torch(group=None):
    import torch
    import torch.distributed as dist

    def reduce(value: float) -> float:
        if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
            return value
        backend = dist.get_backend(group)
        t = torch.tensor([value], dtype=torch.float32, device="cuda" if backend == "nccl" else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
        return float(t.item())
    return reduce


def calibrate_sharded(handle, coords_part, n_layers: int, allreduce_max=None, group=None, stream=None, api=binding):
    """Freeze the handle's per-tensor activation scales on a coordinate set of which this rank
    holds `coords_part` (a CUDA fp32 [n_part][2] tensor, possibly empty).  Every rank calls this
    with its own part; `allreduce_max(float) -> float` returns the maximum over ranks (default:
    torch.distributed all-reduce on `group`).  Returns the frozen values, equal on all ranks and
    equal to what dhq_calibrate gives on the whole set."""
    reduce = allreduce_max or _allreduce_max_torch(group)
    frozen = []
    for layer in range(1, n_layers + 1):
        api.dhq_calibrate_layer(handle, layer, coords_part, stream)
        a = reduce(api.dhq_get_act_absmax(handle, layer, stream))
        api.dhq_set_act_absmax(handle, layer, a, stream)
        frozen.append(a)
    return frozen

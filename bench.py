#!/usr/bin/env python
"""Throughput of the fused DHQ forward (coordinates per second) on N GPUs of one node.

    python bench.py --gpus 1 --steps 200 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

A step is one dhq_forward call over the workload's whole coordinate grid (one launch of the
fused kernel).  Inputs are seeded and synthetic (SIREN-initialised network, pixel grid).  With
N > 1 every rank runs the same grid on its own GPU (independent replicas, no collective on the
data path), so the aggregate is N times the work: weak scaling.

Timing: CUDA events on the launching stream around each step, an L2 flush (a write of a buffer
larger than L2) between steps and outside the events, the per-step times summed; the maximum
over ranks is reported.  SM clocks and throttle reasons are sampled through NVML while the timed
steps run.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import dhq_inputs  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of one fused-kernel launch, from the ncu capture
# summarised in profiles/fused_kernel_w256_C2.md (full C2 grid, rotation on).
NCU_DRAM_BYTES_PER_LAUNCH = {("C2", "input", 65536): 780032 + 0}
METRIC = "coords/sec, fused W8A8 DHQ INR forward"
UNIT = "coords/s"
SM_COUNT = 148
FP32_LANES_PER_SM = 128


def rotations(mode: str) -> int:
    """Hadamard rotations per hidden activation vector: 0 (none), 1 (input side), 2 (both sides)."""
    return {"none": 0, "input": 1, "both": 2}[mode]


def alu_laneops_per_coord(dims, rotate=True) -> float:
    """Plain-ALU lane operations the method needs per coordinate: per element of every hidden
    activation vector log2(w) butterfly adds (none without the rotation) plus 7 (int->float,
    scale+bias fma, 2 for the sine's range handling, quantizer multiply, rounding,
    packing/abs-max)."""
    w = dims[1]
    hidden_vectors = len(dims) - 2
    return float(hidden_vectors * w * (7 + int(rotate) * int(np.log2(w))))


class ClockSampler:
    """Polls NVML for the SM clock and the clock-event reasons of one GPU while running."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _poll(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def work_per_coord(dims, rotate=True):
    """Algorithmic work of the method per coordinate: int8 multiply-adds of all layers (the two
    inputs padded to 4, the outputs of the last layer to 4), sines, and fp32 operations that only
    the fp32 pipe can do (butterfly adds, dequantization fma, quantizer multiply, rounding add)."""
    w, hidden_vectors, hidden_matmuls = dims[1], len(dims) - 2, len(dims) - 3
    macs = 4 * w + hidden_matmuls * w * w + 4 * w
    sines = hidden_vectors * w
    fp32 = hidden_vectors * w * (3 + int(rotate) * int(np.log2(w)))
    return macs, sines, fp32


def time_oracle(workload, steps, warmup, sample_tokens, rotate=True, min_seconds=0.0):
    """The CPU oracle, as it stands, on `sample_tokens` coordinates of the workload; with
    min_seconds the passes repeat until that much CPU time has been measured."""
    from oracle import dhq_oracle as orc
    weights, biases = workload.network()
    net = orc.prepare(weights, biases, workload.dims, workload.omega0, workload.w_bits, workload.a_bits,
                      workload.w_gran, workload.a_gran, rotate=rotate)
    coords = workload.coords()[:sample_tokens]
    if workload.a_gran == 0:
        orc.calibrate(net, coords)
    for _ in range(warmup):
        orc.forward(net, coords[: max(1, sample_tokens // 8)])
    t0 = time.perf_counter()
    done = 0
    while done < steps or time.perf_counter() - t0 < min_seconds:
        orc.forward(net, coords)
        done += 1
    dt = (time.perf_counter() - t0) / done
    return coords.shape[0] / dt, dt, orc.threads(), done


def run_reference(args, workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = min(workload.n, 16384)
    steps = max(1, min(args.steps, 5))
    warmup = min(args.warmup, 1)
    value, dt, cores, _ = time_oracle(workload, steps, warmup, sample, rotations(args.rotation))
    desc = f"first {sample} coordinates of the {workload.grid[0]}x{workload.grid[1]} grid per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 (int64 accumulate, f64 epilogue)", "data": "synthetic",
        "config": {"workload": workload.name, "dims": list(workload.dims), "bits": [workload.w_bits, workload.a_bits]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(values, world, device):
    """Element-wise maximum of per-rank timings (the slowest rank defines the step time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(coords_per_rank, world, ms_per_step):
    """Whole-job coordinates per second: every rank runs its own replica of the grid."""
    return coords_per_rank * world / (ms_per_step * 1e-3)


def run_ours(args, workload):
    import torch
    import torch.distributed as dist
    import paper_2508_13478_b200 as dhq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dhq.load_library()

    weights, biases = workload.network()
    coords_np = workload.coords()
    if args.limit_coords > 0:
        coords_np = np.ascontiguousarray(coords_np[: args.limit_coords])
    n, d_L = coords_np.shape[0], workload.dims[-1]
    W = [torch.from_numpy(w).cuda() for w in weights]
    B = [torch.from_numpy(b).cuda() for b in biases]
    h = dhq.dhq_prepare(workload.dims, W, B, workload.omega0, workload.w_bits, workload.a_bits,
                        workload.w_gran, workload.a_gran, rotation={"input": 0, "both": 1, "none": 2}[args.rotation])
    coords = torch.from_numpy(coords_np).cuda()
    out = torch.empty((n, d_L), dtype=torch.float32, device="cuda")
    coords_host = torch.from_numpy(coords_np).pin_memory()
    out_host = torch.empty((n, d_L), dtype=torch.float32).pin_memory()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")   # > 126 MB of L2
    stream = torch.cuda.current_stream()

    dhq.dhq_calibrate(h, coords)          # per-tensor scales frozen on the workload's grid; no-op per token
    for _ in range(max(args.warmup, 3)):
        dhq.dhq_forward(h, coords, out)
        dhq.dhq_forward_host(h, coords_host, out_host)
    torch.cuda.synchronize()
    if dhq.dhq_last_status(h) != 0:
        raise SystemExit("device-side wait timed out during warm-up")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for a, b in evs:
            flush.fill_(1)
            a.record(stream)
            fn()
            b.record(stream)
        barrier()
        return sum(a.elapsed_time(b) for a, b in evs)   # ms

    launches0 = dhq.dhq_launch_count(h)
    with ClockSampler(physical_gpu_index(local_rank)) as clocks:
        total_ms = timed(lambda: dhq.dhq_forward(h, coords, out), args.steps)
    launches = dhq.dhq_launch_count(h) - launches0
    e2e_ms = timed(lambda: dhq.dhq_forward_host(h, coords_host, out_host), args.steps)
    status = dhq.dhq_last_status(h)

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], world, "cuda")
    ms_per_step = total_ms / args.steps
    value = aggregate_throughput(n, world, ms_per_step)
    e2e_value = aggregate_throughput(n, world, e2e_ms / args.steps)

    if rank == 0:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        sm_max = float(peaks.get("sm_max_mhz", 1965.0))
        alu_peak = SM_COUNT * FP32_LANES_PER_SM * sm_max * 1e6 / 1e12            # T lane-ops/s
        achieved = alu_laneops_per_coord(workload.dims, rotations(args.rotation)) * n / (ms_per_step * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8 (int32 accumulate, f32 epilogue)",
            "data": "synthetic",
            "config": {"workload": workload.name, "dims": list(workload.dims), "coords_per_step": n,
                       "bits": [workload.w_bits, workload.a_bits], "w_gran": workload.w_gran,
                       "a_gran": workload.a_gran, "rotation": args.rotation, "l2": "flushed between steps (256 MB write)",
                       "parallelism": f"{world} independent replica(s)"},
            "clocks": clocks.summary(),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": n * 8, "d2h_bytes_per_step": n * d_L * 4,
                    "ms_per_step": e2e_ms / args.steps,
                    "route": "dhq_forward_host on pinned host buffers: the kernel reads the coordinates and writes "
                             "the result over the host link through the buffers' device mapping, every step "
                             "(whole tiles by bulk copy where the width's kernel has that variant)"},
            "gpu_launches": launches,
            "roofline": {"bound": "alu", "achieved": achieved, "peak": alu_peak, "unit": "Tlaneop/s",
                         "frac": achieved / alu_peak,
                         "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((workload.name, args.rotation, n)),
                         "peak_source": "148 SMs x 128 fp32 lanes x max SM clock (derived, not measured)"},
            "device_status": status,
        }
        # The same launch against the other pipes' ceilings, each measured now on this GPU by the
        # library's own micro-benchmarks (perfect-overlap model: each pipe alone).
        macs, sines, fp32_ops = work_per_coord(workload.dims, rotations(args.rotation))
        per_s = n / (ms_per_step * 1e-3)
        pipes = {}
        for key, pipe, work in (("tensor_i8", "tensor_i8", 2.0 * macs), ("sfu_sine", "mufu_sin", float(sines)),
                                ("fp32", "fadd", float(fp32_ops))):
            try:
                peak, _ = dhq.dhq_measure_pipe(pipe, 2000)
                pipes[key] = {"achieved": work * per_s, "peak_measured": peak, "frac": work * per_s / peak,
                              "unit": "op/s", "per_coord": work}
            except Exception as exc:       # a failed micro-benchmark must not lose the bench line
                pipes[key] = {"error": str(exc)}
        if workload.dims[1] == 256:
            # the kernel's own per-element loops (pass 1 + pass 2 of a hidden layer) run alone:
            # what the arithmetic would reach with every wait hidden, in activation elements per second
            try:
                alone, _ = dhq.dhq_measure_pipe("pass12", 200)
                elems = float((len(workload.dims) - 2) * workload.dims[1])
                pipes["inner_loops_alone"] = {"achieved": elems * per_s, "peak_measured": alone, "frac": elems * per_s / alone,
                                              "unit": "activation elements/s", "per_coord": elems}
            except Exception as exc:
                pipes["inner_loops_alone"] = {"error": str(exc)}
        line["pipes"] = pipes
        if world == 1 and not args.no_cpu_baseline:
            sample = min(n, 65536)
            v, dt, cores, passes = time_oracle(workload, 1, 1, sample, rotations(args.rotation), min_seconds=10.0)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"first {sample} coordinates of the grid, {passes} pass(es) of {dt:.1f} s"}
        print(json.dumps(line), flush=True)
    dhq.dhq_destroy(h)
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args, workload):
    """Batch-size sweep of the workload's network: n = 2^12 .. 2^24 coordinates, activation
    scales frozen once on the workload's own grid (so a coordinate's result does not depend on
    the batch).  One JSON line with the throughput curve; single GPU."""
    import torch
    import paper_2508_13478_b200 as dhq

    torch.cuda.set_device(0)
    weights, biases = workload.network()
    d_L = workload.dims[-1]
    h = dhq.dhq_prepare(workload.dims, [torch.from_numpy(w).cuda() for w in weights],
                        [torch.from_numpy(b).cuda() for b in biases], workload.omega0, workload.w_bits,
                        workload.a_bits, workload.w_gran, workload.a_gran,
                        rotation={"input": 0, "both": 1, "none": 2}[args.rotation])
    dhq.dhq_calibrate(h, torch.from_numpy(workload.coords()).cuda())
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    points = []
    for k in range(12, 25):
        coords = torch.from_numpy(dhq_inputs.sweep_grid(k)).cuda()
        n = coords.shape[0]
        out = torch.empty((n, d_L), dtype=torch.float32, device="cuda")
        for _ in range(3):
            dhq.dhq_forward(h, coords, out)
        times = []
        for _ in range(args.sweep_reps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            dhq.dhq_forward(h, coords, out)
            b.record(stream)
            b.synchronize()
            times.append(a.elapsed_time(b))
        ms = float(np.median(times))
        points.append({"log2_n": k, "n": n, "ms": ms, "coords_per_s": n / (ms * 1e-3)})
    status = dhq.dhq_last_status(h)
    dhq.dhq_destroy(h)
    print(json.dumps({"metric": METRIC, "unit": UNIT, "n_gpus": 1, "data": "synthetic",
                      "config": {"workload": workload.name, "dims": list(workload.dims), "sweep": "n = 2^12 .. 2^24",
                                 "l2": "flushed before every timed call", "timing": f"median of {args.sweep_reps} calls"},
                      "device_status": status, "sweep": points}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C2", choices=sorted(dhq_inputs.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rotation", default="input", choices=["input", "none", "both"],
                    help="input = DHQ; none = the same path without the Hadamard rotation (uniform quantizer); "
                         "both = the two-sided transform of Eq. 4-5, run layer by layer")
    ap.add_argument("--limit-coords", type=int, default=0,
                    help="use only the first N coordinates of the workload's grid (profiling captures)")
    ap.add_argument("--sweep", action="store_true", help="batch-size sweep 2^12..2^24 instead of the timed steps")
    ap.add_argument("--sweep-reps", type=int, default=20)
    args = ap.parse_args()
    workload = dhq_inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, workload)
    elif args.sweep:
        run_sweep(args, workload)
    else:
        run_ours(args, workload)


if __name__ == "__main__":
    main()

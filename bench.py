#!/usr/bin/env python
"""Throughput of the fused DHQ forward (coordinates per second) on N GPUs of one node.

    python bench.py --gpus 1 --steps 200 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

A step is one dhq_forward call over the workload's whole coordinate grid (one launch of the
fused kernel).  The default workload is the largest single-GPU configuration, C5 (width 512,
2048 x 2048 grid); the other configurations are timed briefly in the same process and listed under
"per_config".  Inputs are seeded and synthetic (SIREN-initialised network, pixel grid).  With
N > 1 every rank runs the same grid on its own GPU (independent replicas, no collective on the
data path), so the aggregate is N times the work: weak scaling; with --shard the one grid is
split over the ranks instead (per-tensor scales frozen with an all-reduce(max) per layer):
strong scaling.

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

# dram__bytes_read.sum + dram__bytes_write.sum of one fused-kernel launch as ncu counted it, per
# workload (rotation on): (bytes, coordinates of the captured launch).  Captures of the large grids
# cover a few hundred thousand coordinates; a launch's traffic is the weights once plus a fixed
# amount per coordinate, so it is scaled to the timed launch by the coordinate count.  An entry is
# removed (traffic: null) when the kernel changes after its capture.
NCU_DRAM_BYTES = {
    ("C1", "input"): (99328, 4096),
    ("C2", "input"): (782080, 65536),
    ("C3", "input"): (2504704, 262144),
    ("C4-W4A4", "input"): (2875648, 303104),
    ("C4-W6A6", "input"): (2835968, 303104),
    ("C5", "input"): (3344896, 303104),
}
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


SAMPLE_TOKENS = 16384   # coordinates per pass of the CPU oracle (cpu_baseline and --impl reference)


def oracle_sample(workload, rotation="input"):
    """The bounded sample both CPU legs run: a contiguous block of SAMPLE_TOKENS coordinates from
    the middle of the workload's grid (the whole grid if it is smaller)."""
    coords = workload.coords()
    n = min(coords.shape[0], SAMPLE_TOKENS)
    lo = (coords.shape[0] - n) // 2
    desc = (f"{n} consecutive coordinates from the middle of the {workload.grid[0]}x{workload.grid[1]} grid "
            f"(tokens {lo}..{lo + n - 1}) per pass")
    return np.ascontiguousarray(coords[lo:lo + n]), desc


def time_oracle(workload, steps, warmup, rotate=True, min_seconds=0.0, variant="definition"):
    """The CPU oracle, as it stands, on the bounded sample of the workload; with min_seconds the
    passes repeat until that much time has been measured.  variant "definition" is the parity
    reference (O(n^2) rotation, as the paper's formula reads); "nlogn" the same layer with the
    rotation as a butterfly.  Returns (coords/s, seconds per pass, threads, passes, sample text)."""
    from oracle import dhq_oracle as orc
    from oracle import dhq_oracle_nlogn as orcn
    weights, biases = workload.network()
    net = orc.prepare(weights, biases, workload.dims, workload.omega0, workload.w_bits, workload.a_bits,
                      workload.w_gran, workload.a_gran, rotate=rotate)
    coords, desc = oracle_sample(workload)
    if workload.a_gran == 0:
        orc.calibrate(net, coords)
    fwd = orc.forward if variant == "definition" else orcn.forward
    for _ in range(warmup):
        fwd(net, coords[: max(1, coords.shape[0] // 8)])
    t0 = time.perf_counter()
    done = 0
    while done < steps or time.perf_counter() - t0 < min_seconds:
        fwd(net, coords)
        done += 1
    dt = (time.perf_counter() - t0) / done
    return coords.shape[0] / dt, dt, orc.threads(), done, desc


def config_of(workload, args, world):
    """The `config` object of the JSON line, the same for both arms."""
    mode = "one grid split over the ranks" if args.shard else "independent replica(s)"
    return {"workload": workload.name, "dims": list(workload.dims), "coords_per_step": workload.n if args.limit_coords <= 0 else min(workload.n, args.limit_coords),
            "bits": [workload.w_bits, workload.a_bits], "w_gran": workload.w_gran, "a_gran": workload.a_gran,
            "rotation": args.rotation, "variant": args.variant, "activation": "gabor" if getattr(args, "gabor_s0", 0.0) > 0 else "sine", "l2": "flushed between steps (256 MB write)",
            "parallelism": f"{world} x {mode}"}


def run_reference(args, workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 5))
    warmup = min(args.warmup, 1)
    value, dt, cores, _, desc = time_oracle(workload, steps, warmup, rotations(args.rotation))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "strong" if args.shard else "weak",
        "vs_baseline": None, "dtype": "int8 (int64 accumulate, f64 epilogue)", "data": "synthetic",
        "config": config_of(workload, args, int(os.environ.get("WORLD_SIZE", "1"))),
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


def aggregate_throughput(total_coords, ms_per_step):
    """Whole-job coordinates per second: all coordinates all ranks processed in a step over the
    slowest rank's step time."""
    return total_coords / (ms_per_step * 1e-3)


class Runner:
    """One workload on this rank's GPU: handle, device and pinned host buffers, timed loops."""

    def __init__(self, dhq, workload, rotation, limit_coords=0, shard=None, group=None, gabor_s0=0.0):
        import torch
        self.dhq, self.torch, self.workload = dhq, torch, workload
        weights, biases = workload.network()
        coords_np = workload.coords()
        if limit_coords > 0:
            coords_np = coords_np[:limit_coords]
        self.n_total = coords_np.shape[0]
        if shard is not None:                      # (rank, world): this rank's contiguous block
            lo, hi = dhq.shard_range(self.n_total, shard[0], shard[1])
            coords_np = coords_np[lo:hi]
        coords_np = np.ascontiguousarray(coords_np)
        self.n, self.d_L = coords_np.shape[0], workload.dims[-1]
        self.h = dhq.dhq_prepare(workload.dims, [torch.from_numpy(w).cuda() for w in weights],
                                 [torch.from_numpy(b).cuda() for b in biases], workload.omega0, workload.w_bits,
                                 workload.a_bits, workload.w_gran, workload.a_gran,
                                 rotation={"input": 0, "both": 1, "none": 2}[rotation],
                                 activation=dhq.DHQ_ACT_GABOR if gabor_s0 > 0 else dhq.DHQ_ACT_SINE, act_s0=gabor_s0)
        self.coords = torch.from_numpy(coords_np).cuda()
        self.out = torch.empty((self.n, self.d_L), dtype=torch.float32, device="cuda")
        self.coords_host = torch.from_numpy(coords_np).pin_memory()
        self.out_host = torch.empty((self.n, self.d_L), dtype=torch.float32).pin_memory()
        self.stream = torch.cuda.current_stream()
        # per-tensor scales frozen on the workload's grid (all ranks' blocks together); no-op per token
        if shard is not None:
            dhq.calibrate_sharded(self.h, self.coords, len(workload.dims) - 1, group=group)
        else:
            dhq.dhq_calibrate(self.h, self.coords)

    def warm(self, steps, e2e=True):
        for _ in range(steps):
            self.dhq.dhq_forward(self.h, self.coords, self.out)
            if e2e:
                self.dhq.dhq_forward_host(self.h, self.coords_host, self.out_host)
        self.torch.cuda.synchronize()
        if self.dhq.dhq_last_status(self.h) != 0:
            raise SystemExit("device-side wait timed out during warm-up")

    def timed(self, fn, steps, flush, barrier):
        torch = self.torch
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for a, b in evs:
            flush.fill_(1)
            a.record(self.stream)
            fn()
            b.record(self.stream)
        barrier()
        return sum(a.elapsed_time(b) for a, b in evs)   # ms

    def forward(self):
        self.dhq.dhq_forward(self.h, self.coords, self.out)

    def forward_host(self):
        self.dhq.dhq_forward_host(self.h, self.coords_host, self.out_host)

    def close(self):
        self.dhq.dhq_destroy(self.h)


def launch_clock(dhq, run):
    """SM clock inside a launch of this workload: three back-to-back launches of the observing
    instantiation of the fused kernel (no dump buffers: the same work as the timed kernel), which
    carries a cycle-counter / nanosecond-timer probe that the timed instantiations leave out."""
    try:
        for _ in range(3):
            dhq.dhq_forward_fused_debug(run.h, run.coords, run.out)
        return dhq.dhq_last_launch_clock(run.h)
    except Exception:
        return None, None


def packed_weight_bytes(dims):
    """Bytes of the prepared int8 weights a launch reads once (tensor-core images of the hidden and
    last layers, one word per feature for the first)."""
    w, hidden_matmuls = dims[1], len(dims) - 3
    return 4 * w + hidden_matmuls * w * w + 16 * w


def dram_traffic(workload, rotation, n):
    """DRAM bytes of one launch over n coordinates from the kept ncu counters: the captured launch's
    bytes beyond the weights grow with the coordinate count, the weights are read once."""
    entry = NCU_DRAM_BYTES.get((workload.name, rotation))
    if entry is None:
        return None
    captured, coords = entry
    fixed = min(packed_weight_bytes(workload.dims), captured)
    return fixed + (captured - fixed) * (n / coords)


def roofline_of(workload, rotation, n, ms_per_step, sm_max_mhz, sampled_mhz, fma_peak, kernel_mhz=None):
    """ALU roofline of one launch: algorithmic lane-ops over the CUDA-event duration, against (a) the
    derived peak SMs x fp32 lanes x max SM clock, (b) the same at the SM clock sampled during the
    timed steps, (c) the FMA loop's rate measured in this run."""
    laneops = alu_laneops_per_coord(workload.dims, rotations(rotation))
    if workload.a_bits == 32:      # fp32 datapaths: one fused multiply-add per weight and coordinate on the CUDA cores
        laneops = float(work_per_coord(workload.dims, rotations(rotation))[0])
    achieved = laneops * n / (ms_per_step * 1e-3) / 1e12
    peak = SM_COUNT * FP32_LANES_PER_SM * sm_max_mhz * 1e6 / 1e12
    r = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "Tlaneop/s", "frac": achieved / peak,
         "peak_source": "148 SMs x 128 fp32 lanes x max SM clock (derived from unit counts and clock)"}
    if sampled_mhz:
        r["frac_at_sampled_clock"] = achieved / (SM_COUNT * FP32_LANES_PER_SM * sampled_mhz * 1e6 / 1e12)
    if kernel_mhz:   # cycle counter over nanosecond timer inside a launch of the same work (launch_clock)
        r["frac_at_kernel_clock"] = achieved / (SM_COUNT * FP32_LANES_PER_SM * kernel_mhz * 1e6 / 1e12)
    if fma_peak:
        r["peak_measured_fma"] = fma_peak / 1e12
        r["frac_of_measured_fma"] = achieved / (fma_peak / 1e12)
    r["traffic"] = dram_traffic(workload, rotation, n)
    return r


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
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")   # > 126 MB of L2

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    run = Runner(dhq, workload, args.rotation, args.limit_coords, shard=(rank, world) if args.shard else None, gabor_s0=args.gabor_s0)
    n = run.n
    warmup = max(args.warmup, 3)
    run.warm(warmup)
    launches0 = dhq.dhq_launch_count(run.h)
    with ClockSampler(physical_gpu_index(local_rank)) as clocks:
        total_ms = run.timed(run.forward, args.steps, flush, barrier)
    launches = dhq.dhq_launch_count(run.h) - launches0
    kernel_mhz, kernel_ms = launch_clock(dhq, run)
    e2e_ms = run.timed(run.forward_host, args.steps, flush, barrier)
    status = dhq.dhq_last_status(run.h)

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], world, "cuda")
    ms_per_step = total_ms / args.steps
    coords_per_step = run.n_total if args.shard else n * world
    value = aggregate_throughput(coords_per_step, ms_per_step)
    e2e_value = aggregate_throughput(coords_per_step, e2e_ms / args.steps)

    if rank == 0:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        sm_max = float(peaks.get("sm_max_mhz", 1965.0))
        csum = clocks.summary()
        csum["sm_mhz_in_kernel"] = kernel_mhz
        csum["kernel_ms_in_kernel"] = kernel_ms
        try:
            fma_peak, _ = dhq.dhq_measure_pipe("ffma", 2000)
        except Exception:
            fma_peak = None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "strong" if args.shard else "weak", "vs_baseline": None,
            "dtype": "int8 (int32 accumulate, f32 epilogue)", "data": "synthetic",
            "config": config_of(workload, args, world),
            "clocks": csum,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": n * 8, "d2h_bytes_per_step": n * run.d_L * 4,
                    "ms_per_step": e2e_ms / args.steps,
                    "route": "dhq_forward_host on pinned host buffers: the kernel reads the coordinates and writes "
                             "the result over the host link through the buffers' device mapping, every step "
                             "(whole tiles by bulk copy where the width's kernel has that variant)"},
            "gpu_launches": launches,
            "roofline": roofline_of(workload, args.rotation, n, ms_per_step, sm_max, csum["sm_mhz"], fma_peak, kernel_mhz),
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
    run.close()

    # The other configurations, briefly, in the same process (one GPU, the default invocation only).
    if world == 1 and not args.no_per_config and args.limit_coords <= 0 and args.rotation == "input":
        per = {}
        for name in sorted(dhq_inputs.WORKLOADS):
            if name == workload.name:
                continue
            other = dhq_inputs.WORKLOADS[name]
            r = Runner(dhq, other, args.rotation)
            steps = max(10, min(args.steps, 100))
            r.warm(3, e2e=False)
            with ClockSampler(physical_gpu_index(local_rank)) as ck:
                ms = r.timed(r.forward, steps, flush, barrier) / steps
            st = dhq.dhq_last_status(r.h)
            k_mhz = launch_clock(dhq, r)[0]
            roof = roofline_of(other, args.rotation, r.n, ms, sm_max, ck.summary()["sm_mhz"], fma_peak, k_mhz)
            per[name] = {"coords_per_step": r.n, "steps": steps, "ms_per_step": ms, "value": r.n / (ms * 1e-3),
                         "roofline_frac": roof["frac"], "frac_of_measured_fma": roof.get("frac_of_measured_fma"),
                         "sm_mhz_in_kernel": k_mhz, "frac_at_kernel_clock": roof.get("frac_at_kernel_clock"),
                         "traffic": roof["traffic"], "device_status": st}
            r.close()
        line["per_config"] = per

    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            v, dt, cores, passes, desc = time_oracle(workload, 1, 1, rotations(args.rotation), min_seconds=10.0)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{desc}, {passes} pass(es) of {dt:.1f} s",
                                    "rotation": "O(n^2) product with the explicit Hadamard matrix (the definition)"}
            if args.rotation != "both":
                v2, dt2, _, passes2, _ = time_oracle(workload, 1, 1, rotations(args.rotation), min_seconds=5.0, variant="nlogn")
                line["cpu_baseline"]["nlogn_variant"] = {"value": v2, "unit": UNIT, "cores": cores,
                                                         "sample": f"same sample, {passes2} pass(es) of {dt2:.1f} s",
                                                         "rotation": "O(n log n) butterfly, bit-identical results"}
        print(json.dumps(line), flush=True)
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
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C5", choices=sorted(dhq_inputs.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--shard", action="store_true",
                    help="with N > 1 ranks: split the one grid over the ranks (strong scaling) instead of N replicas")
    ap.add_argument("--rotation", default="input", choices=["input", "none", "both"],
                    help="input = DHQ; none = the same path without the Hadamard rotation (uniform quantizer); "
                         "both = the two-sided transform of Eq. 4-5")
    ap.add_argument("--variant", default="w8a8", choices=["w8a8", "w8a32", "w32a32"],
                    help="datapath (Section I / Table 2 of the paper): the workload's fully quantized network, the same "
                         "with fp32 activations, or the plain fp32 network")
    ap.add_argument("--gabor-s0", type=float, default=0.0,
                    help="> 0: the wavelet activation sin(omega0 z) exp(-(s0 z)^2) instead of the sine (the WIRE reading)")
    ap.add_argument("--limit-coords", type=int, default=0,
                    help="use only the first N coordinates of the workload's grid (profiling captures)")
    ap.add_argument("--sweep", action="store_true", help="batch-size sweep 2^12..2^24 instead of the timed steps")
    ap.add_argument("--sweep-reps", type=int, default=20)
    args = ap.parse_args()
    workload = dhq_inputs.WORKLOADS[args.workload]
    if args.gabor_s0 > 0:
        args.no_per_config = True
        args.no_cpu_baseline = True
    if args.variant != "w8a8":
        import dataclasses
        workload = dataclasses.replace(workload, w_bits=32 if args.variant == "w32a32" else workload.w_bits, a_bits=32)
        args.no_per_config = True
        args.no_cpu_baseline = True
    if args.impl == "reference":
        run_reference(args, workload)
    elif args.sweep:
        run_sweep(args, workload)
    else:
        run_ours(args, workload)


if __name__ == "__main__":
    main()

"""bench.py's bookkeeping without a GPU: algorithmic work per coordinate, the roofline object, the
traffic scaling, the shared `config` object and the reference arm's JSON line."""
import json
import os
import subprocess
import sys
import types

import dhq_inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_algorithmic_work_per_coordinate_matches_the_hand_counts():
    # lane-ops per coordinate: hidden vectors x width x (7 + log2 width)
    assert bench.alu_laneops_per_coord((2, 256, 256, 256, 3)) == 3 * 256 * 15 == 11520
    assert bench.alu_laneops_per_coord((2, 512, 512, 512, 512, 3)) == 4 * 512 * 16 == 32768
    assert bench.alu_laneops_per_coord((2, 256, 256, 256, 3), rotate=0) == 3 * 256 * 7
    macs, sines, _ = bench.work_per_coord((2, 256, 256, 256, 3))
    assert macs == 4 * 256 + 2 * 256 * 256 + 4 * 256 == 133120 and sines == 768
    assert bench.work_per_coord((2, 512, 512, 512, 512, 3))[0] == 790528


def test_roofline_object_and_traffic_scaling():
    w = dhq_inputs.WORKLOADS["C5"]
    r = bench.roofline_of(w, "input", w.n, 7.65, 1965.0, 1965.0, 35.5e12, 1900.0)
    assert r["bound"] == "alu" and r["unit"] == "Tlaneop/s"
    assert abs(r["peak"] - 148 * 128 * 1.965e9 / 1e12) < 1e-9
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-12 and 0.4 < r["frac"] < 0.6
    assert r["frac_at_kernel_clock"] > r["frac"] and abs(r["frac_at_sampled_clock"] - r["frac"]) < 1e-12
    # traffic: the captured launch's bytes beyond the weights grow with the coordinate count
    captured, coords = bench.NCU_DRAM_BYTES[("C5", "input")]
    weights = bench.packed_weight_bytes(w.dims)
    assert weights == 4 * 512 + 3 * 512 * 512 + 16 * 512
    assert bench.dram_traffic(w, "input", coords) == captured
    assert abs(bench.dram_traffic(w, "input", w.n) - (weights + (captured - weights) * w.n / coords)) < 1
    assert bench.dram_traffic(w, "none", w.n) is None               # no capture for that variant: null


def test_config_object_is_the_same_for_both_arms_and_reference_line_is_complete():
    args = types.SimpleNamespace(shard=False, limit_coords=0, rotation="input", variant="w8a8", gabor_s0=0.0)
    w = dhq_inputs.WORKLOADS["C5"]
    cfg = bench.config_of(w, args, 1)
    assert cfg["workload"] == "C5" and cfg["coords_per_step"] == 4194304 and "model" not in cfg
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C1", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["config"] == bench.config_of(dhq_inputs.WORKLOADS["C1"], args, 1)
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": bench.UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["higher_is_better"] is True and line["vs_baseline"] is None and line["gpu_launches"] == 0

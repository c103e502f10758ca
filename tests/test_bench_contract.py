"""The benchmark's command line and JSON line, as far as they can be checked without a GPU: the
reference arm (the CPU oracle timed on a bounded sample) and the byte counts behind the roofline."""
import json
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def _bench(*args, env=None):
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), *args], capture_output=True, text=True,
                         timeout=600, env=env, check=True)
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    return lines


def test_reference_arm_times_exactly_k_steps_on_the_benchmark_config():
    lines = _bench("--impl", "reference", "--steps", "3", "--warmup", "1", "--log2d", "14", "--workers", "4")
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["steps"] == 3 and j["warmup"] == 1 and j["n_gpus"] == 1
    assert j["metric"] == "fused IntSGD step throughput" and j["unit"] == "gradient elements/s"
    assert j["higher_is_better"] is True and j["vs_baseline"] is None and j["data"] == "synthetic"
    assert j["config"]["d"] == 1 << 14 and j["config"]["n_workers"] == 4 and "workload" in j["config"]
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] == 1
    assert j["cpu_baseline"]["value"] == j["value"] and "2^14" in j["cpu_baseline"]["sample"]
    assert j["e2e"] == {"value": j["value"], "unit": j["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert j["value"] > 0 and abs(j["ms_per_step"] * 1e-3 * j["value"] - 4 * (1 << 14)) < 1e-3 * 4 * (1 << 14)


def test_reference_arm_runs_on_rank_zero_only():
    import os
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    assert _bench("--impl", "reference", "--steps", "1", "--warmup", "0", "--log2d", "12", env=env) == []


def test_algorithmic_bytes_per_coordinate():
    sys.path.insert(0, str(ROOT))
    import bench
    f = bench.algorithmic_bytes_per_coordinate
    assert f(16, 4, 4, "fused") == 76            # n gradient reads + x read + x write + aggregate write
    assert f(8, 2, 1, "fused") == 28             # bf16 gradients
    assert f(16, 4, 4, "two_kernel") == 76 + 128  # + n payload writes + n payload reads
    assert f(16, 4, 1, "two_kernel") == 76 + 32
    assert f(16, 4, 4, "fused", "diana") == 12 * 16 + 20
    assert f(16, 4, 4, "fused", "heuristic") == 2 * 64 + 12
    assert f(16, 4, 4, "fused", "blocks") == 76


def test_counter_table_and_multiply_counts():
    """The ncu counter table is keyed by shape, scales with d, and goes silent for anything it was not taken on."""
    sys.path.insert(0, str(ROOT))
    import argparse
    import bench
    base = dict(kind="intsgd", mode="fused", grad="f32", payload="int32", workers=16, rounding="random",
                num_blocks=62, num_bits=16)
    args = argparse.Namespace(**base)
    assert bench.shape_key(args) == "intsgd/fused/f32/int32/n16"
    fresh = bench.kernel_sources_hash() == bench.NCU_COUNTERS["sources_sha256"]
    t = bench.traffic_per_launch(args, 1 << 26)
    if fresh:   # counters taken on these very sources: traffic is within a few per cent of the algorithmic bytes
        assert t is not None and abs(t / (76 * (1 << 26)) - 1.0) < 0.05
        assert bench.traffic_per_launch(args, 1 << 28) == 4 * t
    else:       # the kernels changed since the capture: no stale figure is reported
        assert t is None
    for other in (dict(rounding="compare"), dict(workers=5), dict(kind="blocks", num_blocks=7)):
        assert bench.traffic_per_launch(argparse.Namespace(**{**base, **other}), 1 << 26) is None
    for key, v in bench.NCU_COUNTERS["shapes"].items():
        kind, mode, grad, payload, n = key.split("/")
        n = int(n[1:])
        gb, pb = (2 if grad == "bf16" else 4), (1 if payload == "int8" else 4)
        alg = bench.algorithmic_bytes_per_coordinate(n, gb, pb, mode, kind)
        # never above the algorithmic bytes (no stream is read twice); below them by what is still in L2 at kernel end
        assert 0.8 < v["bytes_per_coordinate"] / alg < 1.02, key
    # 32x32->64-bit products of the random stream per worker unit on the pipelined kernels
    f = bench.wide_multiplies_per_worker_unit
    assert f(argparse.Namespace(rounding="random"), 16) == 16.125 and f(argparse.Namespace(rounding="compare"), 8) == 16.25
    assert f(argparse.Namespace(rounding="random16"), 16) == 8.0625 and f(argparse.Namespace(rounding="nearest"), 16) == 0.0

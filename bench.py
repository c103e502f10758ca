#!/usr/bin/env python
"""Benchmark of the fused IntSGD step (gradient elements/s and HBM roofline fraction).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one whole IntSGD iteration -- scale, encode, integer sum, decode, update, next-norm --
over n workers' gradients of length d that are already in device memory (`value`), and the same
step through the host-buffer entry point with the copies inside the timed region (`e2e`).
Workload: the largest row of the large-model bucket sweep (d = 2^28 fp32 N(0, 1e-3^2), n = 16 workers,
16 GiB of gradients, int32 aggregate, fused single-pass path).  Two timings are printed: the K steps the
command line asks for (a burst when K is small), and a segment of at least two seconds of back-to-back
steps during which the board settles at its power cap (`roofline.sustained`), with the SM clock sampled
through NVML across both.  With N > 1 (torchrun) every rank runs an independent replica on its own
GPU: the path has no exchange step on one node, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "fused IntSGD step throughput"
UNIT = "gradient elements/s"
HBM_FALLBACK_GBS = 6650.0

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) and executed warp instructions of the kernels of one
# step, from ncu captures of the small case (d = 2^24) of each shape this script can time; both grow in proportion
# to d, so a launch at another d is the per-coordinate figure times d.  Valid for the kernel sources with this hash:
# any change to them makes `roofline.traffic` null until the counters are taken again.
NCU_COUNTERS = {
    "sources_sha256": "6b815c37c800d1efc3a2d0b090812e2b30aafeda1886355f944b9f040bdb2dee",
    "captured_log2d": 24,
    # key: kind/mode/grad/payload/n -> bytes per coordinate, warp instructions per coordinate (the vector kernels of a
    # step: fused; encode + aggregate; IntDIANA; block-wise (62 blocks); profiling pass + fused (16 bits))
    "shapes": {
        "intsgd/fused/f32/int32/n16": {"bytes_per_coordinate": 75.411, "warp_instructions_per_coordinate": 8.1028},
        "intsgd/fused/f32/int32/n8": {"bytes_per_coordinate": 42.901, "warp_instructions_per_coordinate": 4.3431},
        "intsgd/fused/f32/int32/n2": {"bytes_per_coordinate": 16.985, "warp_instructions_per_coordinate": 2.0074},
        "intsgd/fused/bf16/int8/n8": {"bytes_per_coordinate": 25.925, "warp_instructions_per_coordinate": 4.4393},
        "intsgd/two_kernel/f32/int32/n16": {"bytes_per_coordinate": 197.976, "warp_instructions_per_coordinate": 9.8018},
        "intsgd/two_kernel/f32/int8/n16": {"bytes_per_coordinate": 103.567, "warp_instructions_per_coordinate": 10.7396},
        "intsgd/two_kernel/bf16/int8/n8": {"bytes_per_coordinate": 38.545, "warp_instructions_per_coordinate": 5.7434},
        "diana/fused/f32/int32/n16": {"bytes_per_coordinate": 209.329, "warp_instructions_per_coordinate": 15.8897},
        "blocks/fused/f32/int32/n16": {"bytes_per_coordinate": 75.49, "warp_instructions_per_coordinate": 9.2365},
        "heuristic/fused/f32/int32/n16": {"bytes_per_coordinate": 139.595, "warp_instructions_per_coordinate": 9.1699},
    },
}


def kernel_sources_hash():
    import hashlib
    h = hashlib.sha256()
    for f in sorted((ROOT / "paper_2102_08374_b200" / "csrc").glob("*")):
        h.update(f.name.encode())
        h.update(f.read_bytes())
    return h.hexdigest()


def shape_key(args):
    return f"{args.kind}/{args.mode}/{args.grad}/{args.payload}/n{args.workers}"


def captured_counters(args):
    """The ncu figures of this shape (default random stream only), or None."""
    if args.rounding != "random" or kernel_sources_hash() != NCU_COUNTERS["sources_sha256"]:
        return None
    if args.kind == "blocks" and args.num_blocks != 62:
        return None
    if args.kind == "heuristic" and args.num_bits != 16:
        return None
    return NCU_COUNTERS["shapes"].get(shape_key(args))


def traffic_per_launch(args, d):
    """Measured DRAM bytes of one step's kernels, scaled to d (traffic is proportional to d), or None."""
    c = captured_counters(args)
    return None if c is None else c["bytes_per_coordinate"] * d


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=50)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--log2d", type=int, default=28)
    p.add_argument("--workers", type=int, default=16)
    p.add_argument("--payload", default="int32", choices=["int32", "int8"])
    p.add_argument("--grad", default="f32", choices=["f32", "bf16"])
    p.add_argument("--mode", default="fused", choices=["fused", "two_kernel"])
    p.add_argument("--kind", default="intsgd", choices=["intsgd", "diana", "heuristic", "blocks"],
                   help="which step is timed: Algorithm 1 (default, the headline), the IntDIANA step (Algorithm 3), "
                        "the heuristic SwitchML-style step (profiling pass + fused pass) or block-wise scales (Algorithm 2)")
    p.add_argument("--num-bits", type=int, default=16, help="--kind heuristic: bits of the heuristic rule")
    p.add_argument("--num-blocks", type=int, default=62, help="--kind blocks: equal contiguous blocks")
    p.add_argument("--rounding", default="random", choices=["random", "nearest", "random16", "compare"],
                   help="random16 = the optional 16-bit draw stream; compare = Int(t) drawn by comparing a 24-bit "
                        "uniform with the fractional part (both: a different random stream; not the default)")
    p.add_argument("--eta", type=float, default=0.1)
    p.add_argument("--e2e-steps", type=int, default=3)
    p.add_argument("--sustain-seconds", type=float, default=2.0,
                   help="length of the second timed segment (steps back to back, SM clock sampled); 0 = skip")
    p.add_argument("--cpu-sample-log2", type=int, default=24,
                   help="coordinates of the oracle sample (all workers), as a power of two")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-cpu-all-cores", action="store_true", help="skip the all-cores leg of the CPU baseline")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--no-variants", action="store_true", help="skip the short runs of the other rounding modes")
    p.add_argument("--threads", type=int, default=0)
    p.add_argument("--blocks-per-sm", type=int, default=0)
    return p.parse_args()


# ------------------------------------------------------------------------------------------
def measured_hbm_peak():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        try:
            return float(json.loads(f.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return HBM_FALLBACK_GBS, "fallback"


class ClockSampler:
    """Samples SM clock, power and clock-event reasons while timed regions run: NVML from a thread (a few
    milliseconds apart, so that a region of tens of milliseconds is covered), else nvidia-smi every 50 ms.
    Reading only; no setting of the GPU is touched."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, uuid: str | None = None, period_s: float = 0.004):
        self.index, self.uuid, self.period = index, uuid, period_s
        self.samples = []      # (time, sm_mhz, max_mhz, watts, [reasons])
        self.proc = self.thread = None
        self.stop_flag = threading.Event()
        self.source = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = None
            if self.uuid:
                for cand in (self.uuid, "GPU-" + self.uuid):
                    try:
                        h = pynvml.nvmlDeviceGetHandleByUUID(cand.encode() if isinstance(cand, str) else cand)
                        break
                    except Exception:
                        h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            mx = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                pynvml.nvmlDeviceGetCurrentClocksThrottleReasons
            float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))    # fails here if NVML cannot be read

            def loop():
                while not self.stop_flag.is_set():
                    try:
                        mhz = float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                        watts = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
                        mask = int(reasons_fn(h))
                        self.samples.append((time.time(), mhz, mx, watts, [n for b, n in self.REASONS.items() if mask & b]))
                    except Exception:
                        pass
                    time.sleep(self.period)

            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            self.source = "nvml"
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
            self.source = "nvidia-smi"
        except Exception:
            self.proc = None

    def _pump(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            try:
                self.samples.append((time.time(), float(parts[0]), float(parts[1]), float(parts[2]),
                                     [n for n, v in zip(names, parts[3:7]) if v.lower().startswith("active")]))
            except (ValueError, IndexError):
                continue

    def stop(self):
        self.stop_flag.set()
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)

    def window(self, t0, t1):
        """Summary of the samples taken between two wall-clock times."""
        rows = [r for r in self.samples if t0 <= r[0] <= t1]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "power_w_max": None, "reasons": [], "samples": 0, "source": self.source}
        reasons = sorted({n for r in rows for n in r[4]})
        return {"sm_mhz": statistics.median(r[1] for r in rows), "sm_max_mhz": max(r[2] for r in rows),
                "sm_mhz_min": min(r[1] for r in rows), "power_w_max": max(r[3] for r in rows), "reasons": reasons,
                "samples": len(rows), "source": self.source}


def algorithmic_bytes_per_coordinate(n, grad_bytes, payload_bytes, mode, kind="intsgd"):
    """Bytes that must cross HBM per coordinate: n gradient reads, x read + write, aggregate write
    (fused); plus n payload writes and n payload reads on the two-kernel path.  IntDIANA also reads and
    writes the n local shifts and the global shift; the heuristic step reads every gradient twice."""
    base = n * grad_bytes + 12
    if mode == "two_kernel":
        base += 2 * n * payload_bytes
    if kind == "diana":
        base += 8 * n + 8
    if kind == "heuristic":
        base += n * grad_bytes
    return base


def wide_multiplies_per_worker_unit(args, n):
    """32x32->64-bit multiplies of Philox4x32-10 per worker unit (4 gradient elements of one worker) on the path
    `bench.py` times.  The pipelined kernels keep a thread on the same units for all workers: the unit's half of
    rounds 1-2 (2 multiplies) is shared by the n workers, the worker's half comes from a table, rounds 3-10 cost
    16.  With 16-bit draws one block serves two units.  Deterministic rounding draws nothing."""
    if args.rounding == "nearest":
        return 0.0
    per = 16.0 + 2.0 / n
    return per / 2 if args.rounding == "random16" else per


# ------------------------------------------------------------------------------------------
def oracle_sample_throughput(n, d, sample_log2, grad_dtype, payload, rounding, seed=77):
    """Time the CPU oracle, as it stands, on one step over the first 2^sample_log2 coordinates of
    all n workers.  Returns (elements/s, seconds, description)."""
    import numpy as np
    import oracle
    from paper_2102_08374_b200 import synth
    w = min(d, 1 << sample_log2)
    grads = [synth.bucket_gradient(i, w) for i in range(n)]
    if grad_dtype == "bf16":
        grads = [synth.to_bf16_bits(g) for g in grads]
    x = synth.iterate(w)
    pd = oracle.PAYLOAD_I8 if payload == "int8" else oracle.PAYLOAD_I32
    rd = {"nearest": oracle.ROUND_NEAREST, "random16": oracle.ROUND_RANDOM16, "compare": oracle.ROUND_RANDOM_COMPARE}.get(rounding, oracle.ROUND_RANDOM)
    oracle.step_window([g[:1024] for g in grads], x[:1024].copy(), np.float32(700.0), np.float32(1e-5), step=1,
                       seed=seed, payload_dtype=pd, rounding=rd)     # load the library, touch the code
    t = time.perf_counter()
    oracle.step_window(grads, x, np.float32(700.0), np.float32(1e-5), step=1, seed=seed, payload_dtype=pd, rounding=rd)
    dt = time.perf_counter() - t
    return n * w / dt, dt, f"one step on the first 2^{sample_log2} coordinates of all {n} workers ({n * w} elements)"


def _oracle_window_task(task):
    """Runs in a spawned worker process: the unchanged oracle on one coordinate window of the sample.
    Returns the wall-clock interval of the timed call (inputs are drawn before it starts)."""
    import numpy as np
    import oracle
    from paper_2102_08374_b200 import synth
    n, j0, count, grad_dtype, payload, rounding, seed = task
    grads = [synth.bucket_gradient(i, count, seed_base=7000 + 64 * (j0 // max(count, 1))) for i in range(n)]
    if grad_dtype == "bf16":
        grads = [synth.to_bf16_bits(g) for g in grads]
    x = synth.iterate(count, seed=8000 + j0 // max(count, 1))
    pd = oracle.PAYLOAD_I8 if payload == "int8" else oracle.PAYLOAD_I32
    rd = {"nearest": oracle.ROUND_NEAREST, "random16": oracle.ROUND_RANDOM16,
          "compare": oracle.ROUND_RANDOM_COMPARE}.get(rounding, oracle.ROUND_RANDOM)
    oracle.step_window([g[:256] for g in grads], x[:256].copy(), np.float32(700.0), np.float32(1e-5), step=1,
                       seed=seed, j0=j0, payload_dtype=pd, rounding=rd)    # load the library, touch the code
    t0 = time.time()
    oracle.step_window(grads, x, np.float32(700.0), np.float32(1e-5), step=1, seed=seed, j0=j0, payload_dtype=pd,
                       rounding=rd)
    return t0, time.time()


def oracle_all_cores_throughput(n, d, sample_log2, grad_dtype, payload, rounding, seed=77):
    """The same oracle on all host cores: the sample's coordinates are cut into one window per core, and
    each window is stepped by an unchanged single-threaded oracle in its own (spawned) process -- valid
    because the random stream is addressed by (seed, step, worker, coordinate).  Returns
    (elements/s, cores, description); the time runs from the first window's start to the last one's end."""
    import multiprocessing as mp
    cores = max(1, min(os.cpu_count() or 1, 64))
    w = min(d, 1 << sample_log2)
    count = max(w // cores // 4 * 4, 4)
    tasks = [(n, k * count, count, grad_dtype, payload, rounding, seed) for k in range(cores)]
    pool = mp.get_context("spawn").Pool(cores)
    try:
        spans = pool.map_async(_oracle_window_task, tasks, chunksize=1).get(timeout=180)
    finally:
        pool.terminate()
        pool.join()
    seconds = max(t1 for _, t1 in spans) - min(t0 for t0, _ in spans)
    return n * count * cores / seconds, cores, (f"{cores} windows of {count} coordinates x {n} workers, one process "
                                                f"per core ({n * count * cores} elements, {seconds:.2f} s)")


def run_reference(args):
    """The reference arm: the CPU oracle as it stands, single-threaded, W untimed and exactly K timed steps,
    each over a window of the workload sized so that the whole run takes about a minute or two."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2102_08374_b200 import synth
    n, d = args.workers, 1 << args.log2d
    K, W = max(args.steps, 1), max(args.warmup, 0)
    # about 1e9 gradient elements in all (the oracle does 1-2e7 per second and core), a power of two per step
    per_step = 1.0e9 / ((K + W) * n)
    sample_log2 = max(10, min(22, args.log2d, int(math.floor(math.log2(max(per_step, 1.0))))))
    w = 1 << sample_log2
    grads = [synth.bucket_gradient(i, w) for i in range(n)]
    if args.grad == "bf16":
        grads = [synth.to_bf16_bits(g) for g in grads]
    x = synth.iterate(w)
    pd = oracle.PAYLOAD_I8 if args.payload == "int8" else oracle.PAYLOAD_I32
    rd = {"nearest": oracle.ROUND_NEAREST, "random16": oracle.ROUND_RANDOM16,
          "compare": oracle.ROUND_RANDOM_COMPARE}.get(args.rounding, oracle.ROUND_RANDOM)

    def one_step(k):
        oracle.step_window(grads, x, np.float32(700.0), np.float32(1e-5), step=k, seed=77, payload_dtype=pd, rounding=rd)

    for k in range(W):
        one_step(1 + k)
    t0 = time.perf_counter()
    for k in range(K):
        one_step(1 + W + k)
    seconds = time.perf_counter() - t0
    value = n * w * K / seconds
    desc = f"each step covers the first 2^{sample_log2} coordinates of all {n} workers ({n * w} elements)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": K, "warmup": W, "ms_per_step": 1e3 * seconds / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(args):
    kind = {"intsgd": "", "diana": ", IntDIANA step", "heuristic": f", heuristic scale with {args.num_bits} bits",
            "blocks": f", block-wise scales over {args.num_blocks} blocks"}[args.kind]
    row = " (the largest row of the bucket sweep)" if (args.log2d, args.workers) == (28, 16) else ""
    return {"workload": f"large-model bucket sweep{row}: d=2^{args.log2d} {args.grad} N(0,1e-3^2), n={args.workers} workers, "
                        f"{args.payload} wire, {args.mode} path, {args.rounding} rounding{kind}",
            "d": 1 << args.log2d, "n_workers": args.workers, "grad_dtype": args.grad, "payload": args.payload,
            "mode": args.mode, "rounding": args.rounding,
            "l2": "inputs larger than L2 (gradients alone are n*d*4 bytes); no flush between iterations"}


# ------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2102_08374_b200 as pkg
    from paper_2102_08374_b200 import replicas, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    n, d = args.workers, 1 << args.log2d
    grad_dtype = pkg.GRAD_BF16 if args.grad == "bf16" else pkg.GRAD_F32
    payload_dtype = pkg.PAYLOAD_I8 if args.payload == "int8" else pkg.PAYLOAD_I32
    rounding = {"nearest": pkg.ROUND_NEAREST, "random16": pkg.ROUND_RANDOM16, "compare": pkg.ROUND_RANDOM_COMPARE}.get(args.rounding, pkg.ROUND_RANDOM)
    mode = pkg.MODE_TWO_KERNEL if args.mode == "two_kernel" else pkg.MODE_FUSED
    gb, pb = (2 if args.grad == "bf16" else 4), (1 if args.payload == "int8" else 4)

    grads = synth.bucket_gradients_device(n, d, device, seed_base=replicas.rank_seed_base(rank),
                                          dtype=torch.bfloat16 if args.grad == "bf16" else None)
    x = synth.iterate_device(d, device)
    agg = torch.empty(d, dtype=torch.int32, device=device)
    scratch = None
    if mode == pkg.MODE_TWO_KERNEL:
        scratch = [torch.empty(d, dtype=torch.int8 if pb == 1 else torch.int32, device=device) for _ in range(n)]
    lib = pkg.IntSGD(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding, seed=2102_08374,
                     device=local_rank)
    lib.intsgd_set_launch(args.threads, args.blocks_per_sm)
    stream = torch.cuda.current_stream().cuda_stream

    h_local = h_global = None
    if args.kind == "diana":
        h_local = [torch.zeros(d, dtype=torch.float32, device=device) for _ in range(n)]
        h_global = torch.zeros(d, dtype=torch.float32, device=device)
    if args.kind == "blocks":
        B = max(1, min(args.num_blocks, d))
        lib.intsgd_set_blocks([(d * b) // B for b in range(B)] + [d])
    if args.kind != "intsgd" and mode != pkg.MODE_FUSED:
        raise SystemExit("--kind diana / heuristic / blocks run the fused path only")

    def step(k):
        if k > 0 and args.kind == "diana":
            lib.intsgd_diana_step(grads, h_local, h_global, x, agg, eta_k=args.eta, stream=stream)
        elif k > 0 and args.kind == "heuristic":
            lib.intsgd_heuristic_step(grads, x, agg, eta_k=args.eta, num_bits=args.num_bits, stream=stream)
        else:
            lib.intsgd_step(grads, x, agg, eta_k=args.eta, mode=pkg.MODE_EXACT if k == 0 else mode,
                            payload_scratch=scratch, stream=stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(run_step, count, per_step):
        """`count` steps between two CUDA events on the launching stream (plus one event per step when
        `per_step`), synchronised on both sides.  Returns (total ms, per-step ms or None, wall t0, wall t1)."""
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(count + 1 if per_step else 2)]
        barrier()
        t0 = time.time()
        ev[0].record()
        for k in range(count):
            run_step(k)
            if per_step:
                ev[k + 1].record()
        if not per_step:
            ev[1].record()
        torch.cuda.synchronize()
        t1 = time.time()
        each = [ev[k].elapsed_time(ev[k + 1]) for k in range(count)] if per_step else None
        return ev[0].elapsed_time(ev[-1]), each, t0, t1

    sms = torch.cuda.get_device_properties(device).multi_processor_count
    bytes_per_launch = algorithmic_bytes_per_coordinate(n, gb, pb, args.mode, args.kind) * d
    peak, peak_kind = measured_hbm_peak()

    def sustained_segment(run_step, ms_guess, seconds):
        """At least `seconds` of steps back to back (no event between steps), with the clock sampled across it."""
        count = max(20, int(math.ceil(seconds * 1e3 / max(ms_guess, 1e-3))))
        ms, _, t0, t1 = timed(run_step, count, per_step=False)
        ck = sampler.window(t0, t1)
        per = ms / count
        out = {"steps": count, "seconds": ms * 1e-3, "ms_per_step": per, "achieved": bytes_per_launch / (per * 1e-3) / 1e9,
               "frac": bytes_per_launch / (per * 1e-3) / 1e9 / peak, "sm_mhz_median": ck["sm_mhz"],
               "sm_mhz_min": ck.get("sm_mhz_min"), "power_w_max": ck["power_w_max"], "reasons": ck["reasons"],
               "samples": ck["samples"]}
        if ck["sm_mhz"]:
            out["sm_clocks_per_worker_unit"] = per * 1e-3 * ck["sm_mhz"] * 1e6 * sms / (n * d / 4)
        return out, count

    # step 0 is the exact first communication; then W warm-up steps; then K timed steps; then the sustained segment
    uuid = None
    try:
        uuid = str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        pass
    sampler = ClockSampler(local_rank, uuid)
    sampler.start()
    step(0)
    W = max(args.warmup, 3)
    for k in range(1, 1 + W):
        step(k)
    barrier()
    time.sleep(0.3)
    K = args.steps
    launches0 = lib.intsgd_launch_count()
    total_ms, per_step_ms, t_wall0, t_wall1 = timed(lambda k: step(1000 + k), K, per_step=True)
    launches = lib.intsgd_launch_count() - launches0
    clocks = sampler.window(t_wall0, t_wall1)
    applied = 1 + W + K
    sustained = None
    if args.sustain_seconds > 0:
        sustained, count = sustained_segment(lambda k: step(5000 + k), total_ms / K, args.sustain_seconds)
        applied += count
    st = lib.intsgd_get_stats()   # raises if a step was refused (scale not finite) or a bounded wait expired
    if st["step"] != applied:
        raise SystemExit(f"bench.py: {st['step']} steps were applied, {applied} were enqueued: the timing is void")
    total_ms = replicas.max_over_ranks(dist, total_ms, device)
    value = world * n * d * K / (total_ms * 1e-3)
    avg_ms = statistics.mean(per_step_ms)
    achieved = bytes_per_launch / (avg_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic_per_launch(args, d), "peak_source": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / 8000.0,
                "algorithmic_bytes_per_launch": bytes_per_launch, "kernel_ms_avg": avg_ms,
                "kernel_ms_median": statistics.median(per_step_ms),
                "note": "per-step CUDA-event time of the K timed steps (one-thread scale kernel + the vector kernel(s)); "
                        "`sustained` is the same step over a segment long enough for the board to settle at its power cap",
                "sustained": sustained}
    if clocks.get("sm_mhz"):
        roofline["sm_clocks_per_worker_unit"] = avg_ms * 1e-3 * clocks["sm_mhz"] * 1e6 * sms / (n * d / 4)
    counters = captured_counters(args)
    if counters is not None:
        roofline["traffic_over_algorithmic"] = counters["bytes_per_coordinate"] * d / bytes_per_launch
        roofline["thread_instructions_per_element"] = counters["warp_instructions_per_coordinate"] * 32 / n

    # ---- second limit: the 32x32->64-bit multiplies of Philox4x32-10, against their rate measured alone, and the
    # issue model that follows from it (on B200 nothing issues while a wide multiply does: times add up) ----
    mults = wide_multiplies_per_worker_unit(args, n)
    if mults > 0 and world == 1:
        def philox_alone(extra):
            """Scheduler cycles one warp spends per Philox block (rounds 3-10) in the register-only kernel, with
            `extra` independent fp32 additions per block; the SM clock is sampled while it runs."""
            lib.intsgd_selftest_philox_rate(256, extra, stream=stream)       # loads the kernel
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            nblocks, t0 = 0, time.time()
            ev0.record()
            for _ in range(6):
                nblocks += lib.intsgd_selftest_philox_rate(1 << 14, extra, stream=stream)
            ev1.record()
            torch.cuda.synchronize()
            ms, ck = ev0.elapsed_time(ev1), sampler.window(t0, time.time())
            if not ck["sm_mhz"]:
                return None, None, ms, None
            clocks_total = ms * 1e-3 * ck["sm_mhz"] * 1e6 * sms
            return clocks_total * 4 / (nblocks / 32), 16.0 * nblocks / clocks_total, ms, ck["sm_mhz"]

        cyc0, per_clock_alone, alone_ms, alone_mhz = philox_alone(0)
        cyc32 = philox_alone(32)[0]
        if cyc0 is not None:
            def per_clock(ms, mhz):
                return mults * (n * d / 4) / (ms * 1e-3 * mhz * 1e6 * sms)

            co = {"bound": "alu", "unit": "32x32->64-bit products per SM clock and SM",
                  "peak": per_clock_alone, "multiplies_per_worker_unit": mults,
                  "peak_source": "rounds 3-10 of Philox4x32-10 alone (register-only kernel, 512 threads per SM, two chains "
                                 f"per thread), {alone_ms:.0f} ms at {alone_mhz:.0f} MHz"}
            if clocks.get("sm_mhz"):
                co["achieved"] = per_clock(avg_ms, clocks["sm_mhz"])
                co["frac"] = co["achieved"] / per_clock_alone
            if sustained and sustained.get("sm_mhz_median"):
                co["sustained_achieved"] = per_clock(sustained["ms_per_step"], sustained["sm_mhz_median"])
                co["sustained_frac"] = co["sustained_achieved"] / per_clock_alone
            if cyc32 is not None and counters is not None:
                # Issue model: a warp's step time on its scheduler = Philox blocks at their measured cost + every other
                # executed instruction at the measured cost of one more independent instruction (they do not overlap).
                other = (cyc32 - cyc0) / 32.0
                instr = counters["warp_instructions_per_coordinate"] * 128.0 / n      # per worker unit of a warp
                philox_instr = 34.0 * mults / 16.0                                    # 16 multiplies + 18 logic ops per block
                predicted = cyc0 * mults / 16.0 + (instr - philox_instr) * other
                model = {"cycles_per_warp_philox_block": cyc0, "cycles_per_other_instruction": other,
                         "warp_instructions_per_worker_unit": instr, "predicted_cycles_per_worker_unit": predicted,
                         "note": "scheduler cycles per worker unit of a warp (32 units x 4 elements of one worker); "
                                 "frac = predicted / measured"}
                per_wuw = lambda ms, mhz: ms * 1e-3 * mhz * 1e6 * sms * 4 / (n * d / 128.0)
                if clocks.get("sm_mhz"):
                    model["measured_cycles_per_worker_unit"] = per_wuw(avg_ms, clocks["sm_mhz"])
                    model["frac"] = predicted / model["measured_cycles_per_worker_unit"]
                if sustained and sustained.get("sm_mhz_median"):
                    model["sustained_frac"] = predicted / per_wuw(sustained["ms_per_step"], sustained["sm_mhz_median"])
                co["issue_model"] = model
            roofline["co_limit"] = co

    # ---- the other rounding modes on the same buffers (context for the headline; 1 GPU only): a burst each, and the
    # comparison-form draw (the first reading of how Int(t) is drawn) through the same sustained segment ----
    variants = None
    if world == 1 and not args.no_variants and mode == pkg.MODE_FUSED and args.kind == "intsgd":
        variants = []
        names = {"random": pkg.ROUND_RANDOM, "compare": pkg.ROUND_RANDOM_COMPARE, "random16": pkg.ROUND_RANDOM16,
                 "nearest": pkg.ROUND_NEAREST}
        for name, rd in names.items():
            time.sleep(0.5)
            with pkg.IntSGD(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rd, seed=1, device=local_rank) as vlib:
                vstep = lambda k: vlib.intsgd_step(grads, x, agg, eta_k=args.eta, mode=mode, stream=stream)
                vlib.intsgd_step(grads, x, agg, eta_k=args.eta, mode=pkg.MODE_EXACT, stream=stream)
                for _ in range(3):
                    vstep(0)
                _, each, _, _ = timed(vstep, 30, per_step=True)
                ms = statistics.median(each)
                entry = {"rounding": name, "burst_ms_median_of_30": ms, "hbm_frac": bytes_per_launch / (ms * 1e-3) / 1e9 / peak}
                if name == "compare" and args.sustain_seconds > 0:
                    entry["sustained"], _ = sustained_segment(vstep, ms, args.sustain_seconds)
            variants.append(entry)

    # ---- end to end through the host-buffer entry point (rank-local; max over ranks) ----
    e2e = None
    if not args.no_e2e and mode == pkg.MODE_FUSED and args.kind == "intsgd":
        hg = [torch.empty(d, dtype=g.dtype, pin_memory=True) for g in grads]
        for h, g in zip(hg, grads):
            h.copy_(g)
        hx = torch.empty(d, dtype=torch.float32, pin_memory=True)
        hx.copy_(x)
        hagg = torch.empty(d, dtype=torch.int32, pin_memory=True)
        lib.intsgd_step_host(hg, hx, hagg, eta_k=args.eta, mode=mode, stream=stream)      # allocates staging
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record()
        for _ in range(args.e2e_steps):
            lib.intsgd_step_host(hg, hx, hagg, eta_k=args.eta, mode=mode, stream=stream)
        ev1.record()
        torch.cuda.synchronize()
        e2e_ms = ev0.elapsed_time(ev1)
        e2e_ms = replicas.max_over_ranks(dist, e2e_ms, device)
        e2e = {"value": world * n * d * args.e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": n * d * gb + d * 4, "d2h_bytes_per_step": d * 8,
               "steps": args.e2e_steps, "ms_per_step": e2e_ms / args.e2e_steps,
               "call": "intsgd_step_host (pinned host gradients, x and aggregate; copies inside the timed region)"}
        del hg, hx, hagg

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.kind == "intsgd":
        v, dt, desc = oracle_sample_throughput(n, d, args.cpu_sample_log2, args.grad, args.payload, args.rounding)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc, "seconds": dt}
        if not args.no_cpu_all_cores:
            try:
                va, cores, desca = oracle_all_cores_throughput(n, d, args.cpu_sample_log2, args.grad, args.payload, args.rounding)
                cpu["all_cores"] = {"value": va, "unit": UNIT, "cores": cores, "sample": desca}
            except Exception as exc:   # a box that cannot spawn processes still reports the one-thread figure
                cpu["all_cores"] = {"unavailable": repr(exc)}

    sampler.stop()
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if args.grad == "f32" else "bf16->f32", "data": "synthetic", "config": workload_config(args),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "hbm_gbs_algorithmic": achieved * world, "rounding_variants": variants,
            "state": {"alpha": st["alpha"], "r": st["r"], "max_abs_agg": st["max_abs_agg"],
                      "clipped": sum(st["clip_count"]), "step": st["step"]},
        }
        print(json.dumps(line))
    lib.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the fused 8-bit Adam step (dt8) on B200.

    python bench.py --gpus N --steps K --warmup W [--impl dt8|reference]

Workload: one flat fp32 tensor of 2^28 elements per GPU, fp32 gradients N(0,1e-3), AdamW
(lr 1e-3, betas 0.9/0.999, eps 1e-8, wd 0.01), block 2048, states pre-warmed by 10 steps.
A step is one call of dt8_adam_step over the whole tensor (one kernel launch).  The metric is the
effective HBM bandwidth: algorithmic bytes of a step (16 B per element + 16 B per block) divided
by the device time of the step, summed over the GPUs (each GPU owns its own tensor: the step
shards on block boundaries with no exchange, so scaling is weak).

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "adam8bit_step_effective_hbm_bandwidth"
UNIT = "GB/s"
WORKLOAD = "adam8bit_flat_2^28_fp32grad_block2048_wd0.01_prewarm10"
DATASHEET_GBS = 8000.0
FALLBACK_PEAK_GBS = 6650.0
# DRAM bytes (read + write) of one launch of the fused Adam kernel on 2^26 elements, from the ncu
# capture summarised in profiles/; traffic is proportional to the element count (every byte is
# touched once), so it is scaled to the launch that is timed.  Set to None when the kernel changes.
NCU_TRAFFIC_BYTES_2P26 = 671457536 + 351272448


def algorithmic_bytes(n: int, block: int) -> int:
    """Adam, fp32 gradients: read w4+g4+m1+r1, write w4+m1+r1 per element; 2 absmax in, 2 out per block."""
    nb = (n + block - 1) // block
    return 16 * n + 16 * nb


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_PEAK_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {
        0x0000000000000004: "sw_power_cap",
        0x0000000000000008: "hw_slowdown",
        0x0000000000000020: "sw_thermal_slowdown",
        0x0000000000000040: "hw_thermal_slowdown",
        0x0000000000000080: "hw_power_brake_slowdown",
    }

    def __init__(self, index: int, uuid: str = None, period_s: float = 0.01):
        self.index, self.uuid, self.period = index, uuid, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(self.uuid) if self.uuid else None
            except Exception:
                self._h = None
            if self._h is None:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nvml = None
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self._nvml
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
               "samples": len(self.samples)}
        if self.samples:
            out["sm_mhz"] = statistics.median(self.samples)
        elif self._nvml is None:
            out.update(self._nvidia_smi_once())
        return out

    def _nvidia_smi_once(self):
        try:
            q = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=clocks.sm,clocks.max.sm",
                                "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10)
            a, b = q.stdout.strip().split(",")
            return {"sm_mhz": float(a), "sm_max_mhz": float(b), "note": "single nvidia-smi sample after the run"}
        except Exception:
            return {}


# --------------------------------------------------------------------------------------------------
# distributed plumbing
# --------------------------------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, device) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


# --------------------------------------------------------------------------------------------------
# the dt8 arm
# --------------------------------------------------------------------------------------------------
def run_dt8(args):
    import torch
    import torch.distributed as dist
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import build as dt8_build
    from paper_2412_01195_b200 import synth

    rank, local_rank, world = dist_env()
    if local_rank == 0:
        dt8_build.build_library()          # no-op when libdt8.so is newer than its sources
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the dt8 path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()                     # the other ranks wait for rank 0's build check
    c = dict(synth.ADAM_FLAT_LARGE)
    n, B = (args.n or c["n"]), c["block_size"]
    hp = (c["lr"], c["beta1"], c["beta2"], c["eps"], c["weight_decay"])
    dt8.dt8_init()

    w, g = synth.flat_adam_inputs(n, c["seed"] + 17 * rank, device=dev)
    mc, ma = dt8.new_state(n, B, True, dev)
    rc, ra = dt8.new_state(n, B, False, dev)
    step = 0
    for _ in range(c["prewarm_steps"]):          # states pre-warmed with fresh gradients
        step += 1
        gt = synth.fresh_grad(n, c["seed"] + 17 * rank, step, device=dev)
        dt8.dt8_adam_step(w, gt, mc, ma, rc, ra, *hp, step, B)
        del gt
    for _ in range(max(args.warmup, 0)):
        step += 1
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, *hp, step, B)
    torch.cuda.synchronize()

    # ---- device-resident timing: K steps between two events on the launching stream -------------
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        uuid = None
    sampler = ClockSampler(local_rank, uuid)
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_head = torch.cuda.Event(enable_timing=True)
    head_steps = min(50, args.steps)       # the GPU lowers its SM clock after ~0.1 s under load
    e0.record()
    for i in range(args.steps):
        step += 1
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, *hp, step, B)
        if i + 1 == head_steps:
            e_head.record()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), dev)
    ms_step = ms_total / args.steps
    ms_head = max_over_ranks(e0.elapsed_time(e_head), dev) / head_steps
    launches = args.steps

    bytes_step = algorithmic_bytes(n, B)
    gbs_per_gpu = bytes_step / (ms_step * 1e-3) / 1e9
    value = gbs_per_gpu * world
    peak, peak_src = measured_peak()
    traffic = args.traffic_bytes
    if traffic is None and NCU_TRAFFIC_BYTES_2P26 is not None:
        traffic = round(NCU_TRAFFIC_BYTES_2P26 * n / float(1 << 26))

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ------------
    e2e = run_e2e(dt8, torch, dev, n, B, hp, step, w, g, mc, ma, rc, ra, args, world)

    out = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_step, 5),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "elements_per_gpu": n, "block_size": B, "grad_dtype": "f32",
                   "optimizer": "AdamW, bias correction", "l2_policy": "inputs larger than L2 (4.3 GB per step)",
                   "parallelism": f"independent block ranges x{world}"},
        "elements_per_s": round(n * world / (ms_step * 1e-3), 1),
        "pct_of_measured_peak": round(100 * gbs_per_gpu / peak, 2),
        "pct_of_datasheet_peak": round(100 * gbs_per_gpu / DATASHEET_GBS, 2),
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": round(gbs_per_gpu, 2), "peak": peak, "unit": "GB/s",
                     "frac": round(gbs_per_gpu / peak, 4), "traffic": traffic,
                     "kernel": "dt8::block_kernel<AdamOp<2048,16,512,f32 grads,AdamW>,SingleArgs>",
                     "algorithmic_bytes_per_launch": bytes_step, "peak_source": peak_src,
                     "per_launch_ms": round(ms_step, 5),
                     "first_steps": {"steps": head_steps, "per_launch_ms": round(ms_head, 5),
                                     "frac": round(bytes_step / (ms_head * 1e-3) / 1e9 / peak, 4)}},
    }
    if rank == 0:
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(c, B)
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(dt8, torch, dev, n, B, hp, step, w, g, mc, ma, rc, ra, args, world):
    """Same step, but the tensors live in pinned host memory: every step copies parameters,
    gradients and states to the device, steps them and copies the results back, through the
    package's chunked, three-stream pipeline (StreamedAdam8bit)."""
    from paper_2412_01195_b200.offload import StreamedAdam8bit
    k = max(1, min(args.e2e_steps, args.steps))
    host = [torch.empty_like(t, device="cpu").pin_memory() for t in (w, g, mc, ma, rc, ra)]
    for h, t in zip(host, (w, g, mc, ma, rc, ra)):
        h.copy_(t)
    torch.cuda.synchronize()
    pipe = StreamedAdam8bit(B, chunk_elems=1 << 24, buffers=3, grad_dtype=g.dtype, device=dev)
    pipe.step(*host, *hp, step + 1)
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(k):
        pipe.step(*host, *hp, step + 2 + i)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), dev) / k
    gbs = algorithmic_bytes(n, B) / (ms * 1e-3) / 1e9 * world
    return {"value": round(gbs, 3), "unit": UNIT, "h2d_bytes_per_step": pipe.h2d_bytes,
            "d2h_bytes_per_step": pipe.d2h_bytes, "ms_per_step": round(ms, 3), "steps": k,
            "path": "pinned host -> device, dt8_adam_step (C ABI), device -> pinned host; 2^24-element "
                    "chunks on three streams (StreamedAdam8bit)"}


# --------------------------------------------------------------------------------------------------
# CPU baseline (the checker, as it stands) and the reference arm
# --------------------------------------------------------------------------------------------------
def oracle_rate(n, B, c, steps, warm, threads):
    """Times the CPU checker's 8-bit Adam step on n elements; returns (seconds per step, threads)."""
    import numpy as np
    import oracle
    from paper_2412_01195_b200 import synth
    oracle.set_threads(threads)
    w, g = (t.numpy() for t in synth.flat_adam_inputs(n, c["seed"]))
    nb = (n + B - 1) // B
    mc, ma = np.full(n, 127, np.uint8), np.zeros(nb, np.float32)
    rc, ra = np.zeros(n, np.uint8), np.zeros(nb, np.float32)
    t = 0
    for _ in range(warm):
        t += 1
        oracle.adam_step(w, g, mc, ma, rc, ra, c["lr"], c["beta1"], c["beta2"], c["eps"], c["weight_decay"], t, B)
    t0 = time.perf_counter()
    for _ in range(steps):
        t += 1
        oracle.adam_step(w, g, mc, ma, rc, ra, c["lr"], c["beta1"], c["beta2"], c["eps"], c["weight_decay"], t, B)
    return (time.perf_counter() - t0) / steps, oracle.get_threads()


def cpu_baseline(c, B):
    cores = os.cpu_count() or 1
    n = 1 << 26
    sec, used = oracle_rate(n, B, c, steps=3, warm=2, threads=cores)
    gbs = algorithmic_bytes(n, B) / sec / 1e9
    return {"value": round(gbs, 3), "unit": UNIT, "cores": used, "kind": "oracle",
            "elements_per_s": round(n / sec, 1),
            "sample": "2^26-element slice of the workload (same distributions), 2 warm + 3 timed steps, OpenMP over blocks"}


def run_reference(args):
    """The reference arm: the CPU checker timed on the host cores on a bounded sample per step."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    from paper_2412_01195_b200 import synth
    c = dict(synth.ADAM_FLAT_LARGE)
    B = c["block_size"]
    cores = os.cpu_count() or 1
    probe_sec, used = oracle_rate(1 << 22, B, c, steps=1, warm=1, threads=cores)
    rate = (1 << 22) / probe_sec                                     # elements per second
    budget_s = 120.0
    total_steps = max(args.steps + args.warmup, 1)
    n = int(rate * budget_s / total_steps)
    n = max(16 * B, min(1 << 26, (n // B) * B))
    sec, used = oracle_rate(n, B, c, steps=args.steps, warm=args.warmup, threads=cores)
    gbs = algorithmic_bytes(n, B) / sec / 1e9
    sample = f"{n} elements per step (a slice of the 2^28-element workload, same distributions)"
    out = {
        "impl": "reference", "metric": METRIC, "value": round(gbs, 3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(sec * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "block_size": B, "grad_dtype": "f32", "sample": sample},
        "elements_per_s": round(n / sec, 1),
        "cpu_baseline": {"value": round(gbs, 3), "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(gbs, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="dt8", choices=["dt8", "reference"])
    ap.add_argument("--n", type=int, default=0, help="elements per GPU (default: the 2^28 workload)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch from an ncu capture, copied into roofline.traffic")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "dt8":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_dt8(args)


if __name__ == "__main__":
    main()

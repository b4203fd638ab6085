#!/usr/bin/env python
"""Benchmark of the dt8 library on B200: the fused 8-bit Adam step and everything around it.

    python bench.py --gpus N --steps K --warmup W [--impl dt8|reference] [--only CASE,...]

Headline workload: one flat fp32 tensor of 2^28 elements per GPU, fp32 gradients N(0,1e-3), AdamW
(lr 1e-3, betas 0.9/0.999, eps 1e-8, wd 0.01), block 2048, states pre-warmed by 10 steps.  A step
is one call of dt8_adam_step over the whole tensor (one kernel launch).  The metric is the
effective HBM bandwidth: algorithmic bytes of a step (16 B per element + 16 B per block) divided
by the device time of the step, summed over the GPUs (each GPU owns its own tensor: the step
shards on block boundaries with no exchange, so scaling is weak).

The same JSON line carries, under "kernels", every other entry point timed the same way (CUDA
events on the launching stream, inputs larger than L2) with its own fraction of the measured copy
bandwidth, a "sustained" leg (seconds of back-to-back Adam launches with the SM clock sampled, as
cycles per element), the end-to-end leg with host buffers, and the CPU checker timed on the host
cores.  With --gpus N > 1 and no launcher environment, the script starts N ranks of itself.

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
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

# DRAM bytes of ONE launch of the fused Adam kernel (fp32 gradients and parameters, block 2048) on
# 2^26 elements, from an ncu capture of `python bench.py --only adam26` (dram__bytes_read.sum,
# dram__bytes_write.sum), with the hash of the kernel sources the capture belongs to.  The capture
# reads below the algorithmic bytes because dirty lines stay in the 126 MB L2 when the kernel
# ends: a constant per launch, not a proportion.  For a launch on n elements the reported traffic
# is therefore this capture plus the algorithmic bytes of the extra n - 2^26 elements.  When the
# kernel sources change the constant no longer applies and traffic is reported as null.
NCU_CAPTURE = {"elements": 1 << 26, "dram_read": 671521792, "dram_write": 350734848,
               "source_hash": "4e58893f68ce4231"}


HEADLINE_KERNEL_SOURCES = ("dt8_kernels.cuh", "dt8_tables.h", "dt8_adam_impl.cuh", "dt8_launch.h", "dt8_adam_ff.cu")


def kernel_source_hash() -> str:
    """Hash of the files the headline kernel is compiled from."""
    h = hashlib.sha256()
    for name in HEADLINE_KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2412_01195_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def adam_bytes(n: int, block: int, g_bytes: int = 4, p_bytes: int = 4) -> int:
    """Adam: read w + g + m1 + r1, write w + m1 + r1 per element; 2 absmax in, 2 out per block."""
    return (2 * p_bytes + g_bytes + 4) * n + 16 * ((n + block - 1) // block)


def sgd_bytes(n: int, block: int, g_bytes: int = 4, p_bytes: int = 4) -> int:
    return (2 * p_bytes + g_bytes + 2) * n + 8 * ((n + block - 1) // block)


def algorithmic_bytes(n: int, block: int) -> int:
    return adam_bytes(n, block)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_PEAK_GBS, "fallback (6.65 TB/s, an earlier measurement of the same GPU model)"


def reported_traffic(n: int, block: int):
    """(bytes or None, note) for roofline.traffic of the headline kernel on n elements."""
    if NCU_CAPTURE["source_hash"] != kernel_source_hash():
        return None, "kernel sources changed since the ncu capture"
    cap = NCU_CAPTURE["dram_read"] + NCU_CAPTURE["dram_write"]
    extra = adam_bytes(n, block) - adam_bytes(NCU_CAPTURE["elements"], block)
    return cap + extra, ("ncu capture at 2^26 elements (%d B, L2 residue included) plus the algorithmic "
                         "bytes of the remaining elements" % cap)


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
        self.samples, self.times, self.reasons = [], [], set()
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
                self.times.append(time.perf_counter())
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


def launched_by_a_launcher() -> bool:
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int) -> int:
    """Started without a launcher but asked for n > 1 GPUs: run n ranks of this script (one per
    GPU) through torch's launcher and pass their output through."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd, cwd=ROOT).returncode


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


def init_ranks(args, device):
    """Joins the process group when there is more than one rank; the line printed at the end
    must never claim fewer GPUs than were asked for."""
    import torch.distributed as dist
    rank, local_rank, world = dist_env()
    if world != args.gpus:
        raise RuntimeError(f"--gpus {args.gpus} but {world} rank(s) are running: start the benchmark with "
                           f"--gpus equal to the number of ranks")
    if world > 1:
        backend = "gloo" if args.plumbing_check else "nccl"
        if backend == "nccl":
            os.environ.setdefault("NCCL_DEBUG", "INFO")       # the communicator lines go to stderr
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
        dist.barrier()
    return rank, local_rank, world


# --------------------------------------------------------------------------------------------------
# timing
# --------------------------------------------------------------------------------------------------
def time_launches(fn, iters: int, warm: int) -> float:
    """Milliseconds per call of fn: `iters` back-to-back calls between two CUDA events on the
    current stream (the stream the binding launches on), after `warm` untimed calls."""
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def time_graph_replay(fn, reps: int = 20, iters: int = 20) -> float:
    """Milliseconds per call of fn with the host out of the way: `reps` calls captured in a CUDA
    graph, the graph replayed `iters` times between two events.  For launches of a few
    microseconds the back-to-back figure of time_launches is the host's submission rate."""
    import torch
    fn()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(reps):
            fn()
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (iters * reps)


def kernel_entry(ms: float, nbytes: int, peak: float, **extra) -> dict:
    gbs = nbytes / (ms * 1e-3) / 1e9
    out = {"ms": round(ms, 5), "GBps": round(gbs, 1), "frac": round(gbs / peak, 4), "bytes_per_launch": nbytes}
    out.update(extra)
    return out


# --------------------------------------------------------------------------------------------------
# the other entry points, each timed like the headline step
# --------------------------------------------------------------------------------------------------
HP = (1e-3, 0.9, 0.999, 1e-8, 0.01)


def case_adam(dev, n, block=2048, g_dtype="f32", p_dtype="f32", flags=None, hp=HP):
    import torch
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import synth
    td = {"f32": torch.float32, "bf16": torch.bfloat16}
    flags = dt8.DEFAULT_ADAM_FLAGS if flags is None else flags
    w, g = synth.flat_adam_inputs(n, 4, device=dev)
    w, g = w.to(td[p_dtype]), g.to(td[g_dtype])
    mc, ma = dt8.new_state(n, block, True, dev)
    rc, ra = dt8.new_state(n, block, False, dev)
    for t in range(1, 6):                      # states away from zero before timing
        gt = synth.fresh_grad(n, 4, t, device=dev, dtype=td[g_dtype])
        dt8.dt8_adam_step(w, gt, mc, ma, rc, ra, *hp, t, block, flags)
    step = [5]

    def fn():
        step[0] += 1
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, *hp, step[0], block, flags)
    return fn, adam_bytes(n, block, g.element_size(), w.element_size()), n


def case_sgd(dev, n, block=2048, g_dtype="f32", p_dtype="f32"):
    import torch
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import synth
    td = {"f32": torch.float32, "bf16": torch.bfloat16}
    w, g = synth.flat_adam_inputs(n, 4, device=dev)
    w, g = w.to(td[p_dtype]), g.to(td[g_dtype])
    mc, ma = dt8.new_state(n, block, True, dev)
    step = [0]

    def fn():
        step[0] += 1
        dt8.dt8_sgd_step(w, g, mc, ma, 0.1, 0.9, 1e-4, step[0], block)
    return fn, sgd_bytes(n, block, g.element_size(), w.element_size()), n


def case_quantize(dev, n, block, signed):
    import torch
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import synth
    x = synth.laplace_outliers(n, 3, device=dev)
    x = x if signed else x.abs()
    codes = torch.empty(n, dtype=torch.uint8, device=dev)
    am = torch.empty(dt8.num_blocks(n, block), device=dev)
    return (lambda: dt8.dt8_quantize_blockwise(x, block, signed, codes, am)), 5 * n + 4 * am.numel(), n


def case_dequantize(dev, n, block, signed):
    import torch
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import synth
    x = synth.laplace_outliers(n, 3, device=dev)
    codes, am = dt8.dt8_quantize_blockwise(x if signed else x.abs(), block, signed)
    del x
    out = torch.empty(n, device=dev)
    return (lambda: dt8.dt8_dequantize_blockwise(codes, am, block, signed, out)), 5 * n + 4 * am.numel(), n


def case_multi_adam(dev):
    """The ~200-tensor ResNet speaker-extractor list, bf16 gradients, one launch (L2-resident)."""
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import synth
    B = 2048
    ps = synth.resnet_adam_params(2, dev)
    gs = synth.resnet_adam_grads(2, 1, dev)
    sm = [dt8.new_state(p.numel(), B, True, dev) for p in ps]
    sr = [dt8.new_state(p.numel(), B, False, dev) for p in ps]
    prepared = dt8.PreparedTensorList(ps, gs, [s[0] for s in sm], [s[1] for s in sm],
                                      [s[0] for s in sr], [s[1] for s in sr])
    k = [0]

    def fn():
        k[0] += 1
        prepared.adam_step(1e-3, 0.9, 0.999, 1e-8, 0.05, k[0], B)
    tot = sum(p.numel() for p in ps)
    return fn, 14 * tot + 16 * sum(dt8.num_blocks(p.numel(), B) for p in ps), tot


def case_multi_sgd(dev):
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import synth
    B = 2048
    ps = synth.conv_sgd_params(1, dev)
    gs = synth.conv_sgd_grads(1, 1, dev)
    sm = [dt8.new_state(p.numel(), B, True, dev) for p in ps]
    prepared = dt8.PreparedTensorList(ps, gs, [s[0] for s in sm], [s[1] for s in sm])
    k = [0]

    def fn():
        k[0] += 1
        prepared.sgd_step(0.1, 0.9, 1e-4, k[0], B)
    tot = sum(p.numel() for p in ps)
    return fn, 14 * tot + 8 * sum(dt8.num_blocks(p.numel(), B) for p in ps), tot


def case_coupling(dev, shape, inverse=False):
    """One half of Eq. revnet4 / revnet5 on an activation of the paper's first reversible stage."""
    import torch
    from paper_2412_01195_b200 import rev, synth
    n, c, f, t = shape
    x = synth.normal(n * c * f * t, 1.0, 31, device=dev).reshape(shape)
    br = synth.normal(n * c * f * t // 2, 1.0, 32, device=dev).reshape(n, c // 2, f, t)
    y = torch.empty_like(x)
    op = rev.dt8_rev_coupling_inverse if inverse else rev.dt8_rev_coupling_forward
    return (lambda: op(x, br, y, 0)), 12 * br.numel(), br.numel()


def case_space_to_depth(dev, shape, inverse=False):
    import torch
    from paper_2412_01195_b200 import rev, synth
    n, c, f, t = shape
    x = synth.normal(n * c * f * t, 1.0, 33, device=dev).reshape(shape)
    y = torch.empty((n, 4 * c, f // 2, t // 2), device=dev)
    if inverse:
        return (lambda: rev.dt8_rev_depth_to_space(y, x)), 8 * x.numel(), x.numel()
    return (lambda: rev.dt8_rev_space_to_depth(x, y)), 8 * x.numel(), x.numel()


def sub_cases():
    """name -> (builder, launches, description).  Sizes: the steps at 2^28 and at 2^26 (the
    smallest size the 80 % target is set on), quantize / dequantize at 2^27 (the largest size of
    the sweep configuration), the reversible kernels on a batch of 128 activations of the first
    reversible stage (48 x 80 x 200)."""
    import paper_2412_01195_b200 as dt8
    BC = dt8.DT8_ADAM_BIAS_CORRECTION
    act = (128, 48, 80, 200)
    c = {
        "adam26": (lambda d: case_adam(d, 1 << 26), 50, "Adam, fp32 grads, 2^26 elements"),
        "adam26_bf16grad": (lambda d: case_adam(d, 1 << 26, g_dtype="bf16"), 50, "Adam, bf16 grads, 2^26"),
        "adam26_bf16param": (lambda d: case_adam(d, 1 << 26, p_dtype="bf16"), 50, "Adam, bf16 params, 2^26"),
        "adam26_coupled_l2": (lambda d: case_adam(d, 1 << 26, flags=BC), 50, "Adam, coupled L2 decay (IEEE parameter path), 2^26"),
        "adam_bf16grad": (lambda d: case_adam(d, 1 << 28, g_dtype="bf16"), 50, "Adam, bf16 grads, 2^28"),
        "adam_bf16param": (lambda d: case_adam(d, 1 << 28, p_dtype="bf16"), 50, "Adam, bf16 params, fp32 grads, 2^28"),
        "adam_bf16both": (lambda d: case_adam(d, 1 << 28, g_dtype="bf16", p_dtype="bf16"), 50, "Adam, bf16 params and grads, 2^28"),
        "adam_coupled_l2": (lambda d: case_adam(d, 1 << 28, flags=BC), 50, "Adam, coupled L2 decay (IEEE parameter path), 2^28"),
        "adam_tiny_eps": (lambda d: case_adam(d, 1 << 28, hp=(1e-3, 0.9, 0.999, 1e-20, 0.01)), 50, "AdamW, eps 1e-20 (subnormal-keeping path), 2^28"),
        "adam_block256": (lambda d: case_adam(d, 1 << 27, block=256), 50, "Adam, block 256, 2^27"),
        "adam_block512": (lambda d: case_adam(d, 1 << 27, block=512), 50, "Adam, block 512, 2^27"),
        "adam_block4096": (lambda d: case_adam(d, 1 << 27, block=4096), 50, "Adam, block 4096, 2^27"),
        "sgd": (lambda d: case_sgd(d, 1 << 28), 50, "SGD momentum, fp32 grads, 2^28"),
        "sgd26": (lambda d: case_sgd(d, 1 << 26), 50, "SGD momentum, fp32 grads, 2^26"),
        "sgd_bf16grad": (lambda d: case_sgd(d, 1 << 28, g_dtype="bf16"), 50, "SGD momentum, bf16 grads, 2^28"),
        "sgd_block256": (lambda d: case_sgd(d, 1 << 27, block=256), 50, "SGD momentum, block 256, 2^27"),
        "quantize_signed": (lambda d: case_quantize(d, 1 << 27, 2048, True), 50, "quantize, signed table, block 2048, 2^27"),
        "quantize_unsigned": (lambda d: case_quantize(d, 1 << 27, 2048, False), 50, "quantize, unsigned table, block 2048, 2^27"),
        "quantize_block256": (lambda d: case_quantize(d, 1 << 27, 256, True), 50, "quantize, signed, block 256, 2^27"),
        "quantize_block4096": (lambda d: case_quantize(d, 1 << 27, 4096, True), 50, "quantize, signed, block 4096, 2^27"),
        "dequantize_signed": (lambda d: case_dequantize(d, 1 << 27, 2048, True), 50, "dequantize, signed, block 2048, 2^27"),
        "dequantize_unsigned": (lambda d: case_dequantize(d, 1 << 27, 2048, False), 50, "dequantize, unsigned, block 2048, 2^27"),
        "multi_adam_resnet": (case_multi_adam, 200, "Adam, 197-tensor list, bf16 grads, one launch (7.0 M elements: L2-resident, not an HBM figure)"),
        "multi_sgd_conv": (case_multi_sgd, 200, "SGD, 37-tensor list, one launch (6.6 M elements: L2-resident, not an HBM figure)"),
        "rev_coupling_forward": (lambda d: case_coupling(d, act), 50, "Eq. revnet4, one half, 128 x 48 x 80 x 200"),
        "rev_coupling_inverse": (lambda d: case_coupling(d, act, True), 50, "Eq. revnet5, one half, 128 x 48 x 80 x 200"),
        "rev_space_to_depth": (lambda d: case_space_to_depth(d, (128, 24, 80, 200)), 50, "Eq. revnet6, 128 x 24 x 80 x 200"),
        "rev_depth_to_space": (lambda d: case_space_to_depth(d, (128, 24, 80, 200), True), 50, "inverse of Eq. revnet6"),
        "rev_space_to_depth_t50": (lambda d: case_space_to_depth(d, (512, 75, 20, 50)), 50, "Eq. revnet6, 512 x 75 x 20 x 50 (rows of 50: 8-byte pieces)"),
    }
    return c


def run_sub_cases(dev, names, peak, clock_of=None):
    """Times the named cases; clock_of = (gpu index, uuid) also samples the SM clock during each
    case (the cases that are bound by instruction issue depend on it)."""
    import gc
    import torch
    cases = sub_cases()
    out, launches = {}, 0
    for name in names:
        build, iters, desc = cases[name]
        fn, nbytes, units = build(dev)
        sampler = None
        if clock_of is not None:
            time_launches(fn, 5, 0)
            sampler = ClockSampler(clock_of[0], clock_of[1], period_s=0.002)
            sampler.start()
        ms = time_launches(fn, iters, 5)
        out[name] = kernel_entry(ms, nbytes, peak, launches=iters, units=units, what=desc)
        if sampler is not None:
            clk = sampler.stop()
            out[name]["sm_mhz"] = clk.get("sm_mhz")
            launches += 5
        launches += iters
        if name.startswith("multi_"):
            # a launch of ~20 us: also the device-side time, free of the host's submission rate
            out[name]["ms_graph_replay"] = round(time_graph_replay(fn), 5)
            launches += 20 * 21 + 1
        del fn
        gc.collect()
        torch.cuda.empty_cache()
    return out, launches


# --------------------------------------------------------------------------------------------------
# sustained leg: seconds of back-to-back launches, the SM clock sampled meanwhile
# --------------------------------------------------------------------------------------------------
def run_sustained(dev, local_rank, uuid, step_fn, n, nbytes, peak, seconds: float, est_ms: float):
    """Back-to-back launches of the headline step for about `seconds`, timed in segments of 100
    launches.  A B200 lowers its SM clock under a long load, and the step is close to the
    instruction-issue ceiling, so the figure that describes a training loop is cycles per element
    (time x SM clock / elements) together with the clock it was measured at."""
    import torch
    seg = 100
    segments = max(3, int(seconds * 1e3 / (est_ms * seg)) + 1)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(segments + 1)]
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank, uuid, period_s=0.005)
    sampler.start()
    t0 = time.perf_counter()
    events[0].record()
    for k in range(segments):
        for _ in range(seg):
            step_fn()
        events[k + 1].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    cum = [events[0].elapsed_time(e) for e in events]            # ms since the first launch started
    total_ms = cum[-1]
    ms_launch = total_ms / (segments * seg)
    out = {"launches": segments * seg, "seconds": round(total_ms * 1e-3, 3), "ms_per_launch": round(ms_launch, 5),
           "frac": round(nbytes / (ms_launch * 1e-3) / 1e9 / peak, 4), "sm_mhz_median": clocks.get("sm_mhz"),
           "sm_max_mhz": clocks.get("sm_max_mhz"), "reasons": clocks.get("reasons"), "clock_samples": clocks.get("samples")}
    if clocks.get("sm_mhz"):
        out["cycles_per_element"] = round(ms_launch * 1e-3 * clocks["sm_mhz"] * 1e6 / n, 6)
    # segments binned by the clock sampled while they ran (the GPU was idle before the first launch,
    # so segment k ran from t0 + cum[k] to t0 + cum[k + 1] on the host's clock)
    bins = {}
    for k in range(segments):
        lo, hi = t0 + cum[k] * 1e-3, t0 + cum[k + 1] * 1e-3
        mhz = [m for m, t in zip(sampler.samples, sampler.times) if lo <= t < hi]
        if not mhz:
            continue
        key = int(round(statistics.median(mhz) / 50.0) * 50)
        bins.setdefault(key, []).append((cum[k + 1] - cum[k]) / seg)
    out["by_clock"] = [{"sm_mhz": key, "segments": len(v), "ms_per_launch": round(statistics.mean(v), 5),
                        "cycles_per_element": round(statistics.mean(v) * 1e-3 * key * 1e6 / n, 6),
                        "frac": round(nbytes / (statistics.mean(v) * 1e-3) / 1e9 / peak, 4)}
                       for key, v in sorted(bins.items(), reverse=True)]
    return out, segments * seg


# --------------------------------------------------------------------------------------------------
# reversible stack: activation memory per sample with and without stored activations
# --------------------------------------------------------------------------------------------------
def run_rev_memory(dev, blocks: int = 8, batch: int = 8, channels: int = 48, freq: int = 80, frames: int = 200):
    """Peak device memory of one training step of a stack of reversible blocks (basic-block
    branches: conv3x3 - ReLU - conv3x3 on C/2 channels, the 'rev_res' stage of the paper's layer
    tables on 80 x 200 features), through RevSequence (Alg. 1, nothing stored between blocks) and
    through ordinary autograd (every activation stored), in bytes per sample."""
    import torch
    from paper_2412_01195_b200 import rev

    def branch():
        c = channels // 2
        return torch.nn.Sequential(torch.nn.Conv2d(c, c, 3, padding=1), torch.nn.ReLU(),
                                   torch.nn.Conv2d(c, c, 3, padding=1))
    torch.manual_seed(0)
    net = rev.RevSequence([rev.RevBlock(branch(), branch()) for _ in range(blocks)]).to(dev)
    from paper_2412_01195_b200 import synth
    x = synth.normal(batch * channels * freq * frames, 1.0, 41, device=dev).reshape(batch, channels, freq, frames)
    c = channels // 2

    def stored(inp):
        h = inp
        for blk in net.blocks:
            h1 = h[:, :c] + blk.F(h[:, c:])
            h = torch.cat([h1, h[:, c:] + blk.G(h1)], 1)
        return h

    def measure(fwd):
        for p in net.parameters():
            p.grad = None
        torch.cuda.synchronize()
        torch.cuda.reset_peak_memory_stats(dev)
        base = torch.cuda.memory_allocated(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fwd(x).square().mean().backward()
        e1.record()
        torch.cuda.synchronize()
        return torch.cuda.max_memory_allocated(dev) - base, e0.elapsed_time(e1)
    measure(net)                                            # warm-up (cuDNN plans, allocator)
    measure(stored)
    rev_bytes, rev_ms = measure(net)
    sto_bytes, sto_ms = measure(stored)
    return {"blocks": blocks, "batch": batch, "activation_shape": [channels, freq, frames],
            "reversible_bytes_per_sample": rev_bytes // batch, "stored_bytes_per_sample": sto_bytes // batch,
            "memory_ratio": round(sto_bytes / max(rev_bytes, 1), 2),
            "reversible_ms": round(rev_ms, 3), "stored_ms": round(sto_ms, 3),
            "time_ratio": round(rev_ms / max(sto_ms, 1e-9), 2),
            "what": "peak extra device memory of forward + backward; branches are library convolutions, "
                    "the coupling steps and Alg. 1's sums are dt8_rev kernels"}


# --------------------------------------------------------------------------------------------------
# the dt8 arm
# --------------------------------------------------------------------------------------------------
DEFAULT_SUBS = ["adam26", "adam_bf16grad", "adam_bf16param", "adam_coupled_l2", "adam_tiny_eps", "adam_block256",
                "adam_block512", "sgd", "sgd26", "sgd_bf16grad", "sgd_block256", "quantize_signed",
                "quantize_unsigned", "quantize_block256", "quantize_block4096", "dequantize_signed",
                "dequantize_unsigned", "multi_adam_resnet", "multi_sgd_conv", "rev_coupling_forward",
                "rev_coupling_inverse", "rev_space_to_depth", "rev_depth_to_space", "rev_space_to_depth_t50"]


def run_plumbing_check(args):
    """No GPU work: the ranks join over gloo, take the barrier and the maximum over ranks, and
    rank 0 prints a line with the number of ranks.  Used to test the launch path on CPU."""
    import torch
    rank, _, world = init_ranks(args, torch.device("cpu"))
    barrier()
    slowest = max_over_ranks(1.0 + rank, torch.device("cpu"))
    barrier()
    if rank == 0:
        print(json.dumps({"plumbing_check": True, "n_gpus": world, "slowest": slowest}), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_dt8(args):
    import torch
    import torch.distributed as dist
    import paper_2412_01195_b200 as dt8
    from paper_2412_01195_b200 import build as dt8_build
    from paper_2412_01195_b200 import synth

    _, local_rank, _ = dist_env()
    if local_rank == 0:
        dt8_build.build_library()          # no-op when libdt8.so is newer than its sources
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the dt8 path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rank, local_rank, world = init_ranks(args, dev)
    peak, peak_src = measured_peak()
    dt8.dt8_init()
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        uuid = None

    if args.only:                              # a few sub-cases alone (what an ncu capture runs)
        names = [s for s in args.only.split(",") if s]
        kernels, launches = run_sub_cases(dev, names, peak, (local_rank, uuid))
        if rank == 0:
            print(json.dumps({"only": names, "kernels": kernels, "gpu_launches": launches,
                              "peak": peak, "peak_source": peak_src}), flush=True)
        return

    c = dict(synth.ADAM_FLAT_LARGE)
    n, B = (args.n or c["n"]), c["block_size"]
    hp = (c["lr"], c["beta1"], c["beta2"], c["eps"], c["weight_decay"])
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

    bytes_step = adam_bytes(n, B)
    gbs_per_gpu = bytes_step / (ms_step * 1e-3) / 1e9
    value = gbs_per_gpu * world
    traffic, traffic_note = (args.traffic_bytes, "given on the command line") if args.traffic_bytes else reported_traffic(n, B)

    # ---- sustained leg (one GPU): seconds of launches, cycles per element by clock ---------------
    sustained = None
    if world == 1 and args.sustained_seconds > 0:
        st = [step]

        def one_step():
            st[0] += 1
            dt8.dt8_adam_step(w, g, mc, ma, rc, ra, *hp, st[0], B)
        sustained, extra = run_sustained(dev, local_rank, uuid, one_step, n, bytes_step, peak,
                                         args.sustained_seconds, ms_step)
        step = st[0]
        launches += extra

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ------------
    e2e = run_e2e(dt8, torch, dev, n, B, hp, step, w, g, mc, ma, rc, ra, args, world)
    del w, g, mc, ma, rc, ra
    torch.cuda.empty_cache()

    # ---- every other entry point, timed the same way (one GPU) ------------------------------------
    kernels, rev_memory = None, None
    if world == 1 and not args.no_kernels:
        kernels, extra = run_sub_cases(dev, DEFAULT_SUBS, peak, (local_rank, uuid))
        launches += extra
        rev_memory = run_rev_memory(dev)
        # the same at two other depths: the reversible figure does not depend on the depth
        rev_memory["by_depth"] = [{k: m[k] for k in ("blocks", "reversible_bytes_per_sample", "stored_bytes_per_sample",
                                                     "memory_ratio", "time_ratio")}
                                  for m in (run_rev_memory(dev, blocks=4), run_rev_memory(dev, blocks=16))]

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
                     "frac": round(gbs_per_gpu / peak, 4), "traffic": traffic, "traffic_note": traffic_note,
                     "kernel": "dt8::block_kernel<AdamOp<2048,16,512,f32 grads,f32 params,AdamW>,SingleArgs>",
                     "algorithmic_bytes_per_launch": bytes_step, "peak_source": peak_src,
                     "per_launch_ms": round(ms_step, 5),
                     "first_steps": {"steps": head_steps, "per_launch_ms": round(ms_head, 5),
                                     "frac": round(bytes_step / (ms_head * 1e-3) / 1e9 / peak, 4)}},
    }
    if sustained is not None:
        out["sustained"] = sustained
    if kernels is not None:
        out["kernels"] = kernels
        out["rev_memory"] = rev_memory
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
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the sustained leg (0: skip it)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernels", action="store_true", help="skip the other entry points")
    ap.add_argument("--only", default="", help="comma-separated sub-cases to time alone: " +
                    "see sub_cases() (adam26, sgd26, quantize_signed, dequantize_signed, rev_space_to_depth, ...)")
    ap.add_argument("--plumbing-check", action="store_true",
                    help="no GPU work: join the ranks over gloo and print the rank count (tests the launch path)")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch from an ncu capture, copied into roofline.traffic")
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    if args.gpus > 1 and not launched_by_a_launcher():
        sys.exit(spawn_ranks(args.gpus))
    if args.warmup < 3 and args.impl == "dt8":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.plumbing_check:
        run_plumbing_check(args)
    else:
        run_dt8(args)


if __name__ == "__main__":
    main()

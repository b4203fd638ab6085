"""Throughput of every dt8 entry point on the current GPU.

    python -m paper_2412_01195_b200.timing [case ...]

Cases: adam adam26 adambf adambf26 adaml2 sgd sgd26 sgdbf blocks quant dequant multi (default: all).
Each case runs the public binding in a loop of 50 launches after 5 warm-ups between two CUDA
events on the launching stream and prints milliseconds per launch, effective GB/s (algorithmic
bytes of the method divided by the time) and the fraction of a reference bandwidth (``--peak``,
GB/s; default: the measured copy bandwidth recorded for this machine, else 6650).  Tensors are larger than the L2 cache
except in the tensor-list cases, which say so.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

import paper_2412_01195_b200 as dt8
from paper_2412_01195_b200 import synth

B = 2048
HP = (1e-3, 0.9, 0.999, 1e-8, 0.01)
ALL = ["adam", "adam26", "adambf", "adambf26", "adaml2", "sgd", "sgd26", "sgdbf", "blocks", "quant",
       "dequant", "multi"]


def timeit(fn, iters=50, warm=5):
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


class Report:
    def __init__(self, peak):
        self.peak = peak

    def __call__(self, name, ms, nbytes):
        gbs = nbytes / (ms * 1e-3) / 1e9
        print(f"{name:52s} {ms:9.4f} ms {gbs:9.1f} GB/s {gbs / self.peak:6.3f} of {self.peak:.0f} GB/s",
              flush=True)


def adam_case(report, dev, n, gdt, tag, block=B, flags=dt8.DEFAULT_ADAM_FLAGS):
    w, g = synth.flat_adam_inputs(n, 4, device=dev)
    g = g.to(gdt)
    mc, ma = dt8.new_state(n, block, True, dev)
    rc, ra = dt8.new_state(n, block, False, dev)
    for t in range(1, 6):                      # states away from zero before timing
        gt = synth.fresh_grad(n, 4, t, device=dev, dtype=gdt)
        dt8.dt8_adam_step(w, gt, mc, ma, rc, ra, *HP, t, block, flags)
    step = [5]

    def f():
        step[0] += 1
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, *HP, step[0], block, flags)
    gb = 2 if gdt == torch.bfloat16 else 4
    report(tag, timeit(f), n * (12 + gb) + 16 * dt8.num_blocks(n, block))


def sgd_case(report, dev, n, gdt, tag, block=B):
    w, g = synth.flat_adam_inputs(n, 4, device=dev)
    g = g.to(gdt)
    mc, ma = dt8.new_state(n, block, True, dev)
    step = [0]

    def f():
        step[0] += 1
        dt8.dt8_sgd_step(w, g, mc, ma, 0.1, 0.9, 1e-4, step[0], block)
    gb = 2 if gdt == torch.bfloat16 else 4
    report(tag, timeit(f), n * (10 + gb) + 8 * dt8.num_blocks(n, block))


def quant_cases(report, dev):
    n = 1 << 27
    x = synth.laplace_outliers(n, 3, device=dev)
    for block in (256, 2048, 4096):
        for signed in (True, False):
            xx = x if signed else x.abs()
            codes = torch.empty(n, dtype=torch.uint8, device=dev)
            am = torch.empty(dt8.num_blocks(n, block), device=dev)
            ms = timeit(lambda: dt8.dt8_quantize_blockwise(xx, block, signed, codes, am))
            report(f"quantize n=2^27 B={block} signed={signed}", ms, n * 5 + 4 * am.numel())


def dequant_cases(report, dev):
    n = 1 << 27
    x = synth.laplace_outliers(n, 3, device=dev)
    for signed in (True, False):
        codes, am = dt8.dt8_quantize_blockwise(x if signed else x.abs(), B, signed)
        out = torch.empty(n, device=dev)
        ms = timeit(lambda: dt8.dt8_dequantize_blockwise(codes, am, B, signed, out))
        report(f"dequantize n=2^27 B={B} signed={signed}", ms, n * 5 + 4 * am.numel())


def multi_cases(report, dev):
    ps = synth.resnet_adam_params(2, dev)
    gs = synth.resnet_adam_grads(2, 1, dev)
    sm = [dt8.new_state(p.numel(), B, True, dev) for p in ps]
    sr = [dt8.new_state(p.numel(), B, False, dev) for p in ps]
    mcs, mas = [s[0] for s in sm], [s[1] for s in sm]
    rcs, ras = [s[0] for s in sr], [s[1] for s in sr]
    prepared = dt8.PreparedTensorList(ps, gs, mcs, mas, rcs, ras)
    k = [0]
    tot = sum(p.numel() for p in ps)
    nbk = sum(dt8.num_blocks(p.numel(), B) for p in ps)
    nbytes = tot * 14 + 16 * nbk

    def one_launch():
        k[0] += 1
        prepared.adam_step(1e-3, 0.9, 0.999, 1e-8, 0.05, k[0], B)
    report(f"adam, {len(ps)}-tensor list, {tot} elts, bf16 grads (in L2)", timeit(one_launch, 200), nbytes)

    def rebuilt():
        k[0] += 1
        dt8.dt8_adam_step_multi(ps, gs, mcs, mas, rcs, ras, 1e-3, 0.9, 0.999, 1e-8, 0.05, k[0], B)
    report("  same, pointer arrays rebuilt per call", timeit(rebuilt, 50), nbytes)

    def per_tensor():
        k[0] += 1
        for i in range(len(ps)):
            dt8.dt8_adam_step(ps[i], gs[i], mcs[i], mas[i], rcs[i], ras[i], 1e-3, 0.9, 0.999, 1e-8,
                              0.05, k[0], B)
    report("  same, one launch per tensor", timeit(per_tensor, 20), nbytes)

    nflat = (tot // B) * B
    wf, gf = synth.flat_adam_inputs(nflat, 4, device=dev)
    gf = gf.to(torch.bfloat16)
    a, b = dt8.new_state(nflat, B, True, dev), dt8.new_state(nflat, B, False, dev)

    def flat():
        k[0] += 1
        dt8.dt8_adam_step(wf, gf, a[0], a[1], b[0], b[1], 1e-3, 0.9, 0.999, 1e-8, 0.05, k[0], B)
    report(f"  one flat tensor of {nflat} elts, bf16 grads (in L2)", timeit(flat, 200),
           nflat * 14 + 16 * (nflat // B))

    ps = synth.conv_sgd_params(1, dev)
    gs = synth.conv_sgd_grads(1, 1, dev)
    sm = [dt8.new_state(p.numel(), B, True, dev) for p in ps]
    prepared_sgd = dt8.PreparedTensorList(ps, gs, [s[0] for s in sm], [s[1] for s in sm])

    def sgd_launch():
        k[0] += 1
        prepared_sgd.sgd_step(0.1, 0.9, 1e-4, k[0], B)
    tot = sum(p.numel() for p in ps)
    nbk = sum(dt8.num_blocks(p.numel(), B) for p in ps)
    report(f"sgd, {len(ps)}-tensor list, {tot} elts, fp32 grads (in L2)", timeit(sgd_launch, 200),
           tot * 14 + 8 * nbk)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("cases", nargs="*", default=ALL)
    ap.add_argument("--peak", type=float, default=None,
                    help="reference bandwidth in GB/s (default: hbm_gbs of MEASURED_PEAKS.json at the "
                         "repository root if present, else 6650)")
    args = ap.parse_args()
    if args.peak is None:
        here = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
        try:
            with open(os.path.join(here, "MEASURED_PEAKS.json")) as fh:
                args.peak = float(json.load(fh)["hbm_gbs"])
        except Exception:
            args.peak = 6650.0
    if not torch.cuda.is_available():
        raise RuntimeError("needs a CUDA device: the dt8 library has no CPU path")
    dev = torch.device("cuda", torch.cuda.current_device())
    dt8.dt8_init()
    report = Report(args.peak)
    f32, bf16 = torch.float32, torch.bfloat16
    for case in args.cases:
        if case == "adam":
            adam_case(report, dev, 1 << 28, f32, "adam fp32 grads n=2^28 B=2048")
        elif case == "adam26":
            adam_case(report, dev, 1 << 26, f32, "adam fp32 grads n=2^26 B=2048")
        elif case == "adambf":
            adam_case(report, dev, 1 << 28, bf16, "adam bf16 grads n=2^28 B=2048")
        elif case == "adambf26":
            adam_case(report, dev, 1 << 26, bf16, "adam bf16 grads n=2^26 B=2048")
        elif case == "adaml2":
            adam_case(report, dev, 1 << 28, f32, "adam fp32 grads, coupled decay (IEEE path) n=2^28",
                      flags=dt8.DT8_ADAM_BIAS_CORRECTION)
        elif case == "adaml226":
            adam_case(report, dev, 1 << 26, f32, "adam fp32 grads, coupled decay (IEEE path) n=2^26",
                      flags=dt8.DT8_ADAM_BIAS_CORRECTION)
        elif case == "sgd":
            sgd_case(report, dev, 1 << 28, f32, "sgd fp32 grads n=2^28 B=2048")
        elif case == "sgd26":
            sgd_case(report, dev, 1 << 26, f32, "sgd fp32 grads n=2^26 B=2048")
        elif case == "sgdbf":
            sgd_case(report, dev, 1 << 28, bf16, "sgd bf16 grads n=2^28 B=2048")
        elif case == "blocks":
            for block in (256, 512, 1024, 4096):
                adam_case(report, dev, 1 << 27, f32, f"adam fp32 grads n=2^27 B={block}", block)
            for block in (256, 512, 1024, 4096):
                sgd_case(report, dev, 1 << 27, f32, f"sgd fp32 grads n=2^27 B={block}", block)
        elif case == "quant":
            quant_cases(report, dev)
        elif case == "dequant":
            dequant_cases(report, dev)
        elif case == "multi":
            multi_cases(report, dev)
        else:
            raise SystemExit(f"unknown case {case!r}; choose from {ALL}")


if __name__ == "__main__":
    main()

"""8-bit Adam step for tensors that live in pinned HOST memory.

Parameters, gradients and the 8-bit states stay on the host; the step streams them through the
GPU in chunks of whole quantization blocks.  Blocks are independent (Section IV-B: every block is
quantized on its own) and the update is element-wise, so cutting the tensor into chunks changes
nothing in the result.  Three CUDA streams overlap the host->device copies of chunk i+1, the
kernel on chunk i and the device->host copies of chunk i-1; the device holds only `buffers`
chunk-sized buffer sets, whatever the size of the tensor.
"""
from __future__ import annotations

from typing import List

import torch

import paper_2412_01195_b200 as dt8


class StreamedAdam8bit:
    """Chunked, pipelined `dt8_adam_step` over host-resident tensors.

    chunk_elems is rounded down to a multiple of block_size.  All host tensors passed to `step`
    must be pinned (page-locked) for the copies to be asynchronous."""

    def __init__(self, block_size: int = 2048, chunk_elems: int = 1 << 24, buffers: int = 3,
                 grad_dtype=torch.float32, device="cuda"):
        if block_size not in dt8.BLOCK_SIZES:
            raise ValueError("unsupported block size")
        self.B = block_size
        self.chunk = max(block_size, (chunk_elems // block_size) * block_size)
        self.device = torch.device(device)
        nb = self.chunk // block_size
        self.sets: List[dict] = []
        for _ in range(max(2, buffers)):
            self.sets.append(dict(
                w=torch.empty(self.chunk, dtype=torch.float32, device=self.device),
                g=torch.empty(self.chunk, dtype=grad_dtype, device=self.device),
                mc=torch.empty(self.chunk, dtype=torch.uint8, device=self.device),
                ma=torch.empty(nb, dtype=torch.float32, device=self.device),
                rc=torch.empty(self.chunk, dtype=torch.uint8, device=self.device),
                ra=torch.empty(nb, dtype=torch.float32, device=self.device),
                loaded=torch.cuda.Event(), stepped=torch.cuda.Event(), drained=torch.cuda.Event()))
        self.s_in = torch.cuda.Stream(self.device)
        self.s_step = torch.cuda.Stream(self.device)
        self.s_out = torch.cuda.Stream(self.device)
        dt8.dt8_init(self.device)
        self.h2d_bytes = 0
        self.d2h_bytes = 0

    def step(self, w, g, m_codes, m_absmax, r_codes, r_absmax, lr, beta1, beta2, eps, weight_decay,
             step, flags=dt8.DEFAULT_ADAM_FLAGS) -> None:
        """One step over host tensors (w, g, codes: n elements; absmax: ceil(n / B) floats),
        in place.  Ordered after the work already queued on the current stream; when it returns,
        the current stream waits for the last device->host copy."""
        n, B = w.numel(), self.B
        for t in (w, g, m_codes, m_absmax, r_codes, r_absmax):
            if t.is_cuda or not t.is_contiguous():
                raise TypeError("host, contiguous tensors are required")
        if g.dtype != self.sets[0]["g"].dtype:
            raise TypeError("g: the gradient dtype this object was built for is required")
        dt8._check_layout("StreamedAdam8bit.step", n, B, w.device,
                          {"g": g, "m_codes": m_codes, "r_codes": r_codes},
                          {"m_absmax": m_absmax, "r_absmax": r_absmax})
        cur = torch.cuda.current_stream(self.device)
        start = torch.cuda.Event()
        start.record(cur)
        for s in (self.s_in, self.s_step, self.s_out):
            s.wait_event(start)
        self.h2d_bytes = self.d2h_bytes = 0
        used = []
        for i, lo in enumerate(range(0, n, self.chunk)):
            hi = min(n, lo + self.chunk)
            cnt = hi - lo
            blo, bhi = lo // B, (hi + B - 1) // B
            bs = self.sets[i % len(self.sets)]
            dev = dict(w=bs["w"][:cnt], g=bs["g"][:cnt], mc=bs["mc"][:cnt], ma=bs["ma"][:bhi - blo],
                       rc=bs["rc"][:cnt], ra=bs["ra"][:bhi - blo])
            host = dict(w=w[lo:hi], g=g[lo:hi], mc=m_codes[lo:hi], ma=m_absmax[blo:bhi],
                        rc=r_codes[lo:hi], ra=r_absmax[blo:bhi])
            with torch.cuda.stream(self.s_in):
                if i >= len(self.sets):
                    self.s_in.wait_event(bs["drained"])          # the buffer set is free again
                for k in ("w", "g", "mc", "ma", "rc", "ra"):
                    dev[k].copy_(host[k], non_blocking=True)
                    self.h2d_bytes += host[k].numel() * host[k].element_size()
                bs["loaded"].record(self.s_in)
            self.s_step.wait_event(bs["loaded"])
            dt8.dt8_adam_step(dev["w"], dev["g"], dev["mc"], dev["ma"], dev["rc"], dev["ra"], lr,
                              beta1, beta2, eps, weight_decay, step, B, flags, stream=self.s_step)
            bs["stepped"].record(self.s_step)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(bs["stepped"])
                for k in ("w", "mc", "ma", "rc", "ra"):
                    host[k].copy_(dev[k], non_blocking=True)
                    self.d2h_bytes += host[k].numel() * host[k].element_size()
                bs["drained"].record(self.s_out)
            used.append(bs)
        for bs in used[-len(self.sets):]:
            cur.wait_event(bs["drained"])

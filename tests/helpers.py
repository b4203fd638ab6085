"""Shared helpers of the GPU parity tests: tolerances and CPU-checker / CUDA-library runners."""
from __future__ import annotations

import os

import numpy as np
import torch

import oracle
import paper_2412_01195_b200 as dt8

F = np.float32


def use_all_cores():
    oracle.set_threads(os.cpu_count() or 1)


def assert_params_close(got: np.ndarray, ref: np.ndarray, rel: float = 1e-6):
    """|got - ref| <= rel*|ref| + rel*rms(ref), element by element (the floor covers ref ~ 0)."""
    ref64 = ref.astype(np.float64)
    rms = float(np.sqrt(np.mean(ref64 * ref64))) if ref.size else 0.0
    err = np.abs(got.astype(np.float64) - ref64)
    bound = rel * np.abs(ref64) + rel * rms
    bad = np.nonzero(err > bound)[0]
    assert bad.size == 0, (f"{bad.size} of {ref.size} params outside {rel:g}: first at {bad[:5]}, "
                           f"got {got[bad[:5]]}, ref {ref[bad[:5]]}")


def assert_codes_match(got: np.ndarray, ref: np.ndarray, max_frac: float = 1e-5, exact: bool = True):
    """Bit-exact codes; with exact=False at most max_frac of them may be one code apart."""
    if exact:
        bad = np.nonzero(got != ref)[0]
        assert bad.size == 0, f"{bad.size} of {ref.size} codes differ, first at {bad[:5]}: {got[bad[:5]]} vs {ref[bad[:5]]}"
        return
    diff = np.abs(got.astype(np.int32) - ref.astype(np.int32))
    assert diff.max(initial=0) <= 1
    assert np.count_nonzero(diff) <= max_frac * max(ref.size, 1)


def assert_bf16_params_match(got: np.ndarray, ref: np.ndarray, max_frac: float = 0.0):
    """bfloat16 parameters as bit patterns: equal, except that at most max_frac of them may be the
    neighbouring bfloat16 value (the binary32 result of an approximate update can fall on the
    other side of a rounding boundary: about 3e-6 of the elements per step for N(0, 0.02)
    parameters, and a parameter that landed on the other side stays there).  Two elements are
    allowed on top of the fraction so that small tensors do not fail on a single such element."""
    assert got.dtype == np.uint16 and ref.dtype == np.uint16
    bad = np.nonzero(got != ref)[0]
    if bad.size == 0:
        return
    allowed = max_frac * ref.size + (2 if max_frac > 0 else 0)
    assert bad.size <= allowed, f"{bad.size} of {ref.size} bf16 params differ (allowed {allowed:g})"
    # apart by at most one bfloat16 ulp of the larger magnitude, plus the floor of the binary32
    # bound (1e-6 of the rms: where the update cancels the parameter, the tiny result carries the
    # absolute error of the update term)
    wide = lambda u: (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    g, r = wide(got[bad]), wide(ref[bad])
    rms = float(np.sqrt(np.mean(wide(ref) ** 2)))
    assert np.all(np.abs(g - r) <= 2.0 ** -7 * np.maximum(np.abs(g), np.abs(r)) + 1e-6 * rms)


def to_np(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.detach().cpu().view(torch.int16).numpy().view(np.uint16).copy()
    return t.detach().cpu().numpy().copy()


class AdamState:
    """One tensor's parameters and 8-bit Adam state, held both on the GPU and for the checker."""

    def __init__(self, w0: torch.Tensor, B: int, device="cuda"):
        n = w0.numel()
        self.n, self.B = n, B
        self.w_gpu = w0.to(device).clone()
        self.mc_gpu, self.ma_gpu = dt8.new_state(n, B, True, device)
        self.rc_gpu, self.ra_gpu = dt8.new_state(n, B, False, device)
        self.w = to_np(w0)
        nb = oracle.num_blocks(n, B)
        self.mc, self.ma = np.full(n, 127, np.uint8), np.zeros(nb, F)
        self.rc, self.ra = np.zeros(n, np.uint8), np.zeros(nb, F)

    def step(self, g: torch.Tensor, step: int, hp: dict, flags=dt8.DEFAULT_ADAM_FLAGS):
        g_gpu = g.to(self.w_gpu.device)
        dt8.dt8_adam_step(self.w_gpu, g_gpu, self.mc_gpu, self.ma_gpu, self.rc_gpu, self.ra_gpu,
                          hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], step,
                          self.B, flags)
        oracle.adam_step(self.w, to_np(g), self.mc, self.ma, self.rc, self.ra, hp["lr"], hp["beta1"],
                         hp["beta2"], hp["eps"], hp["weight_decay"], step, self.B, flags)

    def check(self, rel=1e-6, exact_params=False):
        torch.cuda.synchronize()
        if self.n == 0:
            return
        assert np.array_equal(to_np(self.ma_gpu), self.ma), "m absmax differs"
        assert np.array_equal(to_np(self.ra_gpu), self.ra), "r absmax differs"
        assert_codes_match(to_np(self.mc_gpu), self.mc)
        assert_codes_match(to_np(self.rc_gpu), self.rc)
        if self.w.dtype == np.uint16:
            got = to_np(self.w_gpu)
            assert_bf16_params_match(got, self.w, 0.0 if exact_params else 1e-4)
            # a parameter that fell on the other side of a rounding boundary keeps that distance
            # in later steps; the checker continues from the GPU's parameters so that every step
            # is compared from identical inputs
            self.w[:] = got
        elif exact_params:
            assert np.array_equal(to_np(self.w_gpu), self.w)
        else:
            assert_params_close(to_np(self.w_gpu), self.w, rel)


class SgdState:
    def __init__(self, w0: torch.Tensor, B: int, device="cuda"):
        n = w0.numel()
        self.n, self.B = n, B
        self.w_gpu = w0.to(device).clone()
        self.mc_gpu, self.ma_gpu = dt8.new_state(n, B, True, device)
        self.w = to_np(w0)
        self.mc, self.ma = np.full(n, 127, np.uint8), np.zeros(oracle.num_blocks(n, B), F)

    def step(self, g: torch.Tensor, step: int, hp: dict):
        dt8.dt8_sgd_step(self.w_gpu, g.to(self.w_gpu.device), self.mc_gpu, self.ma_gpu, hp["lr"],
                         hp["momentum"], hp["weight_decay"], step, self.B)
        oracle.sgd_step(self.w, to_np(g), self.mc, self.ma, hp["lr"], hp["momentum"],
                        hp["weight_decay"], step, self.B)

    def check(self):
        torch.cuda.synchronize()
        if self.n == 0:
            return
        assert np.array_equal(to_np(self.ma_gpu), self.ma), "m absmax differs"
        assert_codes_match(to_np(self.mc_gpu), self.mc)
        assert np.array_equal(to_np(self.w_gpu), self.w), "SGD params are computed with IEEE ops: bit-exact"

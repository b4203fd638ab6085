"""Seeded random configurations of the fused steps and of quantize / dequantize against the CPU
checker, through the C ABI: sizes around block multiples, every block size, both gradient types,
all four flag combinations, hyper-parameters over many decades, per-block magnitudes spread over
up to fifty decades, blocks of zeros and scattered zeros.  States (codes and block maxima) must be
equal; parameters equal where the update is made of correctly rounded operations, within the
documented tolerance of the approximate update otherwise."""
import numpy as np
import pytest
import torch

import oracle
import paper_2412_01195_b200 as dt8
from helpers import AdamState, SgdState, to_np, use_all_cores

pytestmark = pytest.mark.gpu
F = np.float32


@pytest.fixture(scope="module", autouse=True)
def _setup():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    dt8.dt8_init()
    use_all_cores()
    yield
    torch.cuda.synchronize()


def _block_scales(rng, n, B, spread, top):
    nb = (n + B - 1) // B
    scale = np.repeat(10.0 ** rng.uniform(-spread, min(spread, top), nb), B)[:n].astype(F)
    if rng.random() < 0.3:
        scale[rng.integers(0, nb) * B:][:B] = 0.0          # a block of zeros
    if rng.random() < 0.3:
        scale[rng.random(n) < 0.2] = 0.0
    if rng.random() < 0.2:
        scale[::7] *= F(1e-9)
    return scale


def _size(rng, B, max_blocks):
    return max(1, int(rng.integers(1, max_blocks)) * B + int(rng.choice([0, 0, 1, 3, B // 2, B - 1, -1, -B + 1])))


@pytest.mark.parametrize("chunk", range(8))
def test_random_step_configurations(chunk):
    checked = 0
    for seed in range(9000 + 60 * chunk, 9000 + 60 * (chunk + 1)):
        rng = np.random.default_rng(seed)
        B = int(rng.choice(dt8.BLOCK_SIZES))
        n = _size(rng, B, 24)
        gdt = torch.bfloat16 if rng.random() < 0.3 else torch.float32
        scale = _block_scales(rng, n, B, int(rng.choice([0, 3, 12, 25])), 15)
        t0, steps = int(rng.choice([1, 1, 7, 1000, 200000])), int(rng.integers(1, 5))
        if rng.random() < 0.67:
            flags = int(rng.choice([0, 1, 2, 3, 3, 3]))
            positive = scale[scale > 0]
            eps_choices = [1e-12, 1e-8, 1e-8, 1e-3, 1.0, 1e13, 1e14] + ([0.0] if positive.size and positive.min() > 1e-9 else [])
            hp = dict(lr=float(10 ** rng.uniform(-6, -1)), beta1=float(rng.choice([0.0, 0.5, 0.9, 0.99])),
                      beta2=float(rng.choice([0.0, 0.9, 0.999, 0.9999])), eps=float(rng.choice(eps_choices)),
                      weight_decay=float(rng.choice([0.0, 1e-4, 0.01, 0.5])))
            if rng.random() < 0.1:
                hp["lr"] = float(rng.choice([1e-25, 1e-21]))      # outside the approximate update's range
            if hp["eps"] == 0.0:
                scale = np.where(scale == 0, F(1.0), scale)         # no 0 / 0 in the update
            w0 = torch.from_numpy((rng.standard_normal(n) * 0.05).astype(F) * np.where(scale > 0, scale, F(1)))
            st = AdamState(w0, B)
            for k in range(steps):
                offset = 0.0 if hp["eps"] else 1e-3                  # eps = 0: no gradient of exactly 0
                g = torch.from_numpy(((rng.standard_normal(n) + offset) * 0.01).astype(F) * scale).to(gdt)
                st.step(g, t0 + k, hp, flags)
            finite = np.all(np.isfinite(st.w)) and np.all(np.isfinite(st.ma)) and np.all(np.isfinite(st.ra))
            exact = (not (flags & dt8.DT8_ADAM_DECOUPLED_WD) and hp["weight_decay"] != 0.0) or hp["lr"] < 1e-20
            if finite:
                # the approximate update's error is relative to the update term, which can be much
                # larger than a parameter it nearly cancels: 1e-5 of the parameters' scale
                st.check(rel=1e-5, exact_params=exact)
                checked += 1
        else:
            hp = dict(lr=float(10 ** rng.uniform(-5, 0)), momentum=float(rng.choice([0.0, 0.5, 0.9, 0.99])),
                      weight_decay=float(rng.choice([0.0, 1e-4, 0.01])))
            w0 = torch.from_numpy((rng.standard_normal(n) * 0.05).astype(F) * np.where(scale > 0, scale, F(1)))
            st = SgdState(w0, B)
            for k in range(steps):
                st.step(torch.from_numpy((rng.standard_normal(n) * 0.01).astype(F) * scale).to(gdt), t0 + k, hp)
            if np.all(np.isfinite(st.w)) and np.all(np.isfinite(st.ma)):
                st.check()
                checked += 1
    assert checked >= 40       # non-finite outcomes (outside the contract) are rare


@pytest.mark.parametrize("chunk", range(4))
def test_random_quantize_configurations(chunk):
    for seed in range(9600 + 60 * chunk, 9600 + 60 * (chunk + 1)):
        rng = np.random.default_rng(seed)
        B = int(rng.choice(dt8.BLOCK_SIZES))
        n = _size(rng, B, 40)
        signed = bool(rng.random() < 0.5)
        scale = _block_scales(rng, n, B, int(rng.choice([0, 5, 30, 44])), 37)
        x = np.nan_to_num((rng.laplace(size=n) * scale).astype(F), posinf=3e38, neginf=-3e38)
        if not signed:
            x = np.abs(x)
        codes, absmax = dt8.dt8_quantize_blockwise(torch.from_numpy(x).cuda(), B, signed)
        out = dt8.dt8_dequantize_blockwise(codes, absmax, B, signed)
        rc, ra = oracle.quantize_blockwise(x, B, signed)
        assert np.array_equal(to_np(absmax), ra), seed
        assert np.array_equal(to_np(codes), rc), seed
        assert np.array_equal(to_np(out).view(np.uint32), oracle.dequantize_blockwise(rc, ra, B, signed).view(np.uint32)), seed

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


@pytest.mark.parametrize("chunk", range(3))
def test_random_pointer_lists(chunk):
    """Lists of 1 to 300 tensors of random sizes (empty and tiny ones, whole blocks, ragged tails),
    Adam or SGD, either gradient type: the pointer-list launch equals the checker tensor by tensor."""
    for seed in range(9900 + 8 * chunk, 9900 + 8 * (chunk + 1)):
        rng = np.random.default_rng(seed)
        B = int(rng.choice(dt8.BLOCK_SIZES))
        count = int(rng.choice([1, 2, 17, 120, 257, 300]))
        kinds = rng.integers(0, 4, count)
        sizes = [0 if k == 0 and rng.random() < 0.2 else
                 int(rng.integers(1, 65)) if k <= 1 else
                 int(rng.integers(1, 4)) * B if k == 2 else
                 int(rng.integers(1, 3 * B)) for k in kinds]
        gdt = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        adam = bool(rng.random() < 0.6)
        steps = int(rng.integers(1, 4))
        ws = [torch.from_numpy((rng.standard_normal(n) * 0.05).astype(F)) for n in sizes]
        if adam:
            hp = (float(10 ** rng.uniform(-4, -2)), 0.9, 0.999, 1e-8, float(rng.choice([0.0, 0.01])))
            flags = int(rng.choice([1, 3, 3]))
            sts = [AdamState(w, B) for w in ws]
        else:
            hp = (float(10 ** rng.uniform(-3, -1)), 0.9, float(rng.choice([0.0, 1e-4])))
            sts = [SgdState(w, B) for w in ws]
        for t in range(1, steps + 1):
            gs = [torch.from_numpy((rng.standard_normal(n) * 0.01).astype(F)).to(gdt) for n in sizes]
            gg = [g.cuda() for g in gs]
            if adam:
                dt8.dt8_adam_step_multi([s.w_gpu for s in sts], gg, [s.mc_gpu for s in sts], [s.ma_gpu for s in sts],
                                        [s.rc_gpu for s in sts], [s.ra_gpu for s in sts], *hp, t, B, flags)
                for s, g in zip(sts, gs):
                    oracle.adam_step(s.w, to_np(g), s.mc, s.ma, s.rc, s.ra, *hp, t, B, flags)
            else:
                dt8.dt8_sgd_step_multi([s.w_gpu for s in sts], gg, [s.mc_gpu for s in sts], [s.ma_gpu for s in sts],
                                       *hp, t, B)
                for s, g in zip(sts, gs):
                    oracle.sgd_step(s.w, to_np(g), s.mc, s.ma, *hp, t, B)
        for s in sts:
            if adam:
                s.check(rel=1e-5, exact_params=not (flags & dt8.DT8_ADAM_DECOUPLED_WD) and hp[4] != 0.0)
            else:
                s.check()


def test_random_reversible_kernel_shapes():
    """Coupling halves and the invertible down-sampling on random N x C x F x T shapes (rows of any
    even length, so that every vector width and the small-plane path are met) against the checker,
    bit for bit, and each followed by its inverse."""
    from oracle import rev as orev
    from paper_2412_01195_b200 import rev
    for seed in range(9950, 9990):
        rng = np.random.default_rng(seed)
        N, C = int(rng.integers(1, 5)), 2 * int(rng.integers(1, 7))
        Fd, T = 2 * int(rng.integers(1, 13)), 2 * int(rng.integers(1, 60))
        x = rng.standard_normal((N, C, Fd, T)).astype(F)
        t = rng.standard_normal((N, C // 2, Fd, T)).astype(F)
        which = int(rng.integers(0, 2))
        xg, tg = torch.from_numpy(x).cuda(), torch.from_numpy(t).cuda()
        yg = xg.clone()
        rev.dt8_rev_coupling_forward(xg, tg, yg, which)
        y = x.copy()
        orev.couple_half(x, t, y, which, +1)
        assert np.array_equal(to_np(yg), y), seed
        back = yg.clone()
        rev.dt8_rev_coupling_inverse(yg, tg, back, which)
        ref_back = y.copy()
        orev.couple_half(y, t, ref_back, which, -1)
        assert np.array_equal(to_np(back), ref_back), seed
        deep = rev.dt8_rev_space_to_depth(xg)
        assert np.array_equal(to_np(deep), orev.space_to_depth(x)), seed
        assert torch.equal(rev.dt8_rev_depth_to_space(deep), xg), seed

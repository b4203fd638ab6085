"""Parity of the CUDA library against the CPU checker, through the C ABI (via the thin binding).

Same seeded inputs on both sides; integer results (codes) and absmax bit-exact, parameters within
1e-6 relative (mixed with an rms floor), 100-step trajectories within 1e-4."""
import numpy as np
import pytest
import torch

import oracle
import paper_2412_01195_b200 as dt8
from paper_2412_01195_b200 import synth
from helpers import (AdamState, SgdState, assert_codes_match, assert_params_close, to_np,
                     use_all_cores)

pytestmark = pytest.mark.gpu
F = np.float32
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _setup():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    dt8.dt8_init()
    use_all_cores()
    yield
    torch.cuda.synchronize()


# ------------------------------------------------------------------------------------------------
# quantize / dequantize
# ------------------------------------------------------------------------------------------------
def quant_roundtrip_check(x: torch.Tensor, B: int, signed: bool):
    codes, absmax = dt8.dt8_quantize_blockwise(x.to(DEV), B, signed)
    out = dt8.dt8_dequantize_blockwise(codes, absmax, B, signed)
    torch.cuda.synchronize()
    rc, ra = oracle.quantize_blockwise(to_np(x), B, signed)
    assert np.array_equal(to_np(absmax), ra)
    assert_codes_match(to_np(codes), rc)
    assert np.array_equal(to_np(out), oracle.dequantize_blockwise(rc, ra, B, signed))


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("B", [256, 512, 1024, 2048, 4096])
def test_quantize_dequantize_sizes_and_tails(B, signed):
    for n in (1, 3, 4, 5, B - 1, B, B + 1, 2 * B + 3, 37 * B + B // 2 + 1, 300 * B + 7):
        x = synth.laplace_outliers(n, seed=300 + n % 97)
        if not signed:
            x = x.abs()
        quant_roundtrip_check(x, B, signed)


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("B", [256, 2048])
def test_quantize_blocks_of_every_magnitude(B, signed):
    """Block maxima from subnormal to close to the largest binary32 number, with the edges of the
    range of the reciprocal-and-correct division (2^-76 = 1.3e-23, 2^100 = 1.3e30) on both sides,
    a block of zeros, and blocks that mix a large maximum with values far below the smallest code."""
    scales = [1e-44, 1e-41, 1e-39, 1e-37, 1e-30, 1.2e-23, 1.4e-23, 1e-10, 1.0, 1e10, 1.2e30, 1.4e30,
              1e34, 3e37, 0.0]
    n = len(scales) * B
    x = synth.laplace_outliers(n, seed=350).clamp(-8, 8)
    for k, s in enumerate(scales):
        x[k * B:(k + 1) * B] *= s
    x[4 * B + 5] = 1e-5        # values 25 decades below the block maximum
    x[9 * B:10 * B:3] *= 1e-30
    if not signed:
        x = x.abs()
    quant_roundtrip_check(x, B, signed)


@pytest.mark.parametrize("signed", [True, False])
def test_quantize_sweep_configuration(signed):
    """Configuration 4 at its smaller sizes: Laplace(0,1) with 1e-3 outliers x100 (the 128M size is
    covered by sampled blocks in the full-size test)."""
    c = synth.QUANT_SWEEP
    for n in c["sizes"][:2]:
        x = synth.laplace_outliers(n, seed=c["seed"])
        x = x if signed else x.abs()
        for B in c["block_sizes"]:
            quant_roundtrip_check(x, B, signed)


def test_quantize_degenerate_blocks():
    B = 256
    x = torch.zeros(5 * B + 9)
    x[B:2 * B] = synth.normal(B, 1e-30, 1)            # tiny maximum: division outside the fast range
    x[2 * B:3 * B] = synth.normal(B, 1e30, 2)         # huge maximum
    x[3 * B:4 * B] = synth.normal(B, 1e-42, 3)        # subnormal block
    x[4 * B] = -7.0                                   # one non-zero element, negative
    for signed in (True, False):
        quant_roundtrip_check(x, B, signed)
    codes, absmax = dt8.dt8_quantize_blockwise(torch.zeros(B, device=DEV), B, True)
    assert torch.all(codes == 127) and torch.all(absmax == 0)
    codes, absmax = dt8.dt8_quantize_blockwise(torch.zeros(0, device=DEV), B, True)
    assert codes.numel() == 0 and absmax.numel() == 0
    # unsigned table with negative inputs: they take the value 0
    quant_roundtrip_check(synth.normal(3 * B + 1, 1.0, 4), B, False)


@pytest.mark.parametrize("signed", [True, False])
def test_quantize_follows_true_division(signed):
    """Inputs on which x/N and x*(1/N) fall on different codes (Eq. quant1 divides)."""
    Q = oracle.codebook(signed)
    Q64 = Q.astype(np.float64)
    mids = ((Q64[:-1] + Q64[1:]) / 2)[Q64[:-1] != Q64[1:]]
    mids = mids[mids > 0].astype(F)
    rng = np.random.default_rng(80)
    B = 256
    nblk = 4000
    N = rng.uniform(0.5, 2.0, nblk).astype(F)
    x = np.zeros((nblk, B), F)
    x[:, 0] = N
    T = rng.choice(mids, (nblk, B - 1))
    x[:, 1:] = (T * N[:, None]).astype(F)             # x / N within an ulp of a mid-point
    x[:, 1:] = np.minimum(np.abs(x[:, 1:]), N[:, None]) * (rng.choice([-1, 1], (nblk, B - 1)) if signed else 1)
    quant_roundtrip_check(torch.from_numpy(x.ravel()), B, signed)


def test_block_reciprocal_is_correctly_rounded_for_every_mantissa():
    """The residual correction of Eq. quant1's division is exact only from the correctly rounded
    reciprocal of the block maximum.  Inside 2^-76 .. 2^100 nothing in its computation overflows
    or underflows, so the mantissa decides: all 2^23 of them, at the two ends and in the middle
    of the range, against 1/N formed in binary64 and rounded once.  Outside the range, and for
    N = 0, the routine reports that it takes the IEEE division (0)."""
    man = np.arange(1 << 23, dtype=np.uint32)
    for e in (-76, -75, -1, 0, 1, 64, 99):
        N = (man | np.uint32((127 + e) << 23)).view(F)
        got = dt8.dt8_selfcheck_reciprocal(torch.from_numpy(N).to(DEV)).cpu().numpy()
        ref = (1.0 / N.astype(np.float64)).astype(F)
        bad = np.nonzero(got != ref)[0]
        assert bad.size == 0, (e, [float(x).hex() for x in N[bad[:4]]], got[bad[:4]], ref[bad[:4]])
    edge = np.array([2.0 ** 100, 2.0 ** -76], F)
    got = dt8.dt8_selfcheck_reciprocal(torch.from_numpy(edge).to(DEV)).cpu().numpy()
    assert np.array_equal(got, np.array([2.0 ** -100, 2.0 ** 76], F))
    outside = np.array([0.0, np.nextafter(F(2.0 ** 100), F(np.inf)), np.nextafter(F(2.0 ** -76), F(0)), 1e-40,
                        np.inf, np.nan, 3e38], F)
    got = dt8.dt8_selfcheck_reciprocal(torch.from_numpy(outside).to(DEV)).cpu().numpy()
    assert np.array_equal(got, np.zeros(outside.size, F))


def test_fast_root_is_correctly_rounded_for_every_mantissa_and_parity():
    """The IEEE form of Eq. adam's parameter update takes sqrt(r'/bc2); inside 2^-80 .. 2^80 the
    kernel forms it from a reciprocal-root approximation and one correction.  The outcome depends
    on the mantissa and on the parity of the exponent only: all 2^24 cases at the ends and in the
    middle of the range, against the root formed in binary64 and rounded once (a binary64 root of
    a binary32 number is never close enough to a binary32 rounding boundary for the second rounding
    to matter).  Outside the range the routine reports 0 (the step then uses the IEEE root)."""
    man = np.arange(1 << 23, dtype=np.uint32)
    for e in (-80, -79, -1, 0, 1, 2, 79):
        x = (man | np.uint32((127 + e) << 23)).view(F)
        got = dt8.dt8_selfcheck_root(torch.from_numpy(x).to(DEV)).cpu().numpy()
        ref = np.sqrt(x.astype(np.float64)).astype(F)
        bad = np.nonzero(got != ref)[0]
        assert bad.size == 0, (e, [float(v).hex() for v in x[bad[:4]]], got[bad[:4]], ref[bad[:4]])
    edge = np.array([2.0 ** 80, 2.0 ** -80], F)
    assert np.array_equal(dt8.dt8_selfcheck_root(torch.from_numpy(edge).to(DEV)).cpu().numpy(),
                          np.array([2.0 ** 40, 2.0 ** -40], F))
    outside = np.array([0.0, -1.0, np.nextafter(F(2.0 ** 80), F(np.inf)), np.nextafter(F(2.0 ** -80), F(0)),
                        np.inf, np.nan], F)
    assert np.array_equal(dt8.dt8_selfcheck_root(torch.from_numpy(outside).to(DEV)).cpu().numpy(),
                          np.zeros(outside.size, F))


def test_reciprocal_and_correct_division_for_quotients_of_any_size():
    """The same reciprocal-and-correct division serves Eq. adam's m-hat / (sqrt(r-hat) + eps) in
    the IEEE parameter update, where the dividend may exceed the divisor: dividends 2^-80 .. 2^80
    over divisors 2^-40 .. 2^46 (the ranges the step guarantees), against the quotient formed in
    binary64 and rounded once."""
    rng = np.random.default_rng(11)
    M = 1 << 23
    d = (rng.uniform(1, 2, M) * 2.0 ** rng.integers(-40, 46, M)).astype(F)
    a = (rng.uniform(1, 2, M) * 2.0 ** rng.integers(-80, 80, M) * rng.choice([-1.0, 1.0], M)).astype(F)
    # special mantissas of the divisor
    d[:1 << 20] = ((rng.integers(0, 1 << 23, 1 << 20).astype(np.uint32) | np.uint32(0x7FFF00)) & np.uint32(0x7FFFFF) | np.uint32(0x3F800000)).view(F)
    got = dt8.dt8_selfcheck_divide(torch.from_numpy(a).to(DEV), torch.from_numpy(d).to(DEV)).cpu().numpy()
    ref = (a.astype(np.float64) / d.astype(np.float64)).astype(F)
    assert np.array_equal(got, ref)


def test_normalising_division_is_correctly_rounded():
    """Eq. quant1 divides: the kernels' reciprocal-and-correct routine must give the correctly
    rounded quotient for every |s| <= N.  The true quotient is formed in binary64 and rounded once
    (a quotient of two binary32 numbers never sits on a binary32 rounding boundary, so the double
    rounding is exact).  Scaling s or N by a power of two only shifts exponents, so the operand
    space is (mantissa of N) x (mantissa of s, two binades): all 2^23 mantissas of s are swept for
    N with all-ones, all-zeros, sparse and random mantissas."""
    rng = np.random.default_rng(5)
    man_n = np.concatenate([
        np.array([0, 1, 2, 3, 0x7FFFFF, 0x7FFFFE, 0x7FFFFD, 0x400000, 0x400001, 0x3FFFFF, 0x555555,
                  0x2AAAAA, 0x7FF000, 0x000FFF, 0x600000, 0x200000], np.uint32),
        rng.integers(0, 1 << 23, 24).astype(np.uint32)])
    man_s = np.arange(1 << 23, dtype=np.uint32)
    for mn in man_n:
        N = np.array([0x3F800000 | int(mn)], np.uint32).view(F)[0]
        for expo in (0x3F800000, 0x3F000000):                 # s in [1, 2) and [0.5, 1)
            s = (man_s | np.uint32(expo)).view(F)
            s = s[s <= N]
            if s.size == 0:
                continue
            got = dt8.dt8_selfcheck_divide(torch.from_numpy(s).to(DEV),
                                           torch.full((s.size,), float(N), device=DEV)).cpu().numpy()
            ref = (s.astype(np.float64) / np.float64(N)).astype(F)
            bad = np.nonzero(got != ref)[0]
            assert bad.size == 0, (float(N).hex(), [float(x).hex() for x in s[bad[:4]]], got[bad[:4]], ref[bad[:4]])
    # random operands over the whole exponent range, the IEEE branch (tiny and huge N) included
    M = 1 << 22
    Nr = (rng.uniform(1, 2, M) * 2.0 ** rng.integers(-120, 120, M)).astype(F)
    sr = np.minimum((Nr.astype(np.float64) * rng.uniform(-1, 1, M)).astype(F), Nr)
    got = dt8.dt8_selfcheck_divide(torch.from_numpy(sr).to(DEV), torch.from_numpy(Nr).to(DEV)).cpu().numpy()
    with np.errstate(under="ignore"):
        ref = (sr.astype(np.float64) / Nr.astype(np.float64)).astype(F)
    assert np.array_equal(got, ref)
    # all-zero block: 0 / 0 is taken as 0
    z = torch.zeros(8, device=DEV)
    assert torch.count_nonzero(dt8.dt8_selfcheck_divide(z, z)).item() == 0


@pytest.mark.parametrize("signed", [True, False])
def test_encoder_over_a_strided_sweep_of_all_floats(signed):
    """Blocks whose maximum is exactly 1, so the normalised value is the input itself: every 13th
    binary32 bit pattern in [0, 1] (and its negative for the signed table)."""
    Q = oracle.codebook(signed)
    B = 256
    bits = np.arange(0, 0x3F800000, 13, dtype=np.uint32)
    bits = bits[: (bits.size // (B - 1)) * (B - 1)].reshape(-1, B - 1)
    for sign in ((0, 0x80000000) if signed else (0,)):
        x = np.empty((bits.shape[0], B), np.uint32)
        x[:, 0] = 0x3F800000
        x[:, 1:] = bits | np.uint32(sign)
        xf = x.view(F).ravel()
        codes, absmax = dt8.dt8_quantize_blockwise(torch.from_numpy(xf).to(DEV), B, signed)
        torch.cuda.synchronize()
        assert torch.all(absmax == 1.0)
        assert_codes_match(to_np(codes), oracle.nearest(Q, xf))


def test_dequantize_every_code_and_scale():
    for signed in (True, False):
        for N in (1.0, 3.7e-5, 2.0 ** -20, 1e4, 0.0):
            codes = torch.arange(256, dtype=torch.uint8, device=DEV)
            absmax = torch.tensor([N], dtype=torch.float32, device=DEV)
            out = dt8.dt8_dequantize_blockwise(codes, absmax, 256, signed)
            ref = oracle.dequantize_blockwise(np.arange(256, dtype=np.uint8), np.array([N], F), 256, signed)
            assert np.array_equal(to_np(out).view(np.uint32), ref.view(np.uint32))


# ------------------------------------------------------------------------------------------------
# Adam
# ------------------------------------------------------------------------------------------------
def test_adam_configuration_1():
    """1,048,576 elements, one AdamW step from the zero state (lr 1e-3, betas 0.9/0.999, wd 0)."""
    c = synth.ADAM_FLAT_SMALL
    w0, g = synth.flat_adam_inputs(c["n"], c["seed"])
    st = AdamState(w0, c["block_size"])
    st.step(g, 1, c)
    st.check()
    # closed form of the first step, straight from the inputs
    g64 = g.numpy().astype(np.float64)
    want = w0.numpy().astype(np.float64) - c["lr"] * g64 / (np.abs(g64) + c["eps"])
    assert np.max(np.abs(to_np(st.w_gpu) - want)) <= 4e-7 * np.max(np.abs(want)) + 1e-10


@pytest.mark.parametrize("B", [256, 512, 1024, 2048, 4096])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_adam_steps_all_block_sizes(B, gdtype):
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    for n in (1, B - 3, 5 * B + 11, 150 * B + B // 2):
        st = AdamState(synth.normal(n, 0.02, 400 + B), B)
        for t in range(1, 6):
            st.step(synth.fresh_grad(n, 41, t, dtype=gdtype), t, hp)
            st.check()


def test_adam_trajectory_100_steps():
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    n, B = 200 * 2048 + 777, 2048
    st = AdamState(synth.normal(n, 0.02, 500), B)
    for t in range(1, 101):
        st.step(synth.fresh_grad(n, 42, t), t, hp)
        if t in (1, 2, 10, 50):
            st.check()
    st.check(rel=1e-4)
    st.check(rel=1e-6)


@pytest.mark.parametrize("flags", [0, dt8.DT8_ADAM_BIAS_CORRECTION, dt8.DT8_ADAM_DECOUPLED_WD])
def test_adam_variants(flags):
    """Literal Eq. adam (no bias correction), coupled L2 decay (IEEE parameter path: bit-exact)."""
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.05)
    n, B = 33 * 2048 + 5, 2048
    st = AdamState(synth.normal(n, 0.02, 600), B)
    for t in range(1, 21):
        st.step(synth.fresh_grad(n, 43, t), t, hp, flags)
    st.check(exact_params=not (flags & dt8.DT8_ADAM_DECOUPLED_WD))


def test_adam_literal_equation_without_decay_and_tiny_eps():
    """Eq. adam exactly as printed (no bias correction, no decay) takes the fast parameter path
    (1e-6); an eps too small to hide a flushed subnormal root takes the forms of the root and
    reciprocal that keep subnormals (1e-6 as well); a learning rate outside the range of the
    approximate paths takes IEEE operations (bit-exact parameters)."""
    n, B = 21 * 2048 + 77, 2048
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    st = AdamState(synth.normal(n, 0.02, 610), B)
    for t in range(1, 11):
        st.step(synth.fresh_grad(n, 44, t), t, hp, 0)
    st.check()
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-20, weight_decay=0.01)
    st = AdamState(synth.normal(n, 0.02, 611), B)
    for t in range(1, 6):
        g = synth.fresh_grad(n, 45, t)
        g[5 * B:6 * B] *= 1e-18                      # second moments down in the subnormal range
        g[6 * B:7 * B] = 0.0
        st.step(g, t, hp)
    st.check()
    hp = dict(lr=1e-25, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    st = AdamState(synth.normal(n, 0.02, 612), B)
    for t in range(1, 6):
        st.step(synth.fresh_grad(n, 46, t), t, hp)
    st.check(exact_params=True)


def test_adam_heavy_tailed_and_sparse_gradients():
    """Student-t gradients, zero gradients, and a block that stays all-zero."""
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    n, B = 20 * 2048, 2048
    st = AdamState(synth.normal(n, 0.02, 700), B)
    for t in range(1, 11):
        g = synth.student_t(n, 3, 1e-3, 7100 + t)
        g[3 * B:5 * B] = 0.0
        g[7 * B:8 * B] *= 1e-20
        g[9 * B + 5] = 50.0
        st.step(g, t, hp)
    st.check()
    assert np.all(st.ma[3:5] == 0) and np.all(to_np(st.ma_gpu)[3:5] == 0)


# ------------------------------------------------------------------------------------------------
# SGD
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("B", [256, 512, 1024, 2048, 4096])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_sgd_steps_all_block_sizes(B, gdtype):
    hp = dict(lr=0.1, momentum=0.9, weight_decay=1e-4)
    for n in (2, B + 1, 7 * B + 13, 120 * B + 1):
        st = SgdState(synth.normal(n, 0.05, 800 + B), B)
        for t in range(1, 6):
            g = synth.student_t(n, 3, 1e-3, 8100 + t)
            st.step(g.to(gdtype), t, hp)
            st.check()


def test_sgd_configuration_2_multi_tensor_100_steps():
    """37 conv3x3 weights (6,561,792 elements), Student-t gradients, momentum 0.9, wd 1e-4, lr 0.1,
    100 steps; the list is stepped in one launch and must equal the checker tensor by tensor."""
    c = synth.SGD_CONV
    B = c["block_size"]
    ws = synth.conv_sgd_params(c["seed"])
    sizes = [w.numel() for w in ws]
    assert sum(sizes) == 6_561_792 and len(sizes) == 37
    w_gpu = [w.to(DEV) for w in ws]
    st_gpu = [dt8.new_state(n, B, True, DEV) for n in sizes]
    w_ref = [to_np(w) for w in ws]
    mc_ref = [np.full(n, 127, np.uint8) for n in sizes]
    ma_ref = [np.zeros(oracle.num_blocks(n, B), F) for n in sizes]
    for t in range(1, c["steps"] + 1):
        gs = synth.conv_sgd_grads(c["seed"], t)
        dt8.dt8_sgd_step_multi(w_gpu, [g.to(DEV) for g in gs], [s[0] for s in st_gpu],
                               [s[1] for s in st_gpu], c["lr"], c["momentum"], c["weight_decay"], t, B)
        oracle.sgd_step_multi(w_ref, [to_np(g) for g in gs], mc_ref, ma_ref, c["lr"], c["momentum"],
                              c["weight_decay"], t, B)
        if t in (1, 2, 10, 100):
            torch.cuda.synchronize()
            for i in range(len(sizes)):
                assert np.array_equal(to_np(st_gpu[i][1]), ma_ref[i])
                assert_codes_match(to_np(st_gpu[i][0]), mc_ref[i])
                assert np.array_equal(to_np(w_gpu[i]), w_ref[i])


def test_adam_configuration_3_multi_tensor_100_steps():
    """~200 tensors of a ResNet speaker extractor, bf16 gradients, AdamW wd 0.05, 100 steps."""
    c = synth.ADAM_RESNET
    B = c["block_size"]
    ws = synth.resnet_adam_params(c["seed"])
    sizes = [w.numel() for w in ws]
    assert len(sizes) == 197 and 7.0e6 < sum(sizes) < 7.1e6 and min(sizes) == 32 and max(sizes) == 1_534_464
    w_gpu = [w.to(DEV) for w in ws]
    m_gpu = [dt8.new_state(n, B, True, DEV) for n in sizes]
    r_gpu = [dt8.new_state(n, B, False, DEV) for n in sizes]
    w_ref = [to_np(w) for w in ws]
    mc = [np.full(n, 127, np.uint8) for n in sizes]
    ma = [np.zeros(oracle.num_blocks(n, B), F) for n in sizes]
    rc = [np.zeros(n, np.uint8) for n in sizes]
    ra = [np.zeros(oracle.num_blocks(n, B), F) for n in sizes]
    for t in range(1, c["steps"] + 1):
        gs = synth.resnet_adam_grads(c["seed"], t)
        dt8.dt8_adam_step_multi(w_gpu, [g.to(DEV) for g in gs], [s[0] for s in m_gpu], [s[1] for s in m_gpu],
                                [s[0] for s in r_gpu], [s[1] for s in r_gpu], c["lr"], c["beta1"],
                                c["beta2"], c["eps"], c["weight_decay"], t, B)
        oracle.adam_step_multi(w_ref, [to_np(g) for g in gs], mc, ma, rc, ra, c["lr"], c["beta1"],
                               c["beta2"], c["eps"], c["weight_decay"], t, B)
        if t in (1, 3, 100):
            torch.cuda.synchronize()
            for i in range(len(sizes)):
                assert np.array_equal(to_np(m_gpu[i][1]), ma[i]) and np.array_equal(to_np(r_gpu[i][1]), ra[i])
                assert_codes_match(to_np(m_gpu[i][0]), mc[i])
                assert_codes_match(to_np(r_gpu[i][0]), rc[i])
                assert_params_close(to_np(w_gpu[i]), w_ref[i], 1e-4 if t == 100 else 1e-6)


def test_multi_equals_single_and_skips_empty_tensors():
    B = 512
    sizes = [0, 5, B, 3 * B + 1, 0, 70 * B + 9]
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.01)
    ws = [synth.normal(n, 0.02, 900 + i).to(DEV) for i, n in enumerate(sizes)]
    gs = [synth.normal(n, 1e-3, 950 + i).to(DEV) for i, n in enumerate(sizes)]
    a = [(w.clone(), *dt8.new_state(n, B, True, DEV), *dt8.new_state(n, B, False, DEV)) for w, n in zip(ws, sizes)]
    b = [(w.clone(), *dt8.new_state(n, B, True, DEV), *dt8.new_state(n, B, False, DEV)) for w, n in zip(ws, sizes)]
    for t in (1, 2, 3):
        dt8.dt8_adam_step_multi([x[0] for x in a], gs, [x[1] for x in a], [x[2] for x in a],
                                [x[3] for x in a], [x[4] for x in a], *hp, t, B)
        for x, g in zip(b, gs):
            dt8.dt8_adam_step(x[0], g, x[1], x[2], x[3], x[4], *hp, t, B)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        for u, v in zip(x, y):
            assert torch.equal(u, v)


def test_prepared_tensor_list_equals_the_per_call_form():
    """Pointer arrays marshalled once give the same steps as arrays rebuilt on every call."""
    B = 2048
    sizes = [33, B, 5 * B + 77, 256, 9 * B]
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.05)
    ws = [synth.normal(n, 0.02, 300 + i).to(DEV) for i, n in enumerate(sizes)]
    gs = [synth.normal(n, 1e-3, 350 + i, dtype=torch.bfloat16).to(DEV) for i, n in enumerate(sizes)]
    mk = lambda: [(w.clone(), *dt8.new_state(n, B, True, DEV), *dt8.new_state(n, B, False, DEV))
                  for w, n in zip(ws, sizes)]
    a, b = mk(), mk()
    col = lambda rows, k: [r[k] for r in rows]
    prepared = dt8.PreparedTensorList(col(a, 0), gs, col(a, 1), col(a, 2), col(a, 3), col(a, 4))
    for t in (1, 2, 3, 4):
        for g in gs:                                   # fresh gradients written in place
            g.copy_(synth.normal(g.numel(), 1e-3, 400 + t, dtype=torch.bfloat16))
        prepared.adam_step(*hp, t, B)
        dt8.dt8_adam_step_multi(col(b, 0), gs, col(b, 1), col(b, 2), col(b, 3), col(b, 4), *hp, t, B)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        for u, v in zip(x, y):
            assert torch.equal(u, v)
    sa, sb = mk(), mk()
    gf = [g.float() for g in gs]
    prepared = dt8.PreparedTensorList(col(sa, 0), gf, col(sa, 1), col(sa, 2))
    for t in (1, 2):
        prepared.sgd_step(0.1, 0.9, 1e-4, t, B)
        dt8.dt8_sgd_step_multi(col(sb, 0), gf, col(sb, 1), col(sb, 2), 0.1, 0.9, 1e-4, t, B)
    torch.cuda.synchronize()
    for x, y in zip(sa, sb):
        assert torch.equal(x[0], y[0]) and torch.equal(x[1], y[1]) and torch.equal(x[2], y[2])


def test_non_finite_gradients_stay_inside_their_block():
    """NaN / Inf are outside the contract, but they must not index outside the tables: a block
    that holds one gets a non-finite maximum and takes the clamped path of the encoder.  Blocks
    without one are unaffected (blocks are independent) and still match the CPU checker."""
    B, nblk = 2048, 24
    n = nblk * B
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    w0 = synth.normal(n, 0.02, 71)
    g1 = synth.normal(n, 1e-3, 72)
    g2 = synth.normal(n, 1e-3, 73)
    bad_blocks = {3: float("nan"), 7: float("inf"), 11: float("-inf"), 12: float("nan")}
    for blk, val in bad_blocks.items():
        g2[blk * B + 5 * blk] = val
    g2[12 * B + 1] = float("inf")
    st = AdamState(w0, B)
    st.step(g1, 1, hp)
    st.check()
    # second step with the poisoned gradient, on the GPU and in the checker
    g2_gpu = g2.to(DEV)
    dt8.dt8_adam_step(st.w_gpu, g2_gpu, st.mc_gpu, st.ma_gpu, st.rc_gpu, st.ra_gpu, hp["lr"],
                      hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], 2, B)
    w_sgd = w0.to(DEV).clone()
    mc, ma = dt8.new_state(n, B, True, DEV)
    dt8.dt8_sgd_step(w_sgd, g2_gpu, mc, ma, 0.1, 0.9, 1e-4, 1, B)
    codes, absmax = dt8.dt8_quantize_blockwise(g2_gpu, B, True)
    codes_u, _ = dt8.dt8_quantize_blockwise(g2_gpu, B, False)
    torch.cuda.synchronize()                          # all four kernels ran to completion
    with np.errstate(all="ignore"):
        oracle.adam_step(st.w, to_np(g2), st.mc, st.ma, st.rc, st.ra, hp["lr"], hp["beta1"],
                         hp["beta2"], hp["eps"], hp["weight_decay"], 2, B)
        q_ref, a_ref = oracle.quantize_blockwise(to_np(g2), B, True)
    good = np.ones(n, bool)
    for blk in bad_blocks:
        good[blk * B:(blk + 1) * B] = False
    good_blk = np.array([b not in bad_blocks for b in range(nblk)])
    assert np.array_equal(to_np(st.mc_gpu)[good], st.mc[good])
    assert np.array_equal(to_np(st.rc_gpu)[good], st.rc[good])
    assert np.array_equal(to_np(st.ma_gpu)[good_blk], st.ma[good_blk])
    assert np.array_equal(to_np(st.ra_gpu)[good_blk], st.ra[good_blk])
    assert_params_close(to_np(st.w_gpu)[good], st.w[good])
    assert np.array_equal(to_np(codes)[good], q_ref[good])
    assert np.array_equal(to_np(absmax)[good_blk], a_ref[good_blk])
    assert not np.isfinite(to_np(st.ma_gpu)[~good_blk]).any()
    assert codes_u.numel() == n


def test_sharded_adam_on_one_rank_equals_the_plain_step():
    """The block-range-sharded optimizer with a single rank (no process group) is the plain step
    on a zero-padded buffer."""
    from paper_2412_01195_b200.sharded import ShardedAdam8bit
    n, B = 13 * 2048 + 300, 2048
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.01)
    opt = ShardedAdam8bit(n, B, device=DEV)
    w0 = synth.normal(n, 0.02, 31).to(DEV)
    opt.params[:n].copy_(w0)
    w = torch.zeros(opt.padded, device=DEV)
    w[:n].copy_(w0)
    mc, ma = dt8.new_state(opt.padded, B, True, DEV)
    rc, ra = dt8.new_state(opt.padded, B, False, DEV)
    for t in (1, 2, 3):
        g = torch.zeros(opt.padded, device=DEV)
        g[:n].copy_(synth.fresh_grad(n, 32, t))
        opt.grads.copy_(g)
        opt.step(*hp)
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, *hp, t, B)
    torch.cuda.synchronize()
    assert torch.equal(opt.params, w) and torch.equal(opt.m_codes, mc) and torch.equal(opt.r_codes, rc)
    assert torch.equal(opt.m_absmax, ma) and torch.equal(opt.r_absmax, ra)


def test_streamed_host_resident_step_equals_the_device_resident_step():
    """Tensors in pinned host memory, streamed through the GPU in chunks of whole blocks on three
    streams: bit-identical to stepping the whole tensor on the device (blocks are independent)."""
    from paper_2412_01195_b200.offload import StreamedAdam8bit
    B = 512
    n = 37 * B + 123                              # 8 chunks of 5 blocks, the last one short and ragged
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.01)
    w0 = synth.normal(n, 0.02, 81)
    ref = [w0.to(DEV), None, *dt8.new_state(n, B, True, DEV), *dt8.new_state(n, B, False, DEV)]
    host = [w0.clone().pin_memory(), torch.empty(n).pin_memory()]
    host += [t.cpu().pin_memory() for t in ref[2:]]
    pipe = StreamedAdam8bit(B, chunk_elems=5 * B + 17, buffers=2, device=DEV)
    assert pipe.chunk == 5 * B
    for t in (1, 2, 3):
        g = synth.fresh_grad(n, 82, t)
        host[1].copy_(g)
        pipe.step(*host, *hp, t)
        dt8.dt8_adam_step(ref[0], g.to(DEV), *ref[2:], *hp, t, B)
    torch.cuda.synchronize()
    assert pipe.h2d_bytes == n * 10 + 8 * dt8.num_blocks(n, B)
    assert pipe.d2h_bytes == n * 6 + 8 * dt8.num_blocks(n, B)
    for h, d in zip([host[0]] + host[2:], [ref[0]] + ref[2:]):
        assert torch.equal(h, d.cpu())


def _tiny_speaker_net():
    torch.manual_seed(0)
    return torch.nn.Sequential(
        torch.nn.Conv2d(1, 32, 3, padding=1), torch.nn.BatchNorm2d(32), torch.nn.ReLU(),
        torch.nn.Conv2d(32, 64, 3, padding=1), torch.nn.BatchNorm2d(64), torch.nn.ReLU(),
        torch.nn.AdaptiveAvgPool2d(1), torch.nn.Flatten(), torch.nn.Linear(64, 10)).to(DEV)


@pytest.mark.parametrize("kind", ["adamw", "sgd"])
def test_torch_optimizer_front_end_steps_and_resumes(kind):
    """AdamW8bit / SGD8bit on a small conv net: every step equals the pointer-list entry point
    called by hand on copies, and a run resumed from state_dict() continues bit-identically."""
    from paper_2412_01195_b200.optim import AdamW8bit, SGD8bit

    def make(model):
        if kind == "adamw":
            return AdamW8bit(model.parameters(), lr=1e-3, weight_decay=0.05, block_size=256)
        return SGD8bit(model.parameters(), lr=0.05, momentum=0.9, weight_decay=1e-4, block_size=256)

    def batch(i):
        g = torch.Generator(device="cpu").manual_seed(100 + i)
        return torch.randn(8, 1, 16, 16, generator=g).to(DEV), torch.randint(0, 10, (8,), generator=g).to(DEV)

    def train(model, opt, steps):
        # seeded gradients written in place (a real backward pass is not bit-reproducible run to
        # run, which would hide what is being compared here: the optimizer)
        for i in steps:
            for k, prm in enumerate(model.parameters()):
                g = synth.normal(prm.numel(), 1e-2, 7000 + 100 * i + k).view_as(prm).to(DEV)
                if prm.grad is None:
                    prm.grad = g
                else:
                    prm.grad.copy_(g)
            opt.step()

    # reference: the same gradients stepped by hand through the multi-tensor entry point
    model = _tiny_speaker_net()
    opt = make(model)
    ps = [p.detach().clone() for p in model.parameters()]
    B = 256
    sm = [dt8.new_state(p.numel(), B, True, DEV) for p in ps]
    sr = [dt8.new_state(p.numel(), B, False, DEV) for p in ps]
    for i in range(1, 4):
        x, y = batch(i)
        opt.zero_grad(set_to_none=False)
        torch.nn.functional.cross_entropy(model(x), y).backward()
        gs = [p.grad.detach().clone() for p in model.parameters()]
        opt.step()
        flat = lambda ts: [t.view(-1) for t in ts]
        if kind == "adamw":
            dt8.dt8_adam_step_multi(flat(ps), flat(gs), [s[0] for s in sm], [s[1] for s in sm],
                                    [s[0] for s in sr], [s[1] for s in sr], 1e-3, 0.9, 0.999, 1e-8,
                                    0.05, i, B)
        else:
            dt8.dt8_sgd_step_multi(flat(ps), flat(gs), [s[0] for s in sm], [s[1] for s in sm], 0.05,
                                   0.9, 1e-4, i, B)
    torch.cuda.synchronize()
    for p, q in zip(model.parameters(), ps):
        assert torch.equal(p.detach(), q)
    expected = sum(dt8.dt8_state_bytes(p.numel(), B) for p in ps) * (2 if kind == "adamw" else 1)
    assert opt.state_bytes() == expected

    # resume: 3 steps, checkpoint, 2 more steps == 5 steps in one go
    a = _tiny_speaker_net()
    oa = make(a)
    train(a, oa, range(1, 6))
    b = _tiny_speaker_net()
    ob = make(b)
    train(b, ob, range(1, 4))
    ckpt = {"model": {k: v.clone() for k, v in b.state_dict().items()},
            "opt": {"state": {i: {k: (v.clone() if torch.is_tensor(v) else v) for k, v in st.items()}
                              for i, st in ob.state_dict()["state"].items()},
                    "param_groups": ob.state_dict()["param_groups"]}}
    c = _tiny_speaker_net()
    c.load_state_dict(ckpt["model"])
    oc = make(c)
    oc.load_state_dict(ckpt["opt"])
    assert all(st["m_codes"].dtype == torch.uint8 for st in oc.state.values())
    train(c, oc, range(4, 6))
    torch.cuda.synchronize()
    for p, q in zip(a.parameters(), c.parameters()):
        assert torch.equal(p.detach(), q.detach())


def test_more_tensors_than_one_launch_holds():
    """600 small tensors: the pointer list is cut into several launches."""
    B = 256
    sizes = [17 + (i * 37) % 700 for i in range(600)]
    ws = [synth.normal(n, 0.05, 1000 + i) for i, n in enumerate(sizes)]
    gs = [synth.normal(n, 1e-3, 2000 + i) for i, n in enumerate(sizes)]
    w_gpu = [w.to(DEV) for w in ws]
    st = [dt8.new_state(n, B, True, DEV) for n in sizes]
    dt8.dt8_sgd_step_multi(w_gpu, [g.to(DEV) for g in gs], [s[0] for s in st], [s[1] for s in st],
                           0.1, 0.9, 1e-4, 1, B)
    torch.cuda.synchronize()
    for i, n in enumerate(sizes):
        w, mc, ma = to_np(ws[i]), np.full(n, 127, np.uint8), np.zeros(oracle.num_blocks(n, B), F)
        oracle.sgd_step(w, to_np(gs[i]), mc, ma, 0.1, 0.9, 1e-4, 1, B)
        assert np.array_equal(to_np(w_gpu[i]), w) and np.array_equal(to_np(st[i][0]), mc)
        assert np.array_equal(to_np(st[i][1]), ma)


# ------------------------------------------------------------------------------------------------
# memory safety, determinism, resume, streams
# ------------------------------------------------------------------------------------------------
def test_no_write_outside_the_buffers():
    """Canary padding around every buffer, ragged sizes, checked after the kernels ran."""
    B, pad = 1024, 64
    for n in (1, B - 1, 3 * B + 2, 9 * B + 1023):
        nb = dt8.num_blocks(n, B)

        def padded(count, dtype, fill):
            buf = torch.full((count + 2 * pad,), fill, dtype=dtype, device=DEV)
            return buf, buf[pad:pad + count]

        wbuf, w = padded(n, torch.float32, 777.0)
        gbuf, g = padded(n, torch.float32, 777.0)
        mcb, mc = padded(n, torch.uint8, 0xAB)
        rcb, rc = padded(n, torch.uint8, 0xAB)
        mab, ma = padded(nb, torch.float32, 777.0)
        rab, ra = padded(nb, torch.float32, 777.0)
        w.copy_(synth.normal(n, 0.02, 1).to(DEV)); g.copy_(synth.normal(n, 1e-3, 2).to(DEV))
        mc.fill_(127); rc.zero_(); ma.zero_(); ra.zero_()
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, 1e-3, 0.9, 0.999, 1e-8, 0.0, 1, B)
        dt8.dt8_sgd_step(w, g, mc, ma, 0.1, 0.9, 0.0, 1, B)
        dt8.dt8_quantize_blockwise(g, B, True, mc, ma)
        dt8.dt8_dequantize_blockwise(mc, ma, B, True, w)
        torch.cuda.synchronize()
        for buf, fill in ((wbuf, 777.0), (gbuf, 777.0), (mab, 777.0), (rab, 777.0), (mcb, 0xAB), (rcb, 0xAB)):
            assert torch.all(buf[:pad] == fill) and torch.all(buf[-pad:] == fill)


def test_run_to_run_bit_reproducible_and_resume():
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.01)
    n, B = 50 * 2048 + 3, 2048
    w0 = synth.normal(n, 0.02, 1100).to(DEV)
    grads = [synth.fresh_grad(n, 44, t).to(DEV) for t in range(1, 9)]

    def run(snapshot_at=None, resume_from=None):
        if resume_from is None:
            state = [w0.clone(), *dt8.new_state(n, B, True, DEV), *dt8.new_state(n, B, False, DEV)]
            start = 1
        else:
            state, start = [t.clone() for t in resume_from[0]], resume_from[1]
        snap = None
        for t in range(start, 9):
            dt8.dt8_adam_step(state[0], grads[t - 1], *state[1:], *hp, t, B)
            if t == snapshot_at:
                snap = ([x.clone() for x in state], t + 1)
        torch.cuda.synchronize()
        return state, snap

    a, snap = run(snapshot_at=4)
    b, _ = run()
    c, _ = run(resume_from=snap)
    for x, y, z in zip(a, b, c):
        assert torch.equal(x, y) and torch.equal(x, z)


def test_side_stream():
    n, B = 10 * 2048, 2048
    s = torch.cuda.Stream()
    w = synth.normal(n, 0.02, 1200).to(DEV)
    g = synth.normal(n, 1e-3, 1201).to(DEV)
    ref = AdamState(w.cpu(), B)
    ref.step(g.cpu(), 1, dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0))
    mc, ma = dt8.new_state(n, B, True, DEV)
    rc, ra = dt8.new_state(n, B, False, DEV)
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, 1e-3, 0.9, 0.999, 1e-8, 0.0, 1, B)
    s.synchronize()
    assert torch.equal(mc, ref.mc_gpu) and torch.equal(ra, ref.ra_gpu) and torch.equal(w, ref.w_gpu)


# ------------------------------------------------------------------------------------------------
# full size, in the launch configuration the benchmark times
# ------------------------------------------------------------------------------------------------
def test_adam_configuration_5_full_size_sampled_blocks():
    """2^28 elements, 10 warm-up AdamW steps + 1, wd 0.01.  Blocks are independent, so the checker
    follows a fixed subset of blocks (first, last, every 64th) through all 11 steps."""
    c = synth.ADAM_FLAT_LARGE
    n, B = c["n"], c["block_size"]
    nb = n // B
    w, _ = synth.flat_adam_inputs(n, c["seed"], device=DEV)
    mc, ma = dt8.new_state(n, B, True, DEV)
    rc, ra = dt8.new_state(n, B, False, DEV)
    blocks = torch.unique(torch.cat([torch.arange(0, nb, 64), torch.tensor([nb - 1])])).to(DEV)
    idx = (blocks[:, None] * B + torch.arange(B, device=DEV)[None, :]).reshape(-1)
    ns = idx.numel()
    w_ref = to_np(w[idx])
    mc_ref, ma_ref = np.full(ns, 127, np.uint8), np.zeros(ns // B, F)
    rc_ref, ra_ref = np.zeros(ns, np.uint8), np.zeros(ns // B, F)
    for t in range(1, c["prewarm_steps"] + 2):
        g = synth.fresh_grad(n, c["seed"], t, device=DEV)
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, c["lr"], c["beta1"], c["beta2"], c["eps"],
                          c["weight_decay"], t, B)
        oracle.adam_step(w_ref, to_np(g[idx]), mc_ref, ma_ref, rc_ref, ra_ref, c["lr"], c["beta1"],
                         c["beta2"], c["eps"], c["weight_decay"], t, B)
        del g
    torch.cuda.synchronize()
    assert np.array_equal(to_np(ma[blocks]), ma_ref) and np.array_equal(to_np(ra[blocks]), ra_ref)
    assert_codes_match(to_np(mc[idx]), mc_ref)
    assert_codes_match(to_np(rc[idx]), rc_ref)
    assert_params_close(to_np(w[idx]), w_ref, 1e-6)
    # properties that hold for every block at any size
    assert torch.all(ma > 0) and torch.all(ra > 0)
    assert int((mc.view(nb, B) == 255).any(1).logical_or((mc.view(nb, B) == 0).any(1)).sum()) == nb
    assert int((rc.view(nb, B) == 255).any(1).sum()) == nb
    assert not bool((mc == 128).any())


def test_quantize_128m_sampled_blocks():
    """Configuration 4 at 2^27 elements: checker on every 128th block."""
    n = synth.QUANT_SWEEP["sizes"][2]
    x = synth.laplace_outliers(n, seed=3, device=DEV)
    for B in (256, 2048, 4096):
        nb = n // B
        blocks = torch.arange(0, nb, 128, device=DEV)
        idx = (blocks[:, None] * B + torch.arange(B, device=DEV)[None, :]).reshape(-1)
        for signed in (True, False):
            xin = x if signed else x.abs()
            codes, absmax = dt8.dt8_quantize_blockwise(xin, B, signed)
            out = dt8.dt8_dequantize_blockwise(codes, absmax, B, signed)
            rc, ra = oracle.quantize_blockwise(to_np(xin[idx]), B, signed)
            assert np.array_equal(to_np(absmax[blocks]), ra)
            assert_codes_match(to_np(codes[idx]), rc)
            assert np.array_equal(to_np(out[idx]), oracle.dequantize_blockwise(rc, ra, B, signed))
            assert torch.equal(absmax, xin.view(nb, B).abs().amax(1))
            del codes, absmax, out

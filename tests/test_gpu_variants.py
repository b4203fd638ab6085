"""Parity of the variants and corners of the fused steps against the CPU checker, through the C
ABI: the IEEE parameter paths with every gradient type, block size and launch form; bfloat16
parameters; long pointer lists; pointers at their minimum alignment; the benchmark's own loop."""
import numpy as np
import pytest
import torch

import oracle
import paper_2412_01195_b200 as dt8
from paper_2412_01195_b200 import synth
from helpers import (AdamState, SgdState, assert_bf16_params_match, assert_codes_match,
                     assert_params_close, to_np, use_all_cores)

pytestmark = pytest.mark.gpu
F = np.float32
DEV = "cuda"
BC, DW = dt8.DT8_ADAM_BIAS_CORRECTION, dt8.DT8_ADAM_DECOUPLED_WD


@pytest.fixture(scope="module", autouse=True)
def _setup():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    dt8.dt8_init()
    use_all_cores()
    yield
    torch.cuda.synchronize()


# ------------------------------------------------------------------------------------------------
# IEEE parameter paths: coupled decay (bit-exact parameters) and an out-of-range learning rate
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("B", [256, 2048, 4096])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("case", ["coupled", "tiny_lr"])
def test_ieee_parameter_paths(case, gdtype, B):
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.05)
    flags = BC if case == "coupled" else (BC | DW)
    if case == "tiny_lr":
        hp["lr"] = 1e-25
    n = 9 * B + B // 2 + 3
    st = AdamState(synth.normal(n, 0.02, 1200 + B), B)
    for t in range(1, 8):
        g = synth.fresh_grad(n, 120, t, dtype=gdtype)
        if t == 3:
            g = g.clone()
            g[2 * B:3 * B] = 0                        # a block whose first moment decays only
            g[4 * B:4 * B + 7] = g[4 * B:4 * B + 7] * 1e-22   # dividends below the fast range
        st.step(g, t, hp, flags)
    st.check(exact_params=True)


@pytest.mark.parametrize("eps", [0.0, 1e-8, 3.0e13, 4.0e13, 1e30])
def test_ieee_update_across_the_edges_of_its_fast_range(eps):
    """The IEEE parameter update replaces the library root and divisions by corrected
    approximations only while every moment of a thread lies in 2^-60 .. 2^60 and eps is at most
    2^45 (3.5e13); blocks of gradients from 1e-30 to 1e15 put moments below, inside, on both sides
    of the edges of, and above that range, and the eps values sit on both sides of its limit.  The
    parameters must equal the checker's bit for bit wherever the update ran."""
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=eps, weight_decay=1e-3)
    B = 2048
    scales = [1e-30, 1e-15, 1e-12, 1e-9, 3e-9, 1e-7, 1e-3, 1.0, 1e3, 1e8, 1e10, 3e10, 1e11, 1e15]
    if eps == 0.0:
        scales[0] = scales[1] = 1e-12     # a squared gradient that underflows to 0 would divide by zero
    n = len(scales) * B + 77
    w0 = synth.normal(n, 1.0, 1250)
    scale = torch.ones(n)
    for k, s in enumerate(scales):
        scale[k * B:(k + 1) * B] = s
    # one block mixes magnitudes inside a thread's sixteen values
    scale[7 * B:8 * B:5] = 1e-12
    st = AdamState(w0 * scale, B)
    for t in range(1, 5):
        st.step(synth.fresh_grad(n, 125, t) * scale, t, hp, BC)
    st.check(exact_params=True)


@pytest.mark.parametrize("B", [256, 2048])
def test_states_of_very_small_and_very_large_gradients(B):
    """Blocks whose maxima leave the range of the reciprocal-and-correct normalisation (below
    2^-76, above 2^100) take the IEEE division, a block of zeros stays zeros, and both can meet in
    one block: a gradient of 1e-30 gives a first moment of 1e-31 and a second moment that
    underflows to exactly 0.  Codes and maxima must equal the checker's; SGD likewise."""
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    scales = [1e-41, 1e-38, 1e-36, 1e-30, 1e-25, 1e-20, 1e-12, 1.0, 1e12, 1e16, 1e18]
    n = len(scales) * B + 5
    scale = torch.ones(n)
    for k, s in enumerate(scales):
        scale[k * B:(k + 1) * B] = s
    st = AdamState(synth.normal(n, 0.02, 1260), B)
    sg = SgdState(synth.normal(n, 0.02, 1261), B)
    sg_small = SgdState(synth.normal(n, 0.02, 1262), B)
    for t in range(1, 5):
        g = synth.fresh_grad(n, 126, t) * scale
        st.step(g, t, hp)
        sg.step(g * 1e14, t, dict(lr=1e-3, momentum=0.9, weight_decay=0.0))
        sg_small.step(g, t, dict(lr=1e-3, momentum=0.9, weight_decay=0.0))
    st.check()
    sg.check()
    sg_small.check()


def test_coupled_decay_from_the_zero_state_with_zero_gradients():
    """All-zero groups (dividend 0) take the IEEE division inside the IEEE path."""
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    n, B = 3 * 2048, 2048
    st = AdamState(synth.normal(n, 0.02, 1300), B)
    g = torch.zeros(n)
    g[5] = 1e-3
    hp["weight_decay"] = 0.1
    for t in (1, 2):
        st.step(g, t, hp, BC)
    st.check(exact_params=True)


@pytest.mark.parametrize("flags", [BC, 0])
def test_ieee_paths_through_the_pointer_list(flags):
    B = 512
    sizes = [7, B, 5 * B + 1, 33 * B + 100]
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.05)
    ws = [synth.normal(n, 0.02, 1400 + i) for i, n in enumerate(sizes)]
    sts = [AdamState(w, B) for w in ws]
    for t in (1, 2, 3):
        gs = [synth.fresh_grad(n, 140 + i, t, dtype=torch.bfloat16) for i, n in enumerate(sizes)]
        dt8.dt8_adam_step_multi([s.w_gpu for s in sts], [g.to(DEV) for g in gs], [s.mc_gpu for s in sts],
                                [s.ma_gpu for s in sts], [s.rc_gpu for s in sts], [s.ra_gpu for s in sts],
                                *hp, t, B, flags)
        for s, g in zip(sts, gs):
            oracle.adam_step(s.w, to_np(g), s.mc, s.ma, s.rc, s.ra, *hp, t, B, flags)
    for s in sts:
        s.check(exact_params=True)


# ------------------------------------------------------------------------------------------------
# bfloat16 parameters without a 32-bit copy
# ------------------------------------------------------------------------------------------------
def bf16_param(n, seed):
    return synth.normal(n, 0.02, seed).to(torch.bfloat16)


@pytest.mark.parametrize("B", [256, 2048])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_adam_with_bf16_parameters(gdtype, B):
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    for n in (1, 3, B - 1, 6 * B + 5, 70 * B + B // 2 + 2):
        st = AdamState(bf16_param(n, 1500 + B), B)
        for t in range(1, 6):
            st.step(synth.fresh_grad(n, 150, t, dtype=gdtype), t, hp)
            st.check()                                  # states exact; <= 1e-4 of params one bf16 ulp off
    # coupled decay: IEEE parameter arithmetic, so the rounded parameters are exact too
    st = AdamState(bf16_param(20 * B + 9, 1501), B)
    for t in range(1, 6):
        st.step(synth.fresh_grad(20 * B + 9, 151, t, dtype=gdtype), t, hp, BC)
    st.check(exact_params=True)


@pytest.mark.parametrize("B", [256, 1024, 4096])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_sgd_with_bf16_parameters(gdtype, B):
    hp = dict(lr=0.1, momentum=0.9, weight_decay=1e-4)
    for n in (2, B + 1, 9 * B + 13, 64 * B + 3):
        st = SgdState(bf16_param(n, 1600 + B), B)
        for t in range(1, 6):
            st.step(synth.student_t(n, 3, 1e-3, 1610 + t).to(gdtype), t, hp)
            st.check()                                  # SGD is IEEE throughout: everything exact


def test_bf16_parameters_through_the_pointer_list():
    B = 2048
    sizes = [32, 300, B, 3 * B + 1, 50 * B + 77]
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.05)
    sts = [AdamState(bf16_param(n, 1700 + i), B) for i, n in enumerate(sizes)]
    prepared = dt8.PreparedTensorList([s.w_gpu for s in sts], [torch.empty(n, device=DEV) for n in sizes],
                                      [s.mc_gpu for s in sts], [s.ma_gpu for s in sts],
                                      [s.rc_gpu for s in sts], [s.ra_gpu for s in sts])
    for t in (1, 2, 3):
        gs = [synth.fresh_grad(n, 170 + i, t) for i, n in enumerate(sizes)]
        for buf, g in zip(prepared._keep[1], gs):
            buf.copy_(g)
        prepared.adam_step(*hp, t, B)
        for s, g in zip(sts, gs):
            oracle.adam_step(s.w, to_np(g), s.mc, s.ma, s.rc, s.ra, *hp, t, B)
    for s in sts:
        s.check()
    with pytest.raises(TypeError):
        dt8.dt8_adam_step_multi([sts[0].w_gpu, torch.zeros(32, device=DEV)], [torch.zeros(32, device=DEV)] * 2,
                                [sts[0].mc_gpu] * 2, [sts[0].ma_gpu] * 2, [sts[0].rc_gpu] * 2,
                                [sts[0].ra_gpu] * 2, *hp, 1, B)


# ------------------------------------------------------------------------------------------------
# long pointer lists, minimum alignment, the benchmark's loop
# ------------------------------------------------------------------------------------------------
def test_adam_pointer_list_longer_than_one_launch():
    """600 tensors: three launches of at most 256 tensors each; equal to the checker tensor by tensor."""
    B = 256
    rng = np.random.default_rng(18)
    sizes = [int(v) for v in rng.integers(1, 3 * B, 600)]
    sizes[100] = 0
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.01)
    sts = [AdamState(synth.normal(n, 0.02, 1800 + i), B) for i, n in enumerate(sizes)]
    for t in (1, 2):
        gs = [synth.fresh_grad(n, 1800 + i, t) for i, n in enumerate(sizes)]
        dt8.dt8_adam_step_multi([s.w_gpu for s in sts], [g.to(DEV) for g in gs], [s.mc_gpu for s in sts],
                                [s.ma_gpu for s in sts], [s.rc_gpu for s in sts], [s.ra_gpu for s in sts],
                                *hp, t, B)
        for s, g in zip(sts, gs):
            oracle.adam_step(s.w, to_np(g), s.mc, s.ma, s.rc, s.ra, *hp, t, B)
    for s in sts:
        s.check()


def _carve(pool: torch.Tensor, offset_bytes: int, n: int, dtype):
    """n elements of `dtype` starting `offset_bytes` into a uint8 pool (a view, no copy)."""
    size = n * torch.empty(0, dtype=dtype).element_size()
    return pool[offset_bytes:offset_bytes + size].view(dtype)


@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_pointers_at_their_minimum_alignment(gdtype):
    """Parameters at a 16-byte-only offset, bf16 gradients at an 8-byte-only offset, codes and
    block maxima at 4-byte-only offsets; a canary pattern around every buffer must survive."""
    B, n = 256, 11 * 256 + 37
    nb = dt8.num_blocks(n, B)
    pool = torch.full((1 << 20,), 0xA5, dtype=torch.uint8, device=DEV)
    assert pool.data_ptr() % 256 == 0
    goff = 4096 + (16 if gdtype == torch.float32 else 8)
    w = _carve(pool, 1024 + 16, n, torch.float32)
    g = _carve(pool, 65536 + goff, n, gdtype)
    mc = _carve(pool, 131072 + 4, n, torch.uint8)
    rc = _carve(pool, 196608 + 12, n, torch.uint8)
    ma = _carve(pool, 262144 + 4, nb, torch.float32)
    ra = _carve(pool, 327680 + 12, nb, torch.float32)
    w0 = synth.normal(n, 0.02, 1900)
    w.copy_(w0)
    mc.fill_(127)
    rc.zero_()
    ma.zero_()
    ra.zero_()
    ref = AdamState(w0, B)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    for t in (1, 2, 3):
        gt = synth.fresh_grad(n, 190, t, dtype=gdtype)
        g.copy_(gt)
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                          hp["weight_decay"], t, B)
        oracle.adam_step(ref.w, to_np(gt), ref.mc, ref.ma, ref.rc, ref.ra, hp["lr"], hp["beta1"],
                         hp["beta2"], hp["eps"], hp["weight_decay"], t, B)
    torch.cuda.synchronize()
    assert np.array_equal(to_np(ma), ref.ma) and np.array_equal(to_np(ra), ref.ra)
    assert_codes_match(to_np(mc), ref.mc)
    assert_codes_match(to_np(rc), ref.rc)
    assert_params_close(to_np(w), ref.w)
    # everything outside the six buffers still holds the canary
    mask = torch.ones(pool.numel(), dtype=torch.bool, device=DEV)
    for t_ in (w, g, mc, rc, ma, ra):
        lo = t_.data_ptr() - pool.data_ptr()
        mask[lo:lo + t_.numel() * t_.element_size()] = False
    assert bool(torch.all(pool[mask] == 0xA5))
    # SGD with the same minimum offsets
    w.copy_(w0)
    mc.fill_(127)
    ma.zero_()
    sref = SgdState(w0, B)
    for t in (1, 2):
        gt = synth.fresh_grad(n, 191, t, dtype=gdtype)
        g.copy_(gt)
        dt8.dt8_sgd_step(w, g, mc, ma, 0.1, 0.9, 1e-4, t, B)
        oracle.sgd_step(sref.w, to_np(gt), sref.mc, sref.ma, 0.1, 0.9, 1e-4, t, B)
    torch.cuda.synchronize()
    assert np.array_equal(to_np(w), sref.w) and np.array_equal(to_np(mc), sref.mc)
    assert bool(torch.all(pool[mask] == 0xA5))


def test_the_benchmark_loop_on_sampled_blocks():
    """bench.py's own sequence at reduced length: 10 pre-warm steps with fresh gradients, then 25
    steps that reuse one gradient tensor; checked on sampled blocks (blocks are independent, so
    the checker can run the sampled ones alone)."""
    c = synth.ADAM_FLAT_LARGE
    B, n = c["block_size"], 1 << 22
    hp = (c["lr"], c["beta1"], c["beta2"], c["eps"], c["weight_decay"])
    w, g = synth.flat_adam_inputs(n, c["seed"], device=DEV)
    mc, ma = dt8.new_state(n, B, True, DEV)
    rc, ra = dt8.new_state(n, B, False, DEV)
    blocks = sorted({0, 1, 777, n // B - 1, *range(5, n // B, 97)})
    idx = np.concatenate([np.arange(b * B, (b + 1) * B) for b in blocks])
    w_ref, g_ref = to_np(w)[idx], to_np(g)[idx]
    nbs = len(blocks)
    s_ref = [np.full(idx.size, 127, np.uint8), np.zeros(nbs, F), np.zeros(idx.size, np.uint8), np.zeros(nbs, F)]
    step = 0
    for _ in range(c["prewarm_steps"]):
        step += 1
        gt = synth.fresh_grad(n, c["seed"], step, device=DEV)
        dt8.dt8_adam_step(w, gt, mc, ma, rc, ra, *hp, step, B)
        oracle.adam_step(w_ref, to_np(gt)[idx], *s_ref, *hp, step, B)
    for _ in range(25):
        step += 1
        dt8.dt8_adam_step(w, g, mc, ma, rc, ra, *hp, step, B)
        oracle.adam_step(w_ref, g_ref, *s_ref, *hp, step, B)
    torch.cuda.synchronize()
    assert np.array_equal(to_np(ma)[blocks], s_ref[1]) and np.array_equal(to_np(ra)[blocks], s_ref[3])
    assert_codes_match(to_np(mc)[idx], s_ref[0])
    assert_codes_match(to_np(rc)[idx], s_ref[2])
    assert_params_close(to_np(w)[idx], w_ref, 1e-6)


# ------------------------------------------------------------------------------------------------
# the constant-divisor division of the IEEE Adam update
# ------------------------------------------------------------------------------------------------
def test_division_by_the_bias_corrections_is_correctly_rounded():
    """m'/(1 - beta1^t) and r'/(1 - beta2^t) use a host-made reciprocal and a residual correction
    instead of the IEEE division.  For every divisor of that form that a run can meet -- beta 0.9
    (t up to where 1 - beta^t rounds to 1), beta 0.999 (t = 1 .. 2000 and 200 steps spread up to
    1e6), a few other betas, and 1 (no bias correction) -- the routine must return the correctly
    rounded quotient: all 2^23 mantissas of the dividend in two binades for a sample of the
    divisors, 2^18 random dividends for each of the others, plus dividends outside the fast range
    (zero, tiny, huge), which take the IEEE division.  The reference is the binary64 quotient
    rounded once (a quotient of two binary32 numbers is never a binary32 rounding boundary)."""
    def bc(beta, t):
        return float(np.float32(1.0 - float(np.float32(beta)) ** t))
    divisors = {1.0}
    for t in range(1, 200):
        divisors.add(bc(0.9, t))
    for t in list(range(1, 2001)) + [int(v) for v in np.logspace(3.3, 6, 200)]:
        divisors.add(bc(0.999, t))
    for beta in (0.5, 0.8, 0.95, 0.98, 0.99, 0.9999):
        for t in (1, 2, 3, 10, 100, 1000):
            divisors.add(bc(beta, t))
    divisors = sorted(d for d in divisors if d > 0)
    assert len(divisors) > 2000
    gen = torch.Generator(device=DEV).manual_seed(77)
    man = torch.arange(1 << 23, dtype=torch.int32, device=DEV)
    full = torch.cat([(man | 0x3F800000).view(torch.float32), (man | 0x40000000).view(torch.float32)])
    rnd_bits = torch.randint(0, 1 << 23, (1 << 18,), generator=gen, device=DEV, dtype=torch.int32)
    expo = torch.randint(90, 160, (1 << 18,), generator=gen, device=DEV, dtype=torch.int32) << 23
    sign = torch.randint(0, 2, (1 << 18,), generator=gen, device=DEV, dtype=torch.int32) << 31
    rnd = (rnd_bits | expo | sign).view(torch.float32)
    edge = torch.tensor([0.0, -0.0, 1e-30, -1e-30, 1e-38, 1e-42, 3e38, -3e38, 2.0 ** -60, 2.0 ** 60,
                         2.0 ** -61, 2.0 ** 61], device=DEV)
    rnd = torch.cat([rnd, edge])
    out_full, out_rnd = torch.empty_like(full), torch.empty_like(rnd)
    for i, d in enumerate(divisors):
        s, out = (full, out_full) if i % 64 == 0 else (rnd, out_rnd)
        got = dt8.dt8_selfcheck_divide_const(s, d, out)
        ref = (s.double() / d).float()
        bad = torch.nonzero(got.view(torch.int32) != ref.view(torch.int32)).flatten()
        assert bad.numel() == 0, (d, s[bad[:4]].tolist(), got[bad[:4]].tolist(), ref[bad[:4]].tolist())
    # divisors outside the range of the routine take the IEEE division
    for d in (2.0 ** -25, 3.0e7, float(np.float32(1.2e-7))):
        got = dt8.dt8_selfcheck_divide_const(rnd, d, out_rnd)
        assert torch.equal(got.view(torch.int32), (rnd.double() / d).float().view(torch.int32))


def test_optimizer_front_end_with_bf16_parameters_steps_and_resumes():
    """AdamW8bit on bfloat16 parameters: equal to the pointer-list entry point called by hand, and
    a run resumed from state_dict() continues bit-identically (codes stay uint8, block maxima
    fp32 through the round trip)."""
    from paper_2412_01195_b200.optim import AdamW8bit
    sizes = [(64, 33), (300,), (5, 7, 3, 3)]
    B = 256

    def params():
        return [torch.nn.Parameter(synth.normal(int(np.prod(s)), 0.05, 2100 + i).reshape(s).to(torch.bfloat16).to(DEV))
                for i, s in enumerate(sizes)]

    def grads(step):
        # torch wants a gradient of the parameter's dtype
        return [synth.normal(int(np.prod(s)), 1e-2, 2200 + 10 * step + i).reshape(s).to(torch.bfloat16).to(DEV)
                for i, s in enumerate(sizes)]

    def run(ps, opt, steps):
        for t in steps:
            for p, g in zip(ps, grads(t)):
                if p.grad is None:
                    p.grad = g.clone()
                else:
                    p.grad.copy_(g)
            opt.step()

    pa = params()
    oa = AdamW8bit(pa, lr=1e-3, weight_decay=0.05, block_size=B)
    run(pa, oa, range(1, 6))
    # by hand
    ph = [p.detach().clone().view(-1) for p in params()]
    sm = [dt8.new_state(p.numel(), B, True, DEV) for p in ph]
    sr = [dt8.new_state(p.numel(), B, False, DEV) for p in ph]
    for t in range(1, 6):
        dt8.dt8_adam_step_multi(ph, [g.view(-1) for g in grads(t)], [s[0] for s in sm], [s[1] for s in sm],
                                [s[0] for s in sr], [s[1] for s in sr], 1e-3, 0.9, 0.999, 1e-8, 0.05, t, B)
    torch.cuda.synchronize()
    for p, q in zip(pa, ph):
        assert p.dtype == torch.bfloat16 and torch.equal(p.detach().view(-1), q)
    # resume after 3 of the 5 steps
    pb = params()
    ob = AdamW8bit(pb, lr=1e-3, weight_decay=0.05, block_size=B)
    run(pb, ob, range(1, 4))
    sd = ob.state_dict()
    pc = [torch.nn.Parameter(p.detach().clone()) for p in pb]
    oc = AdamW8bit(pc, lr=1e-3, weight_decay=0.05, block_size=B)
    oc.load_state_dict(sd)
    assert all(st["m_codes"].dtype == torch.uint8 and st["r_absmax"].dtype == torch.float32 for st in oc.state.values())
    run(pc, oc, range(4, 6))
    torch.cuda.synchronize()
    for p, q in zip(pa, pc):
        assert torch.equal(p.detach(), q.detach())
